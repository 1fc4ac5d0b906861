"""still_hybrid_attn_fwd_static against still_hybrid_attn_fwd.

The static variant is for callers that cannot allocate device memory (code running inside another
runtime's fixed memory plan, or where cudaMalloc is not allowed): its workspace is an array inside
the library.  It must give what the ordinary entry point gives, on every call, although all calls
share that array and find the previous call's leftovers in it.  The file name keeps this test last
in collection order; it must also pass when run alone in a fresh process.
"""
import pytest
import torch

import paper_2602_02180_b200 as still
from paper_2602_02180_b200 import synth
from tests import util_parity as U

pytestmark = pytest.mark.gpu


def _both(w, seed_shift):
    w = w.with_(seed=w.seed + seed_shift)
    Q, K, V = synth.make_qkv(w, "cuda")
    Wq, Wk = synth.make_npmap_weights(w, "cuda")
    G = synth.make_gate(w, "cuda")
    p = U.params_of(w)
    assert 0 < still.workspace_bytes(p, w.N) <= still.binding.STATIC_WORKSPACE_BYTES
    want_Y, want_sc, want_sel = still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, G=G)
    T = -(-w.N // w.C)
    Y = torch.full_like(Q, float("nan"))
    sc = torch.full((w.B, w.H, w.N), float("nan"), dtype=torch.float32, device="cuda")
    sel = torch.full((w.B, w.H, T, w.k), -7, dtype=torch.int32, device="cuda")
    still.hybrid_attn_fwd_static(p, Q, K, V, Wq, Wk, G=G, Y=Y, scores=sc, sel_idx=sel)
    torch.cuda.synchronize()
    return (want_Y, want_sc, want_sel), (Y, sc, sel)


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_static_workspace_matches_the_ordinary_prefill_twice(dtype):
    # ragged length, grouped KV heads, lambda < C so that every workspace part is in use
    w = synth.Workload("na", 1, 4, 2, 64, 64 * 9 + 23, 64, 16, dtype, "iid", 31337)
    tol = U.TOL[w.torch_dtype]
    # Leftovers that matter: a longer call of the other dtype first, so that the array holds foreign bytes
    # beyond every part the calls below write (tile padding of the compacted rows, the linear branch's
    # numerator / denominator), not just their own earlier results.
    other = w.with_(dtype="fp32" if dtype == "bf16" else "bf16", N=64 * 13 + 5, k=8, seed=99)
    _both(other, seed_shift=0)
    for call in range(2):  # the second call finds the first call's contents in the shared array
        (wy, wsc, wsel), (y, sc, sel) = _both(w, seed_shift=call)
        assert torch.isfinite(y.float()).all()
        assert torch.equal(sel, wsel), f"call {call}: selection differs"
        assert (sc - wsc).abs().max().item() <= 1e-6, f"call {call}: scores differ"
        err = (y.float() - wy.float()).abs().max().item()
        assert err <= tol, f"call {call}: max-abs {err:.3e} > {tol}"


def test_static_entry_point_allocates_nothing():
    # The point of the entry point: a caller whose device memory is fixed must see none of it taken.  Every
    # buffer is made beforehand; around the calls neither torch's allocator nor the device's free memory moves.
    w = synth.Workload("na", 1, 4, 2, 64, 64 * 7 + 9, 64, 16, "bf16", "iid", 4711)
    Q, K, V = synth.make_qkv(w, "cuda")
    Wq, Wk = synth.make_npmap_weights(w, "cuda")
    p = U.params_of(w)
    T = -(-w.N // w.C)
    Y = torch.empty_like(Q)
    sc = torch.empty(w.B, w.H, w.N, dtype=torch.float32, device="cuda")
    sel = torch.empty(w.B, w.H, T, w.k, dtype=torch.int32, device="cuda")
    still.hybrid_attn_fwd_static(p, Q, K, V, Wq, Wk, Y=Y, scores=sc, sel_idx=sel)   # first call: address look-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        still.hybrid_attn_fwd_static(p, Q, K, V, Wq, Wk, Y=Y, scores=sc, sel_idx=sel)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    assert free1 >= free0, f"device memory shrank by {free0 - free1} bytes across calls that may not allocate"
    # invalid parameters are rejected also for an empty sequence
    with pytest.raises(still.StillError):
        still.hybrid_attn_fwd_static(still.StillParams(1, 3, 2, 64, 64, 16), Q[:, :, :0], K[:, :, :0], V[:, :, :0],
                                     Wq, Wk, Y=Y, scores=sc, sel_idx=sel)


def test_static_workspace_rejects_what_does_not_fit():
    w = synth.Workload("na", 1, 8, 8, 128, 16384, 64, 16, "bf16", "iid", 5)
    p = U.params_of(w)
    assert still.workspace_bytes(p, w.N) > still.binding.STATIC_WORKSPACE_BYTES
    x = torch.zeros(1, 8, w.N, 128, dtype=torch.bfloat16, device="cuda")
    T = w.N // w.C
    with pytest.raises(still.StillError) as e:
        still.hybrid_attn_fwd_static(p, x, x, x, None, None, Y=torch.empty_like(x),
                                     scores=torch.empty(1, 8, w.N, device="cuda"),
                                     sel_idx=torch.empty(1, 8, T, 16, dtype=torch.int32, device="cuda"))
    assert e.value.code == -3
