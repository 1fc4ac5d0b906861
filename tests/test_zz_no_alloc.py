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
    for call in range(2):  # the second call finds the first call's contents in the shared array
        (wy, wsc, wsel), (y, sc, sel) = _both(w, seed_shift=call)
        assert torch.isfinite(y.float()).all()
        assert torch.equal(sel, wsel), f"call {call}: selection differs"
        assert (sc - wsc).abs().max().item() <= 1e-6, f"call {call}: scores differ"
        err = (y.float() - wy.float()).abs().max().item()
        assert err <= tol, f"call {call}: max-abs {err:.3e} > {tol}"


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
