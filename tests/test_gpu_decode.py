"""Parity of the CUDA decode step (still_hybrid_attn_step) with the CPU oracle, and
prefill -> decode consistency."""
import numpy as np
import pytest
import torch

import paper_2602_02180_b200 as still
from oracle import still_oracle as oracle
from paper_2602_02180_b200 import synth
from tests import util_parity as U

pytestmark = pytest.mark.gpu


def _decode_case(w, n0, n_steps, gate=False, tweak=None):
    """Prefill n0 tokens into a state, decode n_steps more, compare every decoded row with
    the oracle's chunk-wise form over the whole sequence (the GPU's selection forced)."""
    dev = "cuda"
    N = n0 + n_steps
    wN = w.with_(N=N)
    Q, K, V = synth.make_qkv(wN, dev)
    if tweak is not None:
        Q, K, V = tweak(Q, K, V)
    Wq, Wk = synth.make_npmap_weights(wN, dev)
    G = synth.make_gate(wN, dev) if gate else None
    p = U.params_of(w)
    cap = N + 5
    lay = still.state_layout(p, cap)
    state = torch.zeros(lay["total"], dtype=torch.uint8, device=dev)
    if n0 > 0:
        still.hybrid_attn_fwd(p, Q[:, :, :n0].contiguous(), K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous(),
                              Wq, Wk, G=None if G is None else G[:, :, :n0].contiguous(), state=state,
                              state_max_tokens=cap)
    else:
        # an empty prefill initialises the state
        c = p.c()
        import ctypes
        rc = still.binding.lib().still_hybrid_attn_fwd(
            ctypes.byref(c), 0, None, None, None, None, None, None, None, None, None, None, None,
            ctypes.c_void_p(state.data_ptr()), cap, None, 0, None)
        assert rc == 0
    ys = []
    for t in range(n0, N):
        y = still.hybrid_attn_step(p, state, cap, t, Q[:, :, t].contiguous(), K[:, :, t].contiguous(),
                                   V[:, :, t].contiguous(), Wq, Wk,
                                   g=None if G is None else G[:, :, t].contiguous())
        ys.append(y)
    torch.cuda.synchronize()
    assert still.device_status(state) == (0, 0)
    Yd = torch.stack(ys, dim=2)  # [B,H,n_steps,d]
    C, lam = w.C, w.k
    capT = lay["capacity"] // C
    sc = state[lay["score"]: lay["score"] + w.B * w.H * lay["capacity"] * 4].view(torch.float32).view(w.B, w.H, -1)
    n_routed = max(0, (N - 1) // C - 1)  # chunks 0..c_last-2 have been routed
    sel = None
    if lam > 0:
        sel = state[lay["sel_idx"]: lay["sel_idx"] + w.B * w.H * capT * lam * 4].view(torch.int32).view(w.B, w.H, capT, lam)
    rep = w.H // w.Hkv
    rows = list(range(n0, N))
    hp = oracle.HeadParams(C, lam, w.sm_scale)
    T = -(-N // C)
    for b, h in U.sample_heads(w, 4):
        kv = h // rep
        scores = sc[b, h, :N].cpu().numpy().astype(np.float64)
        forced = None
        if lam > 0:
            want = oracle.select(scores, C, lam)
            got = sel[b, h, :n_routed].cpu().numpy()
            np.testing.assert_array_equal(got, want[:n_routed])  # bit-exact on the GPU's own scores
            forced = want.copy()
            forced[:n_routed] = got
        out = oracle.chunkwise(U.f64(Q[b, h]), U.f64(K[b, kv]), U.f64(V[b, kv]), U.f64(Wq[h]), U.f64(Wk[kv]), hp,
                               g=None if G is None else U.f64(G[b, h]), forced_idx=forced, rows=rows)
        assert np.abs(scores - out["score"]).max() < (1e-4 if w.dtype == "fp32" else 1e-3)
        err = np.abs(U.f64(Yd[b, h]) - out["y"]).max()
        assert err <= U.TOL[w.torch_dtype], f"b={b} h={h} max-abs {err:.3e}"


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize(
    "B,H,Hkv,d,C,k,n0,steps",
    [
        (2, 4, 2, 64, 32, 8, 100, 80),     # prefill ends mid-chunk, several routings during decode
        (1, 4, 1, 128, 64, 16, 192, 70),   # prefill ends on a chunk boundary
        (1, 2, 2, 64, 32, 0, 70, 40),      # lambda = 0
        (1, 8, 2, 128, 64, 64, 130, 66),   # lambda = C
        (1, 2, 1, 64, 32, 8, 0, 100),      # decode from an empty state
        (1, 2, 2, 128, 128, 32, 300, 90),
        (1, 16, 1, 64, 32, 8, 90, 50),     # sixteen query heads on one KV head
        (1, 12, 2, 128, 64, 16, 200, 70),  # six heads per group
    ],
)
def test_decode_matches_oracle(dtype, B, H, Hkv, d, C, k, n0, steps):
    w = synth.Workload("t", B, H, Hkv, d, n0, C, k, dtype, "iid", 999)
    _decode_case(w, n0, steps, gate=(k not in (0, C)))


@pytest.mark.parametrize("k", [64, 16])
def test_decode_with_growing_logits(k):
    # Logits that grow by ~7 nats per 128 tokens and one dominant key: the partial results of the key splits
    # differ by many orders of magnitude and the merge has to bring them to one reference.
    def tweak(Q, K, V):
        t = torch.arange(Q.shape[2], device=Q.device)
        Q, K = Q.float(), K.float()
        Q[..., 0] += 8.0
        K[..., 0] += (10.0 * (t // 128)).view(1, 1, -1)
        K[:, :, 128 * 3 + 100, 0] += 60.0
        return Q.to(torch.bfloat16), K.to(torch.bfloat16), V

    w = synth.Workload("t", 2, 4, 2, 128, 0, 64, k, "bf16", "iid", 77)
    _decode_case(w, 128 * 5 + 9, 70, tweak=tweak)


def test_c5_full_size_sampled():
    # The decode workload as benchmarked: batch 64, 32768-token prefix summarised by the prefill into the
    # decode state, then a few steps; sampled (batch, head) pairs against the oracle.
    w = synth.WORKLOADS["c5"]
    _decode_case(w, w.N, 3)


def test_state_full_and_mismatch():
    w = synth.Workload("t", 1, 2, 2, 64, 64, 32, 8, "bf16", "iid", 5)
    p = U.params_of(w)
    Q, K, V = synth.make_qkv(w, "cuda")
    Wq, Wk = synth.make_npmap_weights(w, "cuda")
    state = torch.zeros(still.state_bytes(p, 64), dtype=torch.uint8, device="cuda")
    still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, state=state, state_max_tokens=64)
    q, k, v = synth.make_decode_inputs(w, 0, "cuda")
    with pytest.raises(still.StillError) as e:
        still.hybrid_attn_step(p, state, 64, 64, q, k, v, Wq, Wk)
    assert e.value.code == -4
    # a wrong t_pos is recorded in the state's status word, the context stays usable
    state2 = torch.zeros(still.state_bytes(p, 128), dtype=torch.uint8, device="cuda")
    still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, state=state2, state_max_tokens=128)
    still.hybrid_attn_step(p, state2, 128, 70, q, k, v, Wq, Wk)
    assert still.device_status(state2)[0] == -7
