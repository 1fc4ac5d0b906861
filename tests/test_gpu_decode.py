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


def _decode_case(w, n0, n_steps, gate=False, tweak=None, expect_ties=False, n_heads=4, want_y=True, max_salient=0):
    """Prefill n0 tokens into a state, decode n_steps more, compare every decoded row of the sampled heads
    with the oracle's chunk-wise form over the whole sequence (the GPU's selection forced)."""
    dev = "cuda"
    N = n0 + n_steps
    wN = w.with_(N=N)
    Q, K, V = synth.make_qkv(wN, dev)
    if tweak is not None:
        Q, K, V = tweak(Q, K, V)
    Wq, Wk = synth.make_npmap_weights(wN, dev)
    G = synth.make_gate(wN, dev) if gate else None
    rep = w.H // w.Hkv
    heads = U.sample_heads(w, n_heads)
    # what the oracle needs of the sampled heads, and the decode steps' inputs; the whole-sequence device
    # tensors go before the prefill allocates its workspace (the full-size case would not fit otherwise)
    host = {(b, h): (U.f64(Q[b, h]), U.f64(K[b, h // rep]), U.f64(V[b, h // rep]),
                     None if G is None else U.f64(G[b, h])) for b, h in heads}
    step_in = [t[:, :, n0:].permute(2, 0, 1, 3).contiguous() if t is not None else None for t in (Q, K, V, G)]  # [steps,B,heads,d]
    pre = [t[:, :, :n0].contiguous() if t is not None else None for t in (Q, K, V, G)]
    del Q, K, V, G
    p = U.params_of(w, max_salient=max_salient)
    cap = N + 5
    lay = still.state_layout(p, cap)
    state = torch.zeros(lay["total"], dtype=torch.uint8, device=dev)
    if n0 > 0:
        still.hybrid_attn_fwd(p, pre[0], pre[1], pre[2], Wq, Wk, G=pre[3], state=state, state_max_tokens=cap,
                              want_y=want_y)
    else:
        # an empty prefill initialises the state
        c = p.c()
        import ctypes
        rc = still.binding.lib().still_hybrid_attn_fwd(
            ctypes.byref(c), 0, None, None, None, None, None, None, None, None, None, None, None,
            ctypes.c_void_p(state.data_ptr()), cap, None, 0, None)
        assert rc == 0
    torch.cuda.synchronize()
    del pre
    torch.cuda.empty_cache()
    ys = []
    for i in range(n_steps):
        y = still.hybrid_attn_step(p, state, cap, n0 + i, step_in[0][i], step_in[1][i], step_in[2][i], Wq, Wk,
                                   g=None if step_in[3] is None else step_in[3][i])
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
    rows = list(range(n0, N))
    hp = oracle.HeadParams(C, lam, w.sm_scale, max_salient=max_salient)
    tie_seen = False
    worst = 0.0
    for b, h in heads:
        kv = h // rep
        q64, k64, v64, g64 = host[(b, h)]
        scores = sc[b, h, :N].cpu().numpy().astype(np.float64)
        if expect_ties and n_routed > 0:
            ch = np.sort(scores[: n_routed * C].reshape(n_routed, C)[n0 // C:], axis=1)   # chunks routed by decode steps
            tie_seen |= bool(np.any(np.diff(ch, axis=1) == 0))
        forced = None
        if lam > 0:
            want = oracle.select(scores, C, lam)
            got = sel[b, h, :n_routed].cpu().numpy()
            np.testing.assert_array_equal(got, want[:n_routed])  # bit-exact on the GPU's own scores
            forced = want.copy()
            forced[:n_routed] = got
        out = oracle.chunkwise(q64, k64, v64, U.f64(Wq[h]), U.f64(Wk[kv]), hp, g=g64, forced_idx=forced, rows=rows)
        serr = np.abs(scores - out["score"]).max()
        assert serr <= U.SCORE_TOL[w.torch_dtype], f"b={b} h={h} score max-abs {serr:.3e}"
        err = np.abs(U.f64(Yd[b, h]) - out["y"]).max()
        worst = max(worst, err)
        assert err <= U.TOL[w.torch_dtype], f"b={b} h={h} max-abs {err:.3e}"
    assert tie_seen or not expect_ties, "the constructed input produced no tie in a chunk routed by a decode step"
    return worst


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
        (1, 2, 1, 128, 64, 16, 64 * 36 + 5, 70),   # long prefill on few heads: the state comes out of a segmented scan
    ],
)
def test_decode_matches_oracle(dtype, B, H, Hkv, d, C, k, n0, steps):
    w = synth.Workload("t", B, H, Hkv, d, n0, C, k, dtype, "iid", 999)
    _decode_case(w, n0, steps, gate=(k not in (0, C)))


@pytest.mark.parametrize("B,H,Hkv,d,C,k,budget,n0,steps", [
    (1, 4, 2, 128, 64, 16, 48, 64 * 7 + 11, 64 * 3 + 9),     # prefill already past the budget, three routings while decoding
    (2, 2, 1, 64, 64, 8, 16, 72, 64 * 7),                    # the budget is reached during the decode
    (1, 2, 2, 128, 64, 64, 128, 64 * 5, 64 * 2 + 5),         # every token selected: sliding window + linear state
    (1, 2, 1, 64, 64, 8, 8, 0, 64 * 6),                      # from an empty state
])
def test_decode_with_a_salient_cache_budget(B, H, Hkv, d, C, k, budget, n0, steps):
    # Tokens that a newly routed chunk pushes out of the capped salient cache are folded into (S, z) at that step,
    # and the split-KV pass reads only the chunks still cached.
    w = synth.Workload("t", B, H, Hkv, d, n0, C, k, "bf16", "iid", 4711)
    _decode_case(w, n0, steps, gate=True, max_salient=budget)


def test_budgeted_state_size_does_not_grow_with_the_sequence():
    # with a budget the K / V store of the state is a ring over the cached chunks, the local region and the chunk
    # being routed; what still grows with the capacity are 4-byte scores and the per-chunk index tables
    free = still.StillParams(8, 32, 8, 128, 64, 16)
    capped = still.StillParams(8, 32, 8, 128, 64, 16, max_salient=448)
    small, big = still.state_bytes(capped, 4096), still.state_bytes(capped, 65536)
    assert still.state_bytes(free, 65536) > 12 * still.state_bytes(free, 4096) > 0
    kv_ring = 8 * 8 * (448 // 16 + 3) * 64 * 128 * 2 * 2
    assert big - small < 0.1 * still.state_bytes(free, 65536) and small > kv_ring and big < 3 * small


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


@pytest.mark.parametrize("dtype,C,k", [("bf16", 64, 16), ("bf16", 32, 8), ("fp32", 32, 8)])
@pytest.mark.parametrize("case", ["zero_queries", "periodic_tokens"])
def test_decode_routing_breaks_ties_like_the_oracle(dtype, C, k, case):
    # Equal scores inside a chunk (all logits zero, or tokens repeating with period 16): the chunk routed at a
    # decode step must be ranked under (score descending, position ascending), as the prefill does.
    def tweak(Q, K, V):
        if case == "zero_queries":
            return torch.zeros_like(Q), K, V
        reps = -(-Q.shape[2] // 16)
        rep = lambda x: x[:, :, :16].repeat(1, 1, reps, 1)[:, :, : x.shape[2]].contiguous()  # noqa: E731
        return rep(Q), rep(K), V

    w = synth.Workload("t", 1, 4, 2, 64, 0, C, k, dtype, "iid", 31)
    _decode_case(w, C + 7, 4 * C + 3, tweak=tweak, expect_ties=True)


@pytest.mark.parametrize("k,steps", [(64, 256), (16, 136)])
def test_c5_full_size_sampled(k, steps):
    # The decode workload as benchmarked: batch 64, 32768-token prefix summarised by the prefill into the
    # decode state, then the benchmark's 256 steps (four chunks are routed on the way) with every token
    # selected, and 136 steps (two routings) of the lambda = C/4 companion; sampled (batch, head) pairs
    # against the oracle.
    w = synth.WORKLOADS["c5"].with_(k=k)
    _decode_case(w, w.N, steps, n_heads=4 if k == 64 else 3, want_y=False)


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
    # a wrong t_pos is recorded in the state's status word; the step writes nothing else (state bytes and y
    # unchanged), the context stays usable, and later steps on that state are no-ops until it is rebuilt
    state2 = torch.zeros(still.state_bytes(p, 128), dtype=torch.uint8, device="cuda")
    still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, state=state2, state_max_tokens=128)
    before = state2.clone()
    y = torch.full((w.B, w.H, w.d), 7.0, dtype=w.torch_dtype, device="cuda")
    still.hybrid_attn_step(p, state2, 128, 70, q, k, v, Wq, Wk, y=y)
    assert still.device_status(state2) == (-7, 1)
    still.hybrid_attn_step(p, state2, 128, 64, q, k, v, Wq, Wk, y=y)   # the right position, but the state is flagged
    assert still.device_status(state2) == (-7, 1)
    same = state2 == before
    same[14 * 4: 16 * 4] = True    # the status and detail words
    assert bool(same.all()) and bool((y == 7.0).all())
    # a state built with other parameters (another topk): detail 3
    p_other = U.params_of(w.with_(k=4))
    state3 = torch.zeros(still.state_bytes(p, 128), dtype=torch.uint8, device="cuda")
    still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, state=state3, state_max_tokens=128)
    if still.state_bytes(p_other, 128) <= state3.numel():
        still.hybrid_attn_step(p_other, state3, 128, 64, q, k, v, Wq, Wk, y=y)
        assert still.device_status(state3) == (-7, 3)
    # and the ordinary path still works
    still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, state=state2, state_max_tokens=128)
    still.hybrid_attn_step(p, state2, 128, 64, q, k, v, Wq, Wk, y=y)
    assert still.device_status(state2) == (0, 0) and torch.isfinite(y.float()).all()
