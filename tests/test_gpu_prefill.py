"""Parity of the CUDA prefill (still_hybrid_attn_fwd, through the C ABI) with the CPU oracle."""
import numpy as np
import pytest
import torch

import paper_2602_02180_b200 as still
from paper_2602_02180_b200 import synth
from tests import util_parity as U

pytestmark = pytest.mark.gpu


def _small(name, dtype, B, H, Hkv, d, N, C, k, recipe="iid", seed=1):
    return synth.Workload(name, B, H, Hkv, d, N, C, k, dtype, recipe, 4242 + seed)


def test_c1_fp32_every_row():
    w = synth.WORKLOADS["c1"]
    r = U.run_prefill(w)
    heads = U.sample_heads(w, 99)
    U.check_selection(r["scores"], r["sel"], w.C, w.k, heads)
    worst, serr = U.check_outputs(w, r["Q"], r["K"], r["V"], r["Wq"], r["Wk"], r["Y"], r["scores"], r["sel"], heads)
    assert serr < 1e-4
    print(f"c1 max-abs {worst:.2e} score err {serr:.2e}")


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize(
    "B,H,Hkv,d,N,C,k",
    [
        (1, 2, 1, 64, 200, 32, 8),      # ragged tail, GQA
        (2, 4, 2, 64, 64 * 5 + 17, 64, 16),
        (1, 4, 4, 128, 128 * 3 + 1, 128, 32),
        (1, 2, 2, 64, 300, 64, 0),      # lambda = 0: local softmax + linear attention
        (1, 2, 1, 128, 333, 64, 1),
        (1, 2, 2, 64, 260, 64, 64),     # lambda = C: causal softmax attention
        (1, 2, 1, 128, 40, 64, 16),     # shorter than one chunk
        (1, 1, 1, 64, 1, 32, 4),        # a single token
        (1, 8, 2, 128, 128 * 4, 128, 128),
        (1, 4, 2, 64, 128 * 3 + 70, 128, 32),   # d = 64 with C = 128: two 64-token sub-chunks per chunk
        (1, 2, 1, 128, 64 * 40 + 17, 64, 16),   # many chunks, few heads: the state scan runs as four segments
        (1, 2, 2, 64, 128 * 33 + 5, 128, 32),   # the same with two sub-chunks per chunk (two segments)
    ],
)
def test_small_shapes(dtype, B, H, Hkv, d, N, C, k):
    w = _small("t", dtype, B, H, Hkv, d, N, C, k)
    r = U.run_prefill(w, gate=True, bias=True)
    heads = U.sample_heads(w, 4)
    if k:
        U.check_selection(r["scores"], r["sel"], C, k, heads)
    U.check_outputs(w, r["Q"], r["K"], r["V"], r["Wq"], r["Wk"], r["Y"], r["scores"], r["sel"], heads,
                    G=r["G"], bq=r["bq"], bk=r["bk"])


@pytest.mark.parametrize(
    "B,H,Hkv,d,N,C,k,budget",
    [
        (1, 4, 2, 128, 64 * 12 + 9, 64, 16, 48),      # three chunks' selections stay cached
        (2, 2, 1, 64, 128 * 9 + 40, 128, 32, 64),     # two sub-chunks per chunk
        (1, 2, 2, 128, 64 * 10 + 3, 64, 64, 128),     # every token selected: a sliding window of two chunks + linear state
        (1, 2, 1, 128, 64 * 40 + 17, 64, 16, 64),     # the state scan in four segments
        (1, 4, 2, 128, 64 * 9, 64, 16, 16 * 64),      # a budget that is never reached
        (1, 2, 2, 64, 64 * 30, 64, 8, 8),             # a single chunk's selections
    ],
)
def test_salient_cache_budget(B, H, Hkv, d, N, C, k, budget):
    # max_salient: per head at most `budget` selected tokens stay in the softmax branch; the oldest leave for the
    # linear state when a newly routed chunk pushes them out (this library's rule; the paper caps the cache
    # without stating one).  The oracle applies the same rule.
    w = _small("t", "bf16", B, H, Hkv, d, N, C, k)
    r = U.run_prefill(w, gate=True, max_salient=budget)
    heads = U.sample_heads(w, 4)
    U.check_selection(r["scores"], r["sel"], C, k, heads)
    U.check_outputs(w, r["Q"], r["K"], r["V"], r["Wq"], r["Wk"], r["Y"], r["scores"], r["sel"], heads, G=r["G"],
                    max_salient=budget)
    if budget >= (N // C) * k:   # never reached: the same bits as without a budget
        free = U.run_prefill(w, gate=True)
        assert torch.equal(free["Y"], r["Y"])


def test_salient_cache_budget_must_be_whole_chunks_of_selections():
    p = still.StillParams(1, 2, 2, 64, 64, 16, max_salient=40)
    assert still.workspace_bytes(p, 256) == 0
    assert still.workspace_bytes(still.StillParams(1, 2, 2, 64, 64, 16, torch.float32, max_salient=32), 256) == 0   # FMA path
    assert still.workspace_bytes(still.StillParams(1, 2, 2, 64, 64, 16, max_salient=32), 256) > 0


def _has_tie(scores, C):
    """True when some chunk holds two equal finite scores (so the tie arm of the ranking decided)."""
    sc = scores.cpu().numpy()
    n = sc.shape[-1] // C * C
    ch = np.sort(sc[..., :n].reshape(-1, C), axis=1)
    return bool(np.any((np.diff(ch, axis=1) == 0) & np.isfinite(ch[:, 1:])))


@pytest.mark.parametrize("dtype,d,C,k", [("bf16", 128, 64, 16), ("bf16", 64, 128, 32), ("bf16", 64, 64, 64 - 1),
                                         ("bf16", 64, 32, 8), ("fp32", 64, 64, 16), ("fp32", 128, 32, 8)])
@pytest.mark.parametrize("case", ["zero_queries", "periodic_tokens", "nan_key"])
def test_constructed_ties_and_nan_rank_like_the_oracle(dtype, d, C, k, case):
    # Top-lambda under the total order (score descending, position ascending), NaN lowest: the tie arm of the
    # ranking only runs when two scores of a chunk are equal, which random inputs never produce.
    #   zero_queries     every logit is 0, so every full window has the same score: whole chunks tie
    #   periodic_tokens  q, k repeat with period 16: tokens 16 apart see the same window contents
    #   nan_key          one key is NaN: the C rows whose window holds it have NaN scores
    w = _small("t", dtype, 1, 4, 2, d, C * 6 + C // 2 + 3, C, k)
    Q, K, V = synth.make_qkv(w, "cuda")
    if case == "zero_queries":
        Q = torch.zeros_like(Q)
    elif case == "periodic_tokens":
        reps = -(-w.N // 16)
        Q = Q[:, :, :16].repeat(1, 1, reps, 1)[:, :, : w.N].contiguous()
        K = K[:, :, :16].repeat(1, 1, reps, 1)[:, :, : w.N].contiguous()
    else:
        K = K.clone()
        K[0, 1, 2 * C + 5, 3] = float("nan")
    Wq, Wk = synth.make_npmap_weights(w, "cuda")
    Y, scores, sel = still.hybrid_attn_fwd(U.params_of(w), Q, K, V, Wq, Wk)
    torch.cuda.synchronize()
    heads = U.sample_heads(w, 99)
    U.check_selection(scores, sel, C, k, heads)
    if case == "nan_key":
        sc = scores.cpu().numpy()
        assert np.isnan(sc[0, 2:, 2 * C + 5: 3 * C + 5]).all() and np.isfinite(sc[0, :2]).all()
        assert np.isfinite(sc[0, 2:, : 2 * C + 5]).all() and np.isfinite(sc[0, 2:, 3 * C + 5:]).all()
        # a NaN score ranks below every number: the five finite rows of the chunk (positions 2C .. 2C+4) are
        # taken before any of its NaN rows
        picked = sel[0, 2:, 2].cpu().numpy()
        n_finite = 5
        assert ((picked < 2 * C + 5) & (picked >= 0)).sum(axis=1).min() == min(k, n_finite)
        heads = [(0, 0), (0, 1)]   # the heads of the KV head without the NaN stay finite and are compared
    else:
        assert _has_tie(scores, C), "the constructed input produced no tie"
    U.check_outputs(w, Q, K, V, Wq, Wk, Y, scores, sel, heads)


def test_feature_width_smaller_than_head_dim():
    # d_f = 64 with d = 128: feature dim d' = 128 (other template instance of the NP-Map and scan kernels)
    w = _small("t", "bf16", 1, 4, 2, 128, 64 * 7 + 5, 64, 16)
    Q, K, V = synth.make_qkv(w, "cuda")
    g = torch.Generator(device="cuda").manual_seed(11)
    Wq = (torch.randn(w.H, w.d, 64, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    Wk = (torch.randn(w.Hkv, w.d, 64, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    p = still.StillParams(w.B, w.H, w.Hkv, w.d, w.C, w.k, torch.bfloat16, d_f=64)
    Y, scores, sel = still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk)
    torch.cuda.synchronize()
    heads = U.sample_heads(w, 4)
    U.check_selection(scores, sel, w.C, w.k, heads)
    U.check_outputs(w, Q, K, V, Wq, Wk, Y, scores, sel, heads)


def test_paper_literal_scale_one():
    # sm_scale = 1 is the main text's exp(q k^T); inputs are scaled down so the softmaxes stay soft.
    w = _small("t", "fp32", 1, 2, 2, 64, 256, 64, 16)
    Q, K, V = synth.make_qkv(w, "cuda")
    Q, K = Q * 0.35, K * 0.35
    Wq, Wk = synth.make_npmap_weights(w, "cuda")
    p = still.StillParams(w.B, w.H, w.Hkv, w.d, w.C, w.k, torch.float32, sm_scale=1.0)
    Y, scores, sel = still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk)
    heads = U.sample_heads(w, 2)
    U.check_selection(scores, sel, w.C, w.k, heads)
    from oracle import still_oracle as oracle
    for b, h in heads:
        out = oracle.chunkwise(U.f64(Q[b, h]), U.f64(K[b, h]), U.f64(V[b, h]), U.f64(Wq[h]), U.f64(Wk[h]),
                               oracle.HeadParams(w.C, w.k, 1.0), forced_idx=sel[b, h].cpu().numpy())
        assert np.abs(U.f64(Y[b, h]) - out["y"]).max() < 1e-4


@pytest.mark.parametrize("k", [64, 16])
def test_growing_logits_rescale_the_accumulator(k):
    # The tensor-core kernel keeps a row's softmax reference until a tile's maximum exceeds it by 2^8 and then
    # rescales the output accumulator.  Logits that grow by ~7 nats per 128-key tile, plus one key far above the
    # rest in the second half of a tile, make that happen in every tile and in both halves.
    w = _small("t", "bf16", 1, 4, 2, 128, 128 * 7 + 40, 64, k)
    Q, K, V = synth.make_qkv(w, "cuda")
    t = torch.arange(w.N, device="cuda")
    Q = Q.float()
    K = K.float()
    Q[..., 0] += 8.0
    K[..., 0] += (10.0 * (t // 128)).view(1, 1, -1)
    K[:, :, 128 * 3 + 100, 0] += 60.0
    Q, K = Q.to(torch.bfloat16), K.to(torch.bfloat16)
    Wq, Wk = synth.make_npmap_weights(w, "cuda")
    Y, scores, sel = still.hybrid_attn_fwd(U.params_of(w), Q, K, V, Wq, Wk)
    torch.cuda.synchronize()
    assert torch.isfinite(Y.float()).all()
    heads = U.sample_heads(w, 4)
    U.check_selection(scores, sel, w.C, w.k, heads)
    U.check_outputs(w, Q, K, V, Wq, Wk, Y, scores, sel, heads)


def test_run_to_run_determinism():
    w = _small("t", "bf16", 1, 4, 2, 64, 500, 64, 16)
    a = U.run_prefill(w)
    b = U.run_prefill(w)
    assert torch.equal(a["Y"], b["Y"]) and torch.equal(a["sel"], b["sel"]) and torch.equal(a["scores"], b["scores"])


def test_constant_value_rows():
    # y is a positive-weight average of the values: constant V gives constant y (gate = 1).
    w = _small("t", "fp32", 1, 2, 2, 64, 320, 64, 16)
    Q, K, V = synth.make_qkv(w, "cuda")
    V = torch.ones_like(V) * 0.75
    Wq, Wk = synth.make_npmap_weights(w, "cuda")
    Y, _, _ = still.hybrid_attn_fwd(U.params_of(w), Q, K, V, Wq, Wk)
    assert (Y - 0.75).abs().max().item() < 1e-5


def test_c2_sampled():
    w = synth.WORKLOADS["c2"]
    r = U.run_prefill(w)
    heads = U.sample_heads(w, 6, seed=2)
    rows = U.sample_rows(w.N, 96, w.C, seed=2)
    U.check_selection(r["scores"], r["sel"], w.C, w.k, heads)
    worst, serr = U.check_outputs(w, r["Q"], r["K"], r["V"], r["Wq"], r["Wk"], r["Y"], r["scores"], r["sel"],
                                  heads, rows=rows)
    print(f"c2 max-abs {worst:.2e} score err {serr:.2e}")
    # companion with a non-degenerate selection (lambda = C/4)
    w4 = w.with_(k=w.C // 4)
    r = U.run_prefill(w4)
    U.check_selection(r["scores"], r["sel"], w4.C, w4.k, heads)
    U.check_outputs(w4, r["Q"], r["K"], r["V"], r["Wq"], r["Wk"], r["Y"], r["scores"], r["sel"], heads, rows=rows)


@pytest.mark.parametrize("name,n_heads,n_rows", [("c3", 3, 40), ("c4", 2, 24)])
def test_full_size_workloads_sampled(name, n_heads, n_rows):
    # The benchmark's own shapes and launch configuration; the oracle checks sampled heads and rows
    # (all O(N) steps -- scores, selection -- in full for those heads).
    w = synth.WORKLOADS[name]
    r = U.run_prefill(w)
    assert still.device_status is not None
    heads = U.sample_heads(w, n_heads, seed=3)
    rows = set(U.sample_rows(w.N, n_rows, w.C, seed=3))
    # rows that sit on a key of unusual norm (c3: the 5x outlier keys, c4: the heavy tail) and the rows right
    # after one, where that key dominates the window: the positions these workloads exist for
    for b, h in heads:
        kn = r["K"][b, h // (w.H // w.Hkv)].float().norm(dim=-1)
        top = torch.topk(kn, 4).indices.cpu().tolist()
        for t in top:
            rows.update(x for x in (t, t + 1, t + w.C - 1, t + w.C, t + 2 * w.C) if x < w.N)
    rows = sorted(rows)
    U.check_selection(r["scores"], r["sel"], w.C, w.k, heads)
    rep = {}
    worst, serr = U.check_outputs(w, r["Q"], r["K"], r["V"], r["Wq"], r["Wk"], r["Y"], r["scores"], r["sel"],
                                  heads, rows=rows, report=rep)
    print(f"{name} max-abs {worst:.2e} score err {serr:.2e} on {len(rows)} rows of {len(heads)} heads; "
          f"selection Jaccard (oracle's own vs GPU) {np.mean(rep['jaccard']):.4f}")


def test_c3_companion_quarter_selection_sampled():
    # lambda = C / 4 at the 32K shape: selection, NP-Map, state scan and merge at scale
    w = synth.WORKLOADS["c3"].with_(B=1, k=16)
    r = U.run_prefill(w)
    heads = U.sample_heads(w, 2, seed=4)
    rows = U.sample_rows(w.N, 32, w.C, seed=4)
    U.check_selection(r["scores"], r["sel"], w.C, w.k, heads)
    rep = {}
    worst, serr = U.check_outputs(w, r["Q"], r["K"], r["V"], r["Wq"], r["Wk"], r["Y"], r["scores"], r["sel"],
                                  heads, rows=rows, report=rep)
    print(f"c3 k16 max-abs {worst:.2e} score err {serr:.2e}; selection Jaccard (oracle's own vs GPU) "
          f"{np.mean(rep['jaccard']):.4f}")


def test_invalid_arguments_are_rejected():
    w = _small("t", "bf16", 1, 2, 2, 64, 128, 64, 16)
    Q, K, V = synth.make_qkv(w, "cuda")
    Wq, Wk = synth.make_npmap_weights(w, "cuda")
    p = U.params_of(w)
    with pytest.raises(still.StillError) as e:
        still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, workspace=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -3
    bad = still.StillParams(1, 3, 2, 64, 64, 16)
    assert still.workspace_bytes(bad, 128) == 0
    with pytest.raises(still.StillError):
        still.hybrid_attn_fwd(still.StillParams(1, 2, 2, 64, 64, 65), Q, K, V, Wq, Wk,
                              workspace=torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))
    ws = torch.empty(still.workspace_bytes(p, 128) + 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(still.StillError) as e:  # misaligned workspace pointer
        still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, workspace=ws[1:])
    assert e.value.code == -1


def test_bounded_device_wait_runs_out_and_is_reported():
    # The tensor-core kernels wait on mbarriers with a cycle limit; when a wait runs out the kernel records
    # STILL_ERR_DEVICE_TIMEOUT in the status block and returns.  The self-test kernel is that wait alone, on a
    # barrier nothing arrives on, with a limit of about a millisecond: it must come back, report (-6, 99) and
    # leave the context usable.
    block = torch.full((256,), 0x5A, dtype=torch.uint8, device="cuda")
    still.selftest_wait_timeout(block, 2_000_000)
    assert still.device_status(block) == (-6, 99)
    w = _small("t", "bf16", 1, 2, 2, 64, 300, 64, 16)
    r = U.run_prefill(w)
    assert torch.isfinite(r["Y"].float()).all()
    ws = torch.empty(still.workspace_bytes(r["p"], w.N), dtype=torch.uint8, device="cuda")
    still.hybrid_attn_fwd(r["p"], r["Q"], r["K"], r["V"], r["Wq"], r["Wk"], workspace=ws)
    assert still.device_status(ws) == (0, 0)
