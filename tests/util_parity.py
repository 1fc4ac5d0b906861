"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI and the CPU
oracle on the same (dtype-rounded) inputs and compare."""
from __future__ import annotations

import numpy as np
import torch

import paper_2602_02180_b200 as still
from oracle import still_oracle as oracle
from paper_2602_02180_b200 import synth

TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}  # max-abs on Y, per dtype
# max-abs on the Self-Saliency Score against the oracle's (same rounded inputs on both sides; the kernels
# use the hardware's approximate exp2 / log2, and scores reach log((1 + eps) / eps) = 13.8)
SCORE_TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-3}


def f64(t):
    return t.detach().to("cpu", torch.float32).numpy().astype(np.float64)


def params_of(w: synth.Workload, **kw) -> still.StillParams:
    return still.StillParams(w.B, w.H, w.Hkv, w.d, w.C, w.k, w.torch_dtype, d_f=w.d_f, sm_scale=w.sm_scale, **kw)


def check_selection(scores, sel_idx, C, lam, heads):
    """sel_idx must equal the oracle's selection applied to the GPU's own scores, bit for bit."""
    sc = scores.cpu().numpy()
    si = sel_idx.cpu().numpy()
    for b, h in heads:
        want = oracle.select(sc[b, h].astype(np.float64), C, lam)
        np.testing.assert_array_equal(si[b, h], want, err_msg=f"selection differs at b={b} h={h}")


def jaccard(a, b):
    """Mean Jaccard index over chunks of two [T, lam] selections (-1 = padding)."""
    vals = []
    for ra, rb in zip(np.asarray(a), np.asarray(b)):
        sa, sb = set(ra[ra >= 0].tolist()), set(rb[rb >= 0].tolist())
        if sa or sb:
            vals.append(len(sa & sb) / len(sa | sb))
    return float(np.mean(vals)) if vals else 1.0


def check_outputs(w, Q, K, V, Wq, Wk, Y, scores, sel_idx, heads, rows=None, G=None, bq=None, bk=None,
                  tol=None, eps=1e-6, score_tol=None, report=None, max_salient=0):
    """Y of the sampled heads (and rows) against the oracle run with the GPU's selection, and the GPU's
    scores against the oracle's.  Returns (worst Y error, worst score error); `report`, if a dict, also
    receives the Jaccard agreement between the oracle's own selection and the GPU's (reported, not gated:
    near-ties may flip)."""
    tol = TOL[w.torch_dtype] if tol is None else tol
    score_tol = SCORE_TOL[w.torch_dtype] if score_tol is None else score_tol
    rep = w.H // w.Hkv
    p = oracle.HeadParams(w.C, w.k, w.sm_scale, eps, max_salient=max_salient)
    worst = 0.0
    score_err = 0.0
    for b, h in heads:
        kv = h // rep
        out = oracle.chunkwise(
            f64(Q[b, h]), f64(K[b, kv]), f64(V[b, kv]), f64(Wq[h]), f64(Wk[kv]), p,
            g=None if G is None else f64(G[b, h]),
            bq=None if bq is None else f64(bq[h]), bk=None if bk is None else f64(bk[kv]),
            forced_idx=sel_idx[b, h].cpu().numpy() if w.k > 0 else None, rows=rows,
        )
        got = f64(Y[b, h]) if rows is None else f64(Y[b, h][torch.as_tensor(rows, device=Y.device)])
        assert np.all(np.isfinite(got)), f"non-finite output at b={b} h={h}"
        err = np.abs(got - out["y"]).max()
        worst = max(worst, err)
        serr = np.abs(scores[b, h].cpu().numpy() - out["score"]).max()
        score_err = max(score_err, serr)
        assert err <= tol, f"b={b} h={h}: max-abs {err:.3e} > {tol}"
        assert serr <= score_tol, f"b={b} h={h}: score max-abs {serr:.3e} > {score_tol}"
        if report is not None and w.k > 0:
            pure = oracle.select(out["score"], w.C, w.k)
            report.setdefault("jaccard", []).append(jaccard(pure, sel_idx[b, h].cpu().numpy()))
    return worst, score_err


def run_prefill(w, device="cuda", gate=False, bias=False, max_salient=0, **fwd_kw):
    Q, K, V = synth.make_qkv(w, device)
    Wq, Wk = synth.make_npmap_weights(w, device)
    G = synth.make_gate(w, device) if gate else None
    bq = bk = None
    if bias:
        g = torch.Generator(device=device).manual_seed(w.seed + 77)
        bq = (torch.randn(w.H, w.d_f, generator=g, device=device) * 0.05).to(w.torch_dtype)
        bk = (torch.randn(w.Hkv, w.d_f, generator=g, device=device) * 0.05).to(w.torch_dtype)
    p = params_of(w, max_salient=max_salient)
    Y, scores, sel = still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, G=G, bq=bq, bk=bk, **fwd_kw)
    torch.cuda.synchronize()
    return dict(p=p, Q=Q, K=K, V=V, Wq=Wq, Wk=Wk, G=G, bq=bq, bk=bk, Y=Y, scores=scores, sel=sel)


def sample_heads(w, n, seed=0):
    rng = np.random.default_rng(seed)
    allh = [(b, h) for b in range(w.B) for h in range(w.H)]
    if n >= len(allh):
        return allh
    pick = rng.choice(len(allh), size=n, replace=False)
    return [allh[i] for i in sorted(pick)]


def sample_rows(N, n, C, seed=0):
    """Rows spread over the sequence, always including chunk edges, the first and the last rows."""
    rng = np.random.default_rng(seed)
    fixed = {0, min(N - 1, C - 1), min(N - 1, C), min(N - 1, 2 * C), min(N - 1, 2 * C + 1), N - 1, max(0, N - C)}
    rest = set(rng.choice(N, size=min(N, n), replace=False).tolist())
    return sorted(fixed | rest)
