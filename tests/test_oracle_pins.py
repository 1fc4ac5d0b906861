"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's formula and compares it with itself:
each one is a closed form, an invariant, a special case that reduces to a
library routine (scipy softmax, torch scaled_dot_product_attention, numpy
cumsum), or a brute-force evaluation from the set definitions on tiny inputs.
The paper prints no worked numeric example of the layer, so there is no golden
fixture to load.
"""
import math

import numpy as np
import pytest
import scipy.special as sps
import torch

from oracle import still_oracle as o

RNG = np.random.default_rng(1234)


def _rand_head(N, d, df=None, scale=1.0, rng=RNG):
    df = df or d
    q, k, v = rng.standard_normal((3, N, d)) * scale
    Wq = rng.standard_normal((d, df)) * 0.3
    Wk = rng.standard_normal((d, df)) * 0.3
    return q, k, v, Wq, Wk


# --------------------------------------------------------------------------- score


def _equal_logit_score(n, eps):
    """All logits equal in a window of n tokens: a_diag = 1/n, a_nodiag = 1/(n-1)."""
    if n == 1:
        return math.log((1 + eps) / eps)
    a = 1.0 / n
    return (n - 1) * a * math.log((a + eps) / (1.0 / (n - 1) + eps)) + a * math.log((a + eps) / eps)


@pytest.mark.parametrize("fn", ["token", "chunk"])
@pytest.mark.parametrize("C,N", [(4, 11), (8, 8), (5, 23)])
def test_score_equal_logits_closed_form(fn, C, N):
    # q = 0 makes every logit equal, so the window size alone fixes the score:
    # this catches any off-by-one in W_t = {max(1,t-w+1)..t} (Sec. 3.1).
    d, eps = 3, 1e-6
    q = np.zeros((N, d))
    k = RNG.standard_normal((N, d))
    got = o.score_tokenwise(q, k, C, 1.0, eps) if fn == "token" else o.score_chunkwise(q, k, C, 1.0, eps)
    want = np.array([_equal_logit_score(min(t + 1, C), eps) for t in range(N)])
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("fn", ["token", "chunk"])
def test_score_two_token_window_closed_form(fn):
    # Token 2 sees {1, 2}: a_diag = (1-p, p) with p = sigmoid(l_22 - l_21), a_nodiag = (1, 0).
    eps = 1e-5
    q = np.array([[0.3, -1.0], [0.7, 0.4]])
    k = np.array([[1.2, 0.5], [-0.6, 2.0]])
    s = (o.score_tokenwise if fn == "token" else o.score_chunkwise)(q, k, 4, 1.0, eps)
    l21, l22 = q[1] @ k[0], q[1] @ k[1]
    p = 1.0 / (1.0 + math.exp(l21 - l22))
    want = (1 - p) * math.log((1 - p + eps) / (1 + eps)) + p * math.log((p + eps) / eps)
    assert s[0] == pytest.approx(math.log((1 + eps) / eps), rel=1e-13)
    assert s[1] == pytest.approx(want, rel=1e-12)


@pytest.mark.parametrize("fn", ["token", "chunk"])
def test_score_is_function_of_self_weight(fn):
    # a_nodiag_j = a_diag_j / (1 - p) for j != t, so as eps -> 0 the score tends to
    # (1-p) log(1-p) + p log((p+eps)/eps), p = the token's own softmax weight in its window.
    N, d, C, eps, scale = 64, 16, 16, 1e-9, 16 ** -0.5
    q, k, *_ = _rand_head(N, d)
    s = (o.score_tokenwise if fn == "token" else o.score_chunkwise)(q, k, C, scale, eps)
    for t in range(1, N):
        lo = max(0, t - C + 1)
        p = sps.softmax(scale * (k[lo : t + 1] @ q[t]))[-1]
        want = (1 - p) * math.log1p(-p) + p * math.log((p + eps) / eps)
        assert s[t] == pytest.approx(want, abs=1e-6), t
    assert np.all(s > -1e-6)  # a smoothed KL divergence


def test_score_sm_scale_is_applied_to_logits():
    q, k, *_ = _rand_head(20, 4)
    a = o.score_tokenwise(q, k, 8, 0.25)
    b = o.score_tokenwise(0.25 * q, k, 8, 1.0)
    np.testing.assert_allclose(a, b, rtol=1e-12)


def test_score_two_formulations_agree():
    for N, C in [(37, 8), (64, 16), (5, 8), (16, 16)]:
        q, k, *_ = _rand_head(N, 8, scale=2.0)
        np.testing.assert_allclose(
            o.score_tokenwise(q, k, C, 0.5), o.score_chunkwise(q, k, C, 0.5), rtol=1e-10, atol=1e-12
        )


def test_global_score_is_the_window_score_with_an_unbounded_window():
    # Sec. 3.1 compares the local score with its full-context variant, W_t = {1..t}.  While the sequence is no
    # longer than the window the two coincide (token-wise and chunk-wise forms alike); beyond that they differ;
    # with equal logits the global score of token t is the closed form for a window of t tokens.
    N, d, C = 24, 6, 32
    q, k, _, _, _ = _rand_head(N, d)
    g = o.score_global(q, k, 0.4)
    np.testing.assert_allclose(g, o.score_tokenwise(q, k, C, 0.4), rtol=1e-12)
    np.testing.assert_allclose(g, o.score_chunkwise(q, k, C, 0.4), rtol=1e-10)
    short = o.score_tokenwise(q, k, 8, 0.4)
    np.testing.assert_allclose(g[:8], short[:8], rtol=1e-12)
    assert np.abs(g[8:] - short[8:]).max() > 1e-6
    eps = 1e-6
    flat = o.score_global(np.zeros((N, d)), k, 1.0, eps)
    np.testing.assert_allclose(flat, [_equal_logit_score(t + 1, eps) for t in range(N)], rtol=1e-9)


# --------------------------------------------------------------------------- selection


def _select_reference(score, C, lam):
    N = len(score)
    T = -(-N // C)
    out = np.full((T, lam), -1, dtype=np.int32)
    for c in range(T):
        pos = np.arange(c * C, min(N, (c + 1) * C))
        key = np.where(np.isnan(score[pos]), -np.inf, score[pos])
        order = np.lexsort((pos, -key))  # primary: score descending, secondary: index ascending
        chosen = np.sort(pos[order[: min(lam, len(pos))]])
        out[c, : len(chosen)] = chosen
    return out


@pytest.mark.parametrize("C,lam,N", [(8, 3, 50), (8, 8, 24), (8, 1, 8), (16, 4, 16 * 5 + 3), (4, 4, 6)])
def test_select_matches_sort(C, lam, N):
    score = RNG.standard_normal(N)
    np.testing.assert_array_equal(o.select(score, C, lam), _select_reference(score, C, lam))


def test_select_ties_nan_and_ragged_tail():
    C, lam = 8, 3
    score = np.array([1.0, 5, 5, 5, 5, 0, 0, 0, np.nan, np.nan, -np.inf, np.nan, 2.0, 2.0])
    idx = o.select(score, C, lam)
    np.testing.assert_array_equal(idx[0], [1, 2, 3])  # four-way tie: smallest indices win
    np.testing.assert_array_equal(idx[1], [8, 12, 13])  # NaN ranks with -inf, index breaks the tie
    np.testing.assert_array_equal(idx, _select_reference(score, C, lam))
    short = o.select(np.array([3.0, 1.0]), 8, 4)  # chunk shorter than lambda: take all, pad with -1
    np.testing.assert_array_equal(short, [[0, 1, -1, -1]])


def test_select_partition_sizes():
    N, C, lam = 100, 16, 5
    idx = o.select(RNG.standard_normal(N), C, lam)
    for c in range(idx.shape[0]):
        n_c = min(C, N - c * C)
        sel = idx[c][idx[c] >= 0]
        assert len(sel) == min(lam, n_c)
        assert np.all(np.diff(sel) > 0) and sel.min() >= c * C and sel.max() < c * C + n_c


# --------------------------------------------------------------------------- NP-Map


def test_npmap_with_orthogonal_map_is_dual_softmax_of_rotated_input():
    # f(x) = xR with R orthogonal keeps the norm, so u = xR exactly (Eq. feature_map),
    # also when R is multiplied by any c > 0: the norm of x is reinjected.
    d = 6
    x = RNG.standard_normal((9, d)) * 3
    R, _ = np.linalg.qr(RNG.standard_normal((d, d)))
    for c in (1.0, 7.5, 1e-3):
        phi = o.npmap(x, c * R)
        u = x @ R
        np.testing.assert_allclose(phi[:, :d], sps.softmax(u, axis=1), rtol=1e-10)
        np.testing.assert_allclose(phi[:, d:], sps.softmax(-u, axis=1), rtol=1e-10)


def test_npmap_norm_reinjection_general_map():
    # phi+ = softmax(u): centred log phi+ equals centred u, and u = f ||x|| / ||f||.
    d, df = 5, 7
    x = RNG.standard_normal((11, d))
    W = RNG.standard_normal((d, df))
    b = RNG.standard_normal(df) * 0.1
    phi = o.npmap(x, W, b)
    assert phi.shape == (11, 2 * df)
    lp = np.log(phi[:, :df])
    uc = lp - lp.mean(axis=1, keepdims=True)
    f = x @ W + b
    fc = f - f.mean(axis=1, keepdims=True)
    ratio = np.linalg.norm(x, axis=1) / np.linalg.norm(f, axis=1)
    np.testing.assert_allclose(uc, fc * ratio[:, None], rtol=1e-9, atol=1e-12)
    # invariants: non-negative, each half sums to one, phi+_j * phi-_j is constant in j
    assert np.all(phi > 0)
    np.testing.assert_allclose(phi[:, :df].sum(1), 1, rtol=1e-12)
    np.testing.assert_allclose(phi[:, df:].sum(1), 1, rtol=1e-12)
    prod = phi[:, :df] * phi[:, df:]
    np.testing.assert_allclose(prod, prod[:, :1].repeat(df, 1), rtol=1e-9)


def test_npmap_u_norm_equals_input_norm():
    # With d_f = 2 the two equations softmax(u), softmax(-u) determine u up to nothing:
    # u_0 - u_1 = log(phi+_0 / phi+_1); and sum-free recovery via phi+ and phi-:
    # log(phi+_j / phi-_j) = 2 u_j - log(Z+/Z-)  =>  differences give u_0 - u_1 again, so
    # use the norm identity on a map whose output has zero mean: f = (a, -a).
    x = RNG.standard_normal((13, 4)) * 2
    w = RNG.standard_normal(4)
    W = np.stack([w, -w], axis=1)  # f(x) = (a, -a), u = (+-||x||/sqrt2, -+||x||/sqrt2)
    phi = o.npmap(x, W)
    u0_minus_u1 = np.log(phi[:, 0] / phi[:, 1])
    u_norm = np.abs(u0_minus_u1) / math.sqrt(2.0)  # ||u|| when u = (t, -t): sqrt(2)|t|, u0-u1 = 2t
    np.testing.assert_allclose(u_norm, np.linalg.norm(x, axis=1), rtol=1e-10)


def test_npmap_zero_map_gives_uniform_features():
    # f(x) = 0 (W = 0, no bias): the direction of f is undefined; the norm in the denominator is
    # clamped, so u = 0 and both softmaxes are uniform, 1 / d_f each -- whatever the norm of x.
    d, df = 6, 5
    x = RNG.standard_normal((7, d)) * np.array([1e-3, 1.0, 50.0, 1.0, 1.0, 1e3, 1.0])[:, None]
    phi = o.npmap(x, np.zeros((d, df)))
    np.testing.assert_allclose(phi, 1.0 / df, rtol=0, atol=1e-15)
    # a zero input row with any map: f = 0 and ||x|| = 0, again uniform
    phi0 = o.npmap(np.zeros((2, d)), RNG.standard_normal((d, df)))
    np.testing.assert_allclose(phi0, 1.0 / df, rtol=0, atol=1e-15)


# --------------------------------------------------------------------------- whole layer


def _sdpa(q, k, v, scale, mask=None):
    tq, tk, tv = (torch.from_numpy(a)[None, None] for a in (q, k, v))
    if mask is None:
        out = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)
    else:
        out = torch.nn.functional.scaled_dot_product_attention(
            tq, tk, tv, attn_mask=torch.from_numpy(mask)[None, None], scale=scale
        )
    return out[0, 0].numpy()


@pytest.mark.parametrize("form", ["chunk", "rec"])
@pytest.mark.parametrize("N,C", [(48, 8), (45, 8), (16, 16), (7, 16)])
def test_lambda_equals_chunk_is_causal_softmax_attention(form, N, C):
    # lambda = C: every token is salient, the LA set is empty and the layer is the
    # textbook causal softmax attention (App. A.1, Eq. softmax_attention).
    d = 8
    q, k, v, Wq, Wk = _rand_head(N, d)
    p = o.HeadParams(C, C, d ** -0.5)
    g = RNG.random((N, d))
    fn = o.chunkwise if form == "chunk" else o.recurrent
    y = fn(q, k, v, Wq, Wk, p, g=g)["y"]
    np.testing.assert_allclose(y, _sdpa(q, k, v, d ** -0.5), rtol=1e-9, atol=1e-12)


def test_lambda_zero_parts_are_local_softmax_and_lagged_linear_attention():
    # lambda = 0: the SA branch is softmax over chunk c-1 (whole) and chunk c (causal);
    # the LA branch is normalised linear attention (App. A.1, Eq. linear_attention) over
    # all tokens of chunks <= c-2, with phi = NP-Map built from scipy's softmax here.
    N, C, d, df = 40, 8, 6, 4
    q, k, v, Wq, Wk = _rand_head(N, d, df)
    R, _ = np.linalg.qr(RNG.standard_normal((d, d)))
    Wq, Wk = R[:, :df] * 2.0, R[:, :df] * 0.5  # not norm preserving (df < d): general case
    p = o.HeadParams(C, 0, 0.4)
    out = o.chunkwise(q, k, v, Wq, Wk, p, want_parts=True)
    parts = out["parts"]
    n_sa, d_sa, n_la, d_la, m = parts[:, :d], parts[:, d], parts[:, d + 1 : 2 * d + 1], parts[:, 2 * d + 1], parts[:, 2 * d + 2]

    def phi_of(x, W):
        f = x @ W
        u = f * (np.linalg.norm(x, axis=1) / np.linalg.norm(f, axis=1))[:, None]
        return np.concatenate([sps.softmax(u, 1), sps.softmax(-u, 1)], 1)

    pq, pk = phi_of(q, Wq), phi_of(k, Wk)
    kv_cum = np.cumsum(np.einsum("nf,ne->nfe", pk, v), axis=0)
    z_cum = np.cumsum(pk, axis=0)
    mask = np.zeros((N, N), dtype=bool)
    for t in range(N):
        c = t // C
        mask[t, max(0, (c - 1) * C) : t + 1] = True
        n_prefix = max(0, (c - 1) * C)  # tokens of chunks <= c-2
        if n_prefix == 0:
            assert d_la[t] == 0 and np.all(n_la[t] == 0)
        else:
            np.testing.assert_allclose(n_la[t], pq[t] @ kv_cum[n_prefix - 1], rtol=1e-10)
            np.testing.assert_allclose(d_la[t], pq[t] @ z_cum[n_prefix - 1], rtol=1e-10)
    np.testing.assert_allclose(n_sa / d_sa[:, None], _sdpa(q, k, v, 0.4, mask), rtol=1e-9, atol=1e-12)
    # D_SA carries exp(-m); undo it and compare with the plain sum of exponentials
    logits = 0.4 * q @ k.T
    np.testing.assert_allclose(d_sa * np.exp(m), np.where(mask, np.exp(logits), 0).sum(1), rtol=1e-10)
    # merge under one denominator
    e0 = np.exp(-m)
    y = (n_sa + e0[:, None] * n_la) / (d_sa + e0 * d_la)[:, None]
    np.testing.assert_allclose(out["y"], y, rtol=1e-12)


def _brute_force(q, k, v, g, Wq, Wk, C, lam, scale, eps, cap=0):
    """The layer from its set definitions, token by token, 1-based as in the paper."""
    N, d = q.shape
    chunk = lambda i: -(-i // C)  # noqa: E731  1-based token -> 1-based chunk
    score = {}
    for t in range(1, N + 1):
        W = list(range(max(1, t - C + 1), t + 1))
        e = {j: math.exp(scale * float(q[t - 1] @ k[j - 1])) for j in W}
        zd = sum(e.values())
        zn = sum(e[j] for j in W if j != t)
        s = 0.0
        for j in W:
            ad = e[j] / zd
            an = 0.0 if j == t else e[j] / zn
            s += ad * math.log((ad + eps) / (an + eps))
        score[t] = s
    T = chunk(N)
    M_SA = {}
    for c in range(1, T + 1):
        toks = [i for i in range(1, N + 1) if chunk(i) == c]
        ranked = sorted(toks, key=lambda i: (-score[i], i))
        M_SA[c] = set(ranked[:lam])

    def phi(x, W):
        f = x @ W
        u = f / np.linalg.norm(f) * np.linalg.norm(x)
        a, b = np.exp(u - u.max()), np.exp(-u - (-u).max())
        return np.concatenate([a / a.sum(), b / b.sum()])

    y = np.zeros((N, d))
    sets = []
    for t in range(1, N + 1):
        ct = chunk(t)
        local = {i for i in range(1, t + 1) if chunk(i) >= ct - 1}
        salient = set().union(*[M_SA[c] for c in range(1, ct - 1)]) if ct > 2 else set()
        if cap > 0:  # budget: of the routed selected tokens only the `cap` most recent stay in the cache
            salient = set(sorted(salient)[-cap:])
        la = {i for i in range(1, t + 1) if chunk(i) <= ct - 2} - salient
        sets.append((local, salient, la))
        num = np.zeros(d)
        den = 0.0
        for i in sorted(local | salient):
            w = math.exp(scale * float(q[t - 1] @ k[i - 1]))
            num += w * v[i - 1]
            den += w
        pq = phi(q[t - 1], Wq)
        S = np.zeros((len(pq), d))
        z = np.zeros(len(pq))
        for i in la:
            pk = phi(k[i - 1], Wk)
            S += np.outer(pk, v[i - 1])
            z += pk
        num += (pq @ S) * g[t - 1]
        den += pq @ z
        y[t - 1] = num / den
    idx = np.full((T, lam), -1, dtype=np.int32)
    for c in range(1, T + 1):
        s = sorted(M_SA[c])
        idx[c - 1, : len(s)] = np.array(s) - 1
    return y, np.array([score[t] for t in range(1, N + 1)]), idx, sets


@pytest.mark.parametrize("N,C,lam", [(19, 4, 1), (24, 4, 2), (13, 4, 3), (9, 4, 0), (30, 8, 3)])
def test_brute_force_tiny(N, C, lam):
    d, df = 3, 2
    rng = np.random.default_rng(N * 100 + C * 10 + lam)
    q, k, v = rng.standard_normal((3, N, d))
    Wq, Wk = rng.standard_normal((2, d, df))
    g = rng.random((N, d))
    y, score, idx, sets = _brute_force(q, k, v, g, Wq, Wk, C, lam, 0.7, 1e-6)
    for local, salient, la in sets:  # every past token is in exactly one of the three sets
        t = max(local)
        assert local | salient | la == set(range(1, t + 1))
        assert not (local & salient) and not (local & la) and not (salient & la)
    p = o.HeadParams(C, lam, 0.7, 1e-6)
    for fn in (o.chunkwise, o.recurrent):
        out = fn(q, k, v, Wq, Wk, p, g=g)
        np.testing.assert_allclose(out["score"], score, rtol=1e-10, atol=1e-12)
        if lam:
            np.testing.assert_array_equal(out["idx"], idx)
        np.testing.assert_allclose(out["y"], y, rtol=1e-9, atol=1e-12)


@pytest.mark.parametrize("N,C,lam", [(100, 16, 4), (128, 16, 16), (77, 8, 2), (64, 32, 8), (50, 16, 0)])
def test_recurrent_equals_chunkwise(N, C, lam):
    d = 8
    q, k, v, Wq, Wk = _rand_head(N, d, scale=1.5)
    g = RNG.random((N, d))
    bq, bk = RNG.standard_normal((2, d)) * 0.1
    p = o.HeadParams(C, lam, d ** -0.5)
    a = o.chunkwise(q, k, v, Wq, Wk, p, g=g, bq=bq, bk=bk)
    b = o.recurrent(q, k, v, Wq, Wk, p, g=g, bq=bq, bk=bk)
    np.testing.assert_array_equal(a["idx"], b["idx"])
    np.testing.assert_allclose(a["y"], b["y"], rtol=1e-9, atol=1e-12)


def test_constant_value_gives_constant_output():
    # y is a positive-weight average of the v_i (gate = 1), so v_i = c gives y_t = c.
    N, C, lam, d = 60, 8, 3, 5
    q, k, _, Wq, Wk = _rand_head(N, d)
    c = RNG.standard_normal(d)
    v = np.tile(c, (N, 1))
    y = o.chunkwise(q, k, v, Wq, Wk, o.HeadParams(C, lam, 0.5))["y"]
    np.testing.assert_allclose(y, v, rtol=1e-10)


def test_every_past_token_has_positive_weight_exactly_once():
    # One-hot values expose the weight of each token: positive for i <= t, zero for i > t,
    # and the weights of a row sum to one.
    N = d = 24
    C, lam = 4, 1
    q, k = RNG.standard_normal((2, N, d)) * 0.3
    Wq, Wk = RNG.standard_normal((2, d, 3))
    y = o.chunkwise(q, k, np.eye(N), Wq, Wk, o.HeadParams(C, lam, 1.0))["y"]
    assert np.all(np.triu(y, 1) == 0)
    assert np.all(y[np.tril_indices(N)] > 0)
    np.testing.assert_allclose(y.sum(1), 1, rtol=1e-12)


def test_gate_scales_only_the_linear_numerator():
    N, C, lam, d = 40, 8, 2, 4
    q, k, v, Wq, Wk = _rand_head(N, d)
    g = RNG.random((N, d)) + 0.5
    p = o.HeadParams(C, lam, 0.5)
    a = o.chunkwise(q, k, v, Wq, Wk, p, want_parts=True)["parts"]
    b = o.chunkwise(q, k, v, Wq, Wk, p, g=g, want_parts=True)["parts"]
    np.testing.assert_allclose(b[:, d + 1 : 2 * d + 1], a[:, d + 1 : 2 * d + 1] * g, rtol=1e-12)
    np.testing.assert_array_equal(np.delete(b, np.s_[d + 1 : 2 * d + 1], 1), np.delete(a, np.s_[d + 1 : 2 * d + 1], 1))


def test_linear_normaliser_counts_la_tokens():
    # sum_f z_f = 2 |LA tokens so far| because each half of phi sums to one; with q-map
    # features summing to 2 as well, a constant-feature check: D_LA <= 2 * n_LA.
    N, C, lam, d = 64, 8, 3, 4
    q, k, v, Wq, Wk = _rand_head(N, d)
    parts = o.chunkwise(q, k, v, Wq, Wk, o.HeadParams(C, lam, 0.5), want_parts=True)["parts"]
    d_la = parts[:, 2 * d + 1]
    for t in range(N):
        n_la = max(0, t // C - 1) * (C - lam)
        assert 0 <= d_la[t] <= 2 * n_la + 1e-12
        assert (d_la[t] > 0) == (n_la > 0)


def test_forced_indices_and_row_sampling():
    N, C, lam, d = 96, 8, 3, 4
    q, k, v, Wq, Wk = _rand_head(N, d)
    p = o.HeadParams(C, lam, 0.5)
    full = o.chunkwise(q, k, v, Wq, Wk, p)
    rows = [0, 7, 8, 23, 50, 95]
    part = o.chunkwise(q, k, v, Wq, Wk, p, rows=rows)
    np.testing.assert_array_equal(part["y"], full["y"][rows])
    forced = full["idx"].copy()
    forced[2] = [16, 17, 18]  # override one chunk's selection
    a = o.chunkwise(q, k, v, Wq, Wk, p, forced_idx=forced)
    b = o.recurrent(q, k, v, Wq, Wk, p, forced_idx=forced)
    np.testing.assert_allclose(a["y"], b["y"], rtol=1e-9)
    assert np.abs(a["y"][32:] - full["y"][32:]).max() > 1e-6  # chunk 2 is visible from chunk 4 on
    np.testing.assert_array_equal(a["y"][:32], full["y"][:32])


def test_layer_gqa_mapping():
    # query head h reads KV head h // (H / Hkv); NP-Map weights are per query head / per KV head
    B, H, Hkv, N, d, C, lam = 2, 4, 2, 40, 4, 8, 2
    Q = RNG.standard_normal((B, H, N, d))
    K, V = RNG.standard_normal((2, B, Hkv, N, d))
    Wq = RNG.standard_normal((H, d, d))
    Wk = RNG.standard_normal((Hkv, d, d))
    p = o.HeadParams(C, lam, 0.5)
    out = o.layer(Q, K, V, Wq, Wk, p)
    for b in range(B):
        for h in range(H):
            one = o.chunkwise(Q[b, h], K[b, h // 2], V[b, h // 2], Wq[h], Wk[h // 2], p)
            np.testing.assert_array_equal(out["y"][b, h], one["y"])
            np.testing.assert_array_equal(out["idx"][b, h], one["idx"])


def test_layer_forced_indices_are_taken_per_head():
    # forced_idx [B,H,T,lam]: head (b,h) must use its own slice (a wrong offset would show as another
    # head's selection, or as the head's own top-lambda)
    B, H, Hkv, N, d, C, lam = 2, 2, 1, 48, 4, 8, 2
    Q = RNG.standard_normal((B, H, N, d))
    K, V = RNG.standard_normal((2, B, Hkv, N, d))
    Wq = RNG.standard_normal((H, d, d))
    Wk = RNG.standard_normal((Hkv, d, d))
    p = o.HeadParams(C, lam, 0.5)
    T = N // C
    forced = np.empty((B, H, T, lam), dtype=np.int32)
    for b in range(B):
        for h in range(H):
            for c in range(T):
                forced[b, h, c] = c * C + np.array([(b + 2 * h) % C, (b + 2 * h + 3) % C])
    forced.sort(axis=-1)
    out = o.layer(Q, K, V, Wq, Wk, p, forced_idx=forced)
    for b in range(B):
        for h in range(H):
            one = o.chunkwise(Q[b, h], K[b, 0], V[b, 0], Wq[h], Wk[0], p, forced_idx=forced[b, h])
            np.testing.assert_array_equal(out["y"][b, h], one["y"])
            np.testing.assert_array_equal(out["idx"][b, h], forced[b, h])


# --------------------------------------------------------------------------- salient-cache budget
# The paper caps the salient cache in its long-context experiments without stating a rule; the rule taken
# (oldest out, folded into the linear state) is this implementation's choice.  These tests pin the
# implementation to that stated rule, not the rule to the paper.


@pytest.mark.parametrize("N,C,lam,cap", [(30, 4, 2, 4), (29, 4, 2, 3), (40, 4, 1, 2), (26, 4, 3, 1), (33, 8, 3, 6)])
def test_budget_brute_force_tiny(N, C, lam, cap):
    d, df = 3, 2
    rng = np.random.default_rng(N * 1000 + C * 100 + lam * 10 + cap)
    q, k, v = rng.standard_normal((3, N, d))
    Wq, Wk = rng.standard_normal((2, d, df))
    g = rng.random((N, d))
    y, score, idx, sets = _brute_force(q, k, v, g, Wq, Wk, C, lam, 0.7, 1e-6, cap=cap)
    for local, salient, la in sets:  # still a partition of the prefix, with at most `cap` salient tokens
        t = max(local)
        assert local | salient | la == set(range(1, t + 1))
        assert not (local & salient) and not (local & la) and not (salient & la)
        assert len(salient) <= cap
    p = o.HeadParams(C, lam, 0.7, 1e-6, max_salient=cap)
    for fn in (o.chunkwise, o.recurrent):
        out = fn(q, k, v, Wq, Wk, p, g=g)
        np.testing.assert_array_equal(out["idx"], idx)   # the budget does not change which tokens are selected
        np.testing.assert_allclose(out["y"], y, rtol=1e-9, atol=1e-12)


def test_budget_that_is_never_reached_changes_nothing():
    N, C, lam, d = 96, 8, 3, 5
    q, k, v, Wq, Wk = _rand_head(N, d)
    free = o.chunkwise(q, k, v, Wq, Wk, o.HeadParams(C, lam, 0.5))
    big = o.chunkwise(q, k, v, Wq, Wk, o.HeadParams(C, lam, 0.5, max_salient=(N // C) * lam))
    np.testing.assert_array_equal(big["y"], free["y"])
    tight = o.chunkwise(q, k, v, Wq, Wk, o.HeadParams(C, lam, 0.5, max_salient=2 * lam))
    first_diff = (2 + 2) * C + C   # the third routed chunk pushes the first one out: rows of chunk 4 on
    np.testing.assert_array_equal(tight["y"][: 4 * C], free["y"][: 4 * C])
    assert np.abs(tight["y"][4 * C: first_diff] - free["y"][4 * C: first_diff]).max() > 1e-9


@pytest.mark.parametrize("N,C,lam,cap", [(100, 16, 4, 8), (128, 16, 16, 32), (77, 8, 2, 5), (90, 8, 8, 8)])
def test_budget_recurrent_equals_chunkwise(N, C, lam, cap):
    d = 8
    q, k, v, Wq, Wk = _rand_head(N, d, scale=1.5)
    g = RNG.random((N, d))
    p = o.HeadParams(C, lam, d ** -0.5, max_salient=cap)
    a = o.chunkwise(q, k, v, Wq, Wk, p, g=g)
    b = o.recurrent(q, k, v, Wq, Wk, p, g=g)
    np.testing.assert_allclose(a["y"], b["y"], rtol=1e-9, atol=1e-12)


def test_budget_keeps_every_past_token_counted_once():
    # one-hot values expose each token's weight: positive for every i <= t whether the token is local, cached
    # or folded into the state after leaving the cache; zero for i > t; the weights of a row sum to one
    N = d = 32
    C, lam, cap = 4, 2, 4
    q, k = RNG.standard_normal((2, N, d)) * 0.3
    Wq, Wk = RNG.standard_normal((2, d, d)) * 0.3
    y = o.chunkwise(q, k, np.eye(N), Wq, Wk, o.HeadParams(C, lam, 0.5, max_salient=cap))["y"]
    for t in range(N):
        assert np.all(y[t, : t + 1] > 0) and np.all(y[t, t + 1:] == 0)
    np.testing.assert_allclose(y.sum(1), 1, rtol=1e-12)
    const = o.chunkwise(q, k, np.full((N, d), 0.25), Wq, Wk, o.HeadParams(C, lam, 0.5, max_salient=cap))["y"]
    np.testing.assert_allclose(const, 0.25, rtol=1e-12)
