"""ctypes binding of the CPU oracle (oracle/still_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
CPU-baseline leg of the benchmark.  The CUDA library never imports this module
and this module never imports the CUDA package.

All arrays cross this boundary as C-contiguous float64 / int32 / int64 numpy
arrays; the callers round their inputs to the GPU dtype first, so both sides see
the same values.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "still_oracle.c")
_LIB = os.path.join(_HERE, "libstill_oracle.so")

_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int32)
_lp = ctypes.POINTER(ctypes.c_int64)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over heads).  Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.still_oracle_layer.restype = ctypes.c_int
    return _lib


def _d(a):
    if a is None:
        return None
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_dp)


def _i32(a):
    if a is None:
        return None
    assert a.dtype == np.int32 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_ip)


def _i64(a):
    if a is None:
        return None
    assert a.dtype == np.int64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_lp)


def _f64(a):
    return None if a is None else np.ascontiguousarray(np.asarray(a, dtype=np.float64))


@dataclass
class HeadParams:
    """Hyper-parameters of one call (Algorithm 1 inputs: C, lambda, epsilon; plus the
    logit scale and the NP-Map width)."""

    C: int
    lam: int
    sm_scale: float
    eps: float = 1e-6
    max_salient: int = 0  # salient-cache budget per head; 0 = unbounded (rule: oldest out, folded into the LA state)


def score_tokenwise(q, k, w, sm_scale, eps=1e-6):
    """Self-Saliency Score from the window-set definition (Sec. 3.1)."""
    q, k = _f64(q), _f64(k)
    N, d = q.shape
    out = np.empty(N, dtype=np.float64)
    _load().still_oracle_score_tokenwise(
        _d(q), _d(k), ctypes.c_int64(N), d, int(w), ctypes.c_double(sm_scale), ctypes.c_double(eps), _d(out)
    )
    return out


def score_global(q, k, sm_scale, eps=1e-6):
    """Self-Saliency Score with the full causal context as the window, W_t = {1..t}: the global variant the
    local score is compared with in Sec. 3.1 (local-global consistency).  It is the window-set definition with
    a window that is never shorter than the prefix."""
    return score_tokenwise(q, k, max(int(np.asarray(q).shape[0]), 1), sm_scale, eps)


def score_chunkwise(q, k, C, sm_scale, eps=1e-6):
    """Self-Saliency Score from chunk tiles and masks (Algorithm 1)."""
    q, k = _f64(q), _f64(k)
    N, d = q.shape
    out = np.empty(N, dtype=np.float64)
    _load().still_oracle_score_chunkwise(
        _d(q), _d(k), ctypes.c_int64(N), d, int(C), ctypes.c_double(sm_scale), ctypes.c_double(eps), _d(out)
    )
    return out


def select(score, C, lam):
    """Top-lambda per chunk -> [T, lam] absolute positions, ascending, -1 padded."""
    score = _f64(score)
    N = score.shape[0]
    T = (N + C - 1) // C
    idx = np.full((T, max(lam, 0)), -1, dtype=np.int32)
    if lam > 0:
        _load().still_oracle_select(_d(score), ctypes.c_int64(N), int(C), int(lam), _i32(idx))
    return idx


def npmap(x, W, b=None):
    """Norm-Preserved Feature Map of the rows of x: [n, d] -> [n, 2 d_f]."""
    x, W, b = _f64(x), _f64(W), _f64(b)
    n, d = x.shape
    df = W.shape[1]
    assert W.shape[0] == d
    phi = np.empty((n, 2 * df), dtype=np.float64)
    _load().still_oracle_npmap(_d(x), ctypes.c_int64(n), d, df, _d(W), _d(b), _d(phi))
    return phi


def chunkwise(q, k, v, Wq, Wk, p: HeadParams, g=None, bq=None, bk=None, forced_idx=None, rows=None,
              want_parts=False):
    """Algorithm 1 for one head.  Returns dict(y, score, idx[, parts])."""
    q, k, v, g, Wq, Wk, bq, bk = map(_f64, (q, k, v, g, Wq, Wk, bq, bk))
    N, d = q.shape
    df = Wq.shape[1]
    T = (N + p.C - 1) // p.C
    rows_a = None if rows is None else np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    n_out = N if rows_a is None else rows_a.shape[0]
    if rows_a is not None and n_out > 1:
        assert np.all(np.diff(rows_a) > 0), "rows must be strictly ascending"
    y = np.empty((n_out, d), dtype=np.float64)
    score = np.empty(N, dtype=np.float64)
    idx = np.full((T, max(p.lam, 1)), -1, dtype=np.int32)
    fi = None
    if forced_idx is not None:
        fi = np.ascontiguousarray(np.asarray(forced_idx, dtype=np.int32).reshape(T, p.lam))
    parts = np.empty((n_out, 2 * d + 3), dtype=np.float64) if want_parts else None
    _load().still_oracle_chunkwise(
        _d(q), _d(k), _d(v), _d(g), ctypes.c_int64(N), d, df, int(p.C), int(p.lam),
        ctypes.c_double(p.sm_scale), ctypes.c_double(p.eps), ctypes.c_int64(p.max_salient), _d(Wq), _d(bq), _d(Wk), _d(bk),
        _i32(fi), _i64(rows_a), ctypes.c_int64(n_out if rows_a is not None else 0),
        _d(y), _d(score), _i32(idx) if p.lam > 0 else None, _d(parts),
    )
    out = {"y": y, "score": score, "idx": idx[:, : p.lam]}
    if want_parts:
        out["parts"] = parts
    return out


def recurrent(q, k, v, Wq, Wk, p: HeadParams, g=None, bq=None, bk=None, forced_idx=None):
    """Recurrent Form (Sec. 3.3) for one head.  Returns dict(y, score, idx)."""
    q, k, v, g, Wq, Wk, bq, bk = map(_f64, (q, k, v, g, Wq, Wk, bq, bk))
    N, d = q.shape
    df = Wq.shape[1]
    T = (N + p.C - 1) // p.C
    y = np.empty((N, d), dtype=np.float64)
    score = np.empty(N, dtype=np.float64)
    idx = np.full((T, max(p.lam, 1)), -1, dtype=np.int32)
    fi = None
    if forced_idx is not None:
        fi = np.ascontiguousarray(np.asarray(forced_idx, dtype=np.int32).reshape(T, p.lam))
    _load().still_oracle_recurrent(
        _d(q), _d(k), _d(v), _d(g), ctypes.c_int64(N), d, df, int(p.C), int(p.lam),
        ctypes.c_double(p.sm_scale), ctypes.c_double(p.eps), ctypes.c_int64(p.max_salient), _d(Wq), _d(bq), _d(Wk), _d(bk),
        _i32(fi), _d(y), _d(score), _i32(idx) if p.lam > 0 else None,
    )
    return {"y": y, "score": score, "idx": idx[:, : p.lam]}


def layer(Q, K, V, Wq, Wk, p: HeadParams, G=None, bq=None, bk=None, forced_idx=None, rows=None):
    """Whole layer, heads in parallel (OpenMP).  Q,G [B,H,N,d]; K,V [B,Hkv,N,d];
    Wq [H,d,df]; Wk [Hkv,d,df].  Returns dict(y [B,H,n_out,d], score [B,H,N],
    idx [B,H,T,lam], threads)."""
    Q, K, V, G, Wq, Wk, bq, bk = map(_f64, (Q, K, V, G, Wq, Wk, bq, bk))
    B, H, N, d = Q.shape
    Hkv = K.shape[1]
    df = Wq.shape[2]
    T = (N + p.C - 1) // p.C
    rows_a = None if rows is None else np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    n_out = N if rows_a is None else rows_a.shape[0]
    Y = np.empty((B, H, n_out, d), dtype=np.float64)
    score = np.empty((B, H, N), dtype=np.float64)
    idx = np.full((B, H, T, max(p.lam, 1)), -1, dtype=np.int32)
    fi = None
    if forced_idx is not None:
        fi = np.ascontiguousarray(np.asarray(forced_idx, dtype=np.int32).reshape(B, H, T, p.lam))
    threads = _load().still_oracle_layer(
        _d(Q), _d(K), _d(V), _d(G), B, H, Hkv, ctypes.c_int64(N), d, df, int(p.C), int(p.lam),
        ctypes.c_double(p.sm_scale), ctypes.c_double(p.eps), ctypes.c_int64(p.max_salient), _d(Wq), _d(bq), _d(Wk), _d(bk),
        _i32(fi), _i64(rows_a), ctypes.c_int64(n_out if rows_a is not None else 0),
        _d(Y), _d(score), _i32(idx) if p.lam > 0 else None,
    )
    return {"y": Y, "score": score, "idx": idx[..., : p.lam], "threads": threads}
