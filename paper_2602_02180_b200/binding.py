"""Thin Python binding of the C ABI in include/still.h (argument marshalling only).

Every step of the layer runs in the CUDA kernels of libstill.so; torch is used for
device memory and streams.  There is no CPU fallback: if the library has not been
built, or there is no CUDA device, the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from .build import LIB_PATH

STILL_OK = 0
DTYPE_FP32, DTYPE_BF16 = 0, 1


class _CParams(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("d", ctypes.c_int32),
        ("d_f", ctypes.c_int32), ("chunk", ctypes.c_int32), ("topk", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("sm_scale", ctypes.c_float), ("eps", ctypes.c_float),
        ("max_salient", ctypes.c_int64),
    ]


class _CStateLayout(ctypes.Structure):
    _fields_ = [(n, ctypes.c_size_t) for n in
                ("header", "k_cache", "v_cache", "score", "sel_idx", "sel_mask", "S", "z", "scratch", "total")] + [
        ("capacity", ctypes.c_int64)]


class StillError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


@dataclass
class StillParams:
    """still_params_t: problem description (Algorithm 1 inputs)."""

    B: int
    H: int
    Hkv: int
    d: int
    chunk: int
    topk: int
    dtype: torch.dtype = torch.bfloat16
    d_f: int | None = None
    sm_scale: float | None = None
    eps: float = 1e-6
    max_salient: int = 0  # salient-cache budget per query head (a multiple of topk); 0 = unbounded

    def c(self) -> _CParams:
        return _CParams(
            self.B, self.H, self.Hkv, self.d, self.d if self.d_f is None else self.d_f, self.chunk, self.topk,
            DTYPE_FP32 if self.dtype == torch.float32 else DTYPE_BF16,
            float(self.d) ** -0.5 if self.sm_scale is None else self.sm_scale, self.eps, self.max_salient,
        )


_lib = None


def lib():
    """Loads libstill.so (built by `python -m paper_2602_02180_b200.build` or __graft_entry__.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it first (python -m paper_2602_02180_b200.build); "
                "there is no fallback path"
            )
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, i64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int64
        pp = ctypes.POINTER(_CParams)
        L.still_workspace_bytes.restype = sz
        L.still_workspace_bytes.argtypes = [pp, i64]
        L.still_state_bytes.restype = sz
        L.still_state_bytes.argtypes = [pp, i64]
        L.still_state_layout.restype = ctypes.c_int
        L.still_state_layout.argtypes = [pp, i64, ctypes.POINTER(_CStateLayout)]
        L.still_hybrid_attn_fwd.restype = ctypes.c_int
        L.still_hybrid_attn_fwd.argtypes = [pp, i64] + [vp] * 12 + [i64, vp, sz, vp]
        L.still_hybrid_attn_step.restype = ctypes.c_int
        L.still_hybrid_attn_step.argtypes = [pp, vp, i64, i64] + [vp] * 9 + [vp]
        L.still_host_arena_bytes.restype = sz
        L.still_host_arena_bytes.argtypes = [pp, i64]
        L.still_hybrid_attn_fwd_host.restype = ctypes.c_int
        L.still_hybrid_attn_fwd_host.argtypes = [pp, i64] + [vp] * 11 + [vp, sz, vp]
        L.still_hybrid_attn_fwd_static.restype = ctypes.c_int
        L.still_hybrid_attn_fwd_static.argtypes = [pp, i64] + [vp] * 11 + [vp]
        L.still_device_status.restype = ctypes.c_int
        L.still_device_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int)]
        L.still_last_launch_count.restype = ctypes.c_int
        L.still_selftest_wait_timeout.restype = ctypes.c_int
        L.still_selftest_wait_timeout.argtypes = [vp, i64, vp]
        L.still_profile_enable.restype = ctypes.c_int
        L.still_profile_enable.argtypes = [ctypes.c_int]
        L.still_profile_collect.restype = ctypes.c_int
        L.still_profile_collect.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
        L.still_strerror.restype = ctypes.c_char_p
        L.still_strerror.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().still_strerror(int(code)).decode()


def _ptr(t):
    if t is None:
        return None
    assert t.is_contiguous(), "tensors must be contiguous"
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def workspace_bytes(p: StillParams, N: int) -> int:
    c = p.c()
    return lib().still_workspace_bytes(ctypes.byref(c), N)


def state_bytes(p: StillParams, max_tokens: int) -> int:
    c = p.c()
    return lib().still_state_bytes(ctypes.byref(c), max_tokens)


def state_layout(p: StillParams, max_tokens: int) -> dict:
    c, out = p.c(), _CStateLayout()
    rc = lib().still_state_layout(ctypes.byref(c), max_tokens, ctypes.byref(out))
    if rc != STILL_OK:
        raise StillError(rc, "still_state_layout")
    return {n: getattr(out, n) for n, _ in _CStateLayout._fields_}


def host_arena_bytes(p: StillParams, N: int) -> int:
    c = p.c()
    return lib().still_host_arena_bytes(ctypes.byref(c), N)


def last_launch_count() -> int:
    return lib().still_last_launch_count()


def hybrid_attn_fwd(p: StillParams, Q, K, V, Wq=None, Wk=None, G=None, bq=None, bk=None, Y=None,
                    scores=None, sel_idx=None, state=None, state_max_tokens=0, workspace=None,
                    want_y=True):
    """still_hybrid_attn_fwd.  Returns (Y, scores, sel_idx); allocates outputs / workspace with
    torch when they are not passed in."""
    if not Q.is_cuda:
        raise RuntimeError("still_hybrid_attn_fwd needs CUDA tensors; there is no CPU path")
    N = Q.shape[2]
    T = (N + p.chunk - 1) // p.chunk
    dev = Q.device
    if Y is None and want_y:
        Y = torch.empty_like(Q)
    if scores is None:
        scores = torch.empty(p.B, p.H, N, dtype=torch.float32, device=dev)
    if sel_idx is None:
        sel_idx = torch.empty(p.B, p.H, T, max(p.topk, 1), dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = torch.empty(workspace_bytes(p, N), dtype=torch.uint8, device=dev)
    c = p.c()
    rc = lib().still_hybrid_attn_fwd(
        ctypes.byref(c), N, _ptr(Q), _ptr(K), _ptr(V), _ptr(G), _ptr(Wq), _ptr(bq), _ptr(Wk), _ptr(bk),
        _ptr(Y), _ptr(scores), _ptr(sel_idx), _ptr(state), state_max_tokens, _ptr(workspace),
        workspace.numel(), _stream(),
    )
    if rc != STILL_OK:
        raise StillError(rc, "still_hybrid_attn_fwd")
    return Y, scores, sel_idx[..., : p.topk]


STATIC_WORKSPACE_BYTES = 16 << 20


def hybrid_attn_fwd_static(p: StillParams, Q, K, V, Wq=None, Wk=None, G=None, bq=None, bk=None, *, Y, scores,
                           sel_idx):
    """still_hybrid_attn_fwd_static: the prefill with its workspace inside the library (for callers
    that cannot allocate device memory).  Every output buffer is passed in; this wrapper allocates
    nothing either.  Returns (Y, scores, sel_idx)."""
    if not Q.is_cuda:
        raise RuntimeError("still_hybrid_attn_fwd_static needs CUDA tensors; there is no CPU path")
    c = p.c()
    rc = lib().still_hybrid_attn_fwd_static(
        ctypes.byref(c), Q.shape[2], _ptr(Q), _ptr(K), _ptr(V), _ptr(G), _ptr(Wq), _ptr(bq), _ptr(Wk), _ptr(bk),
        _ptr(Y), _ptr(scores), _ptr(sel_idx), _stream(),
    )
    if rc != STILL_OK:
        raise StillError(rc, "still_hybrid_attn_fwd_static")
    return Y, scores, sel_idx


def hybrid_attn_step(p: StillParams, state, state_max_tokens, t_pos, q, k, v, Wq=None, Wk=None, g=None,
                     bq=None, bk=None, y=None):
    """still_hybrid_attn_step.  Returns y [B,H,d]."""
    if not q.is_cuda:
        raise RuntimeError("still_hybrid_attn_step needs CUDA tensors; there is no CPU path")
    if y is None:
        y = torch.empty_like(q)
    c = p.c()
    rc = lib().still_hybrid_attn_step(
        ctypes.byref(c), _ptr(state), state_max_tokens, t_pos, _ptr(q), _ptr(k), _ptr(v), _ptr(g),
        _ptr(Wq), _ptr(bq), _ptr(Wk), _ptr(bk), _ptr(y), _stream(),
    )
    if rc != STILL_OK:
        raise StillError(rc, "still_hybrid_attn_step")
    return y


def hybrid_attn_fwd_host(p: StillParams, hQ, hK, hV, hWq=None, hWk=None, hG=None, hbq=None, hbk=None,
                         hY=None, hscores=None, hsel_idx=None, arena=None):
    """still_hybrid_attn_fwd_host: host (ideally pinned) tensors in, host tensors out."""
    N = hQ.shape[2]
    if hY is None:
        hY = torch.empty_like(hQ).pin_memory()
    if arena is None:
        arena = torch.empty(host_arena_bytes(p, N), dtype=torch.uint8, device="cuda")
    c = p.c()
    rc = lib().still_hybrid_attn_fwd_host(
        ctypes.byref(c), N, _ptr(hQ), _ptr(hK), _ptr(hV), _ptr(hG), _ptr(hWq), _ptr(hbq), _ptr(hWk),
        _ptr(hbk), _ptr(hY), _ptr(hscores), _ptr(hsel_idx), _ptr(arena), arena.numel(), _stream(),
    )
    if rc != STILL_OK:
        raise StillError(rc, "still_hybrid_attn_fwd_host")
    return hY


def profile_enable(max_records: int) -> None:
    rc = lib().still_profile_enable(max_records)
    if rc != STILL_OK:
        raise StillError(rc, "still_profile_enable")


def profile_collect(capacity: int = 4096) -> list[float]:
    """Milliseconds of the dominant kernel for every call since profile_enable."""
    buf = (ctypes.c_float * capacity)()
    n = ctypes.c_int(0)
    rc = lib().still_profile_collect(buf, capacity, ctypes.byref(n))
    if rc != STILL_OK:
        raise StillError(rc, "still_profile_collect")
    return [buf[i] for i in range(n.value)]


def selftest_wait_timeout(status_block, limit_cycles: int) -> None:
    """still_selftest_wait_timeout: a bounded device wait that runs out after limit_cycles."""
    rc = lib().still_selftest_wait_timeout(_ptr(status_block), int(limit_cycles), _stream())
    if rc != STILL_OK:
        raise StillError(rc, "still_selftest_wait_timeout")


def device_status(buf) -> tuple[int, int]:
    st, det = ctypes.c_int(0), ctypes.c_int(0)
    rc = lib().still_device_status(_ptr(buf), _stream(), ctypes.byref(st), ctypes.byref(det))
    if rc != STILL_OK:
        raise StillError(rc, "still_device_status")
    return st.value, det.value
