"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares,
and its host-side logic (validation, size planning, error strings) behaves.  No kernel runs."""
import ctypes
import os
import re

import pytest
import torch

import paper_2602_02180_b200 as still
from paper_2602_02180_b200 import build as still_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    still_build.build_library()
    return still.binding.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "still.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(still_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert "still_hybrid_attn_fwd" in names and "still_hybrid_attn_step" in names
    for n in names:
        assert hasattr(lib, n), f"libstill.so does not export {n}"


def test_validation_and_sizes(lib):
    ok = still.StillParams(2, 32, 8, 128, 64, 64)
    assert still.workspace_bytes(ok, 32768) > 0
    assert still.workspace_bytes(ok, 32768) <= still.workspace_bytes(still.StillParams(2, 32, 8, 128, 64, 16), 32768)
    for bad in [
        still.StillParams(2, 32, 7, 128, 64, 64),      # H % Hkv
        still.StillParams(2, 32, 8, 96, 64, 64),       # head dim
        still.StillParams(2, 32, 8, 128, 48, 16),      # chunk
        still.StillParams(2, 32, 8, 128, 64, 65),      # topk > chunk
        still.StillParams(2, 32, 8, 128, 64, -1),
        still.StillParams(0, 32, 8, 128, 64, 64),
        still.StillParams(2, 32, 8, 128, 64, 64, sm_scale=0.0),
        still.StillParams(2, 32, 8, 64, 64, 64, d_f=128),
    ]:
        assert still.workspace_bytes(bad, 1024) == 0
        assert still.state_bytes(bad, 1024) == 0
    lay = still.state_layout(still.StillParams(1, 4, 2, 64, 64, 16), 1000)
    assert lay["capacity"] == 1024 and lay["total"] == still.state_bytes(still.StillParams(1, 4, 2, 64, 64, 16), 1000)
    order = [lay[k] for k in ("header", "k_cache", "v_cache", "score", "sel_idx", "sel_mask", "S", "z", "scratch", "total")]
    assert order == sorted(order) and all(o % 256 == 0 for o in order)
    with pytest.raises(still.StillError):
        still.state_layout(still.StillParams(1, 4, 3, 64, 64, 16), 1000)


def test_null_and_error_codes_without_a_device(lib):
    c = still.StillParams(1, 2, 2, 64, 64, 16).c()
    rc = lib.still_hybrid_attn_fwd(ctypes.byref(c), 128, None, None, None, None, None, None, None, None, None,
                                   None, None, None, 0, None, 0, None)
    assert rc == -1
    rc = lib.still_hybrid_attn_step(ctypes.byref(c), None, 0, 0, None, None, None, None, None, None, None, None,
                                    None, None)
    assert rc == -1
    assert still.strerror(0) == "ok"
    assert {still.strerror(k) for k in range(-7, 0)}.isdisjoint({"unknown status"})
    assert still.strerror(-99) == "unknown status"


def test_binding_refuses_cpu_tensors(lib):
    p = still.StillParams(1, 2, 2, 64, 64, 16, torch.float32)
    x = torch.zeros(1, 2, 128, 64)
    with pytest.raises(RuntimeError, match="no CPU path"):
        still.hybrid_attn_fwd(p, x, x, x, None, None)
    with pytest.raises(RuntimeError, match="no CPU path"):
        still.hybrid_attn_step(p, None, 0, 0, x[:, :, 0], x[:, :, 0], x[:, :, 0])
