"""still_hybrid_attn_fwd_host (host buffers in, host buffers out) against still_hybrid_attn_fwd."""
import pytest
import torch

import paper_2602_02180_b200 as still
from paper_2602_02180_b200 import synth
from tests import util_parity as U

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,H,Hkv,d,N,k", [(2, 8, 4, 64, 64 * 6, 16), (1, 4, 2, 64, 64 * 5 + 3, 16), (3, 4, 4, 64, 256, 64),
                                           (2, 32, 8, 128, 64 * 20, 64), (2, 32, 8, 128, 64 * 12, 16)])
def test_host_buffers_match_device_buffers(B, H, Hkv, d, N, k):
    # pipelined over (batch, KV-head group) parts when the slices are aligned, single shot otherwise; the
    # last two cases have the benchmark's head structure (batch 2 x 8 KV heads x 4 query heads, d = 128:
    # sixteen parts computing alternately on two streams with a workspace each)
    w = synth.Workload("h", B, H, Hkv, d, N, 64, k, "bf16", "iid", 77)
    Q, K, V = synth.make_qkv(w, "cuda")
    Wq, Wk = synth.make_npmap_weights(w, "cuda")
    G = synth.make_gate(w, "cuda")
    p = U.params_of(w)
    want_Y, want_sc, want_sel = still.hybrid_attn_fwd(p, Q, K, V, Wq, Wk, G=G)
    pin = lambda t: t.cpu().pin_memory()  # noqa: E731
    T = -(-N // w.C)
    hY = torch.empty_like(Q, device="cpu").pin_memory()
    hsc = torch.empty(B, H, N, dtype=torch.float32).pin_memory()
    hsel = torch.empty(B, H, T, k, dtype=torch.int32).pin_memory()
    for _ in range(2):
        still.hybrid_attn_fwd_host(p, pin(Q), pin(K), pin(V), pin(Wq), pin(Wk), hG=pin(G), hY=hY, hscores=hsc,
                                   hsel_idx=hsel)
        assert torch.equal(hsel, want_sel.cpu())
        assert torch.equal(hsc, want_sc.cpu())
        assert torch.equal(hY, want_Y.cpu())
