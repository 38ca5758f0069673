"""Mixture-of-experts MLP block on the GPU against the oracle: router logits, chosen experts
(ties to the lower id), routing weights, each chosen expert's intermediate vector, and the
weighted sum -- the second operator teacher-forced on the GPU's own 16-bit intermediate."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import oracle.layer as ol
from paper_2504_08378_b200 import afx, synth
from gpu_util import dev_bits, rel_err
from test_gpu_layer import hm_close

pytestmark = pytest.mark.gpu


def run_moe(dt, hidden, mlp, E, top, experts_np, Wr, x, k_gu, k_down, accumulate=0, y0=None):
    gu = [dev_bits(synth.interleave_gate_up(e["w_gate"], e["w_up"])) for e in experts_np]
    down = [dev_bits(e["w_down"]) for e in experts_np]
    gu_tab = torch.tensor([t.data_ptr() for t in gu], dtype=torch.int64, device="cuda")
    down_tab = torch.tensor([t.data_ptr() for t in down], dtype=torch.int64, device="cuda")
    wr = dev_bits(Wr)
    desc = afx.MoeDesc(dtype=afx.DTYPES[dt], hidden=hidden, mlp=mlp, n_experts=E, top=top, select_mode=afx.MODE_TOPK,
                       k_gu=k_gu, k_down=k_down, tau_gu=0.0, tau_down=0.0, w_router=wr.data_ptr(), ld_router=Wr.shape[1],
                       w_gu_table=gu_tab.data_ptr(), w_down_table=down_tab.data_ptr())
    nbytes = afx.afx_moe_workspace_bytes(desc)
    raw = torch.zeros(nbytes + 256, dtype=torch.uint8, device="cuda")
    off = (-raw.data_ptr()) % 256
    ws = raw[off:off + nbytes]
    y = torch.full((1, hidden), float("nan"), device="cuda") if y0 is None else torch.from_numpy(y0).cuda()
    afx.afx_moe_block(desc, dev_bits(x), y, accumulate, ws, nbytes)
    torch.cuda.synchronize()
    head = ws[:96].cpu().numpy()
    logits = head[:64].view(np.float32)[:E]
    sel = head[64:80].view(np.int32)[:top]
    wsel = head[80:96].view(np.float32)[:top]
    stride = (mlp * 2 + 255) // 256 * 256
    hm = [ws[256 + r * stride: 256 + r * stride + mlp * 2].cpu().numpy().view(np.uint16) for r in range(top)]
    return logits, sel, wsel, hm, y.cpu().numpy()


@pytest.mark.parametrize("dt,hidden,mlp,E,top", [("bf16", 512, 768, 8, 2), ("f16", 384, 520, 5, 2), ("bf16", 512, 768, 8, 1),
                                                ("bf16", 4096, 14336, 8, 2)])
def test_moe_block_matches_the_oracle(dt, hidden, mlp, E, top):
    k_gu, k_down = synth.keep_count(hidden, 50), synth.keep_count(mlp, 50)
    experts_np = [synth.layer_weights(501, e, hidden, 1, 1, mlp, dt) for e in range(E)]
    lws = [ol.LayerWeights(None, None, e["w_gate"], e["w_up"], e["w_down"], None, None, k={"gu": k_gu, "down": k_down})
           for e in experts_np]
    Wr = synth.weight(501, 99, hidden, E, dt, sigma=0.05)
    x = synth.laplace_bits(501, 7, (1, hidden), dt)
    cfg = ol.Config(dt, hidden, 1, 1, mlp, mode=oracle.TOPK)
    ids, w, logits = ol.moe_router(x, Wr, dt, top)
    y0 = synth.laplace(501, 8, (1, hidden)).astype(np.float32)
    for accumulate in (0, 1):
        lg, sel, wsel, hm, y = run_moe(dt, hidden, mlp, E, top, experts_np, Wr, x, k_gu, k_down, accumulate, y0.copy())
        assert np.allclose(lg, logits, rtol=1e-4, atol=1e-4 * np.abs(logits).max())
        assert sel.tolist() == ids.tolist()
        assert np.allclose(wsel, w, rtol=1e-4)
        y_ref = y0.astype(np.float64) if accumulate else np.zeros((1, hidden))
        idx_gu = oracle.select_active(x, dt, oracle.TOPK, k=k_gu)
        for r in range(top):
            e = int(sel[r])
            ref = ol.mlp_block(cfg, lws[e], x)
            assert hm_close(experts_np[e], dt, mlp, x, idx_gu, hm[r][None, :], ref["hm"]), r
            idx_d = oracle.select_active(hm[r], dt, oracle.TOPK, k=k_down)
            y_ref = y_ref + float(wsel[r]) * oracle.sparse_gemv(experts_np[e]["w_down"], dt, hidden, hm[r], idx_d)
        assert rel_err(y, y_ref) <= 2e-3, accumulate


def test_router_breaks_ties_toward_the_lower_expert():
    """Integer-valued router rows make the logits exact in fp32: experts 2 and 5 tie for the
    first place, 1 and 6 for the next."""
    dt, hidden, mlp, E = "f16", 256, 264, 8
    experts_np = [synth.layer_weights(502, e, hidden, 1, 1, mlp, dt) for e in range(E)]
    Wr = np.zeros((hidden, E), np.float32)
    Wr[0] = [0, 2, 3, 1, 0, 3, 2, -1]
    x = np.zeros((1, hidden), np.float32)
    x[0, 0] = 1.0
    x[0, 1:] = 0.001 * synth.laplace(502, 3, (hidden - 1,))
    xb = synth.f32_to_bits(x, dt)
    for top, want in ((1, [2]), (2, [2, 5]), (3, [2, 5, 1]), (4, [2, 5, 1, 6])):
        lg, sel, wsel, hm, y = run_moe(dt, hidden, mlp, E, top, experts_np, synth.f32_to_bits(Wr, dt), xb, 128, 132)
        assert sel.tolist() == want and lg.tolist() == Wr[0].tolist()
        assert abs(wsel.sum() - 1.0) < 1e-6 and np.isfinite(y).all()
        ids, w, _ = ol.moe_router(xb, synth.f32_to_bits(Wr, dt), dt, top)
        assert ids.tolist() == want and np.allclose(wsel, w, rtol=1e-5)
