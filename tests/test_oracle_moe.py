"""Pins for the oracle's mixture-of-experts block (router, top-2, weighted combination)."""
import math

import numpy as np

import oracle
import oracle.layer as ol
from paper_2504_08378_b200 import synth


def bits(a, dt="f16"):
    return synth.f32_to_bits(np.asarray(a, np.float32), dt)


def test_router_hand_case():
    """x = e_0 + 2 e_1; router rows r0 = [1, 3, 1, 0], r1 = [0, 0, 1, 0]: logits = [1, 3, 3, 0].
    Experts 1 and 2 tie at 3: the lower id ranks first; equal logits -> weights 1/2 each."""
    x = bits([1, 2, 0, 0])
    Wr = bits([[1, 3, 1, 0], [0, 0, 1, 0], [5, 5, 5, 5], [7, 7, 7, 7]])
    ids, w, logits = ol.moe_router(x, Wr, "f16")
    assert logits.tolist() == [1, 3, 3, 0] and ids.tolist() == [1, 2] and w.tolist() == [0.5, 0.5]
    # logits [2, 0, 1, -1] (x = e_0, r0 as given): experts 0 and 2, weights e^0 : e^-1
    ids, w, _ = ol.moe_router(bits([1, 0, 0, 0]), bits([[2, 0, 1, -1]] + [[0] * 4] * 3), "f16")
    assert ids.tolist() == [0, 2]
    assert np.allclose(w, [1 / (1 + math.exp(-1)), math.exp(-1) / (1 + math.exp(-1))], rtol=1e-15)
    ids, w, _ = ol.moe_router(bits([1, 0, 0, 0]), bits([[2, 0, 1, -1]] + [[0] * 4] * 3), "f16", top=1)
    assert ids.tolist() == [0] and w.tolist() == [1.0]


def test_identical_experts_give_the_plain_mlp_block():
    """If every expert holds the same weights, the weighted sum (weights add up to 1) must be the
    MLP block itself, whichever experts the router picks."""
    dt, hidden, mlp, E = "bf16", 256, 384, 4
    L = synth.layer_weights(71, 0, hidden, 2, 2, mlp, dt)
    lw = ol.LayerWeights(None, None, L["w_gate"], L["w_up"], L["w_down"], None, None, k={"gu": 128, "down": 192})
    cfg = ol.Config(dt, hidden, 2, 2, mlp, mode=oracle.TOPK)
    x = synth.laplace_bits(71, 5, (1, hidden), dt)
    Wr = synth.weight(71, 9, hidden, E, dt, sigma=0.5)
    out = ol.moe_block(cfg, x, Wr, [lw] * E)
    ref = ol.mlp_block(cfg, lw, x)
    assert abs(out["weights"].sum() - 1.0) < 1e-15 and len(set(out["experts"].tolist())) == 2
    assert np.allclose(out["y"], ref["y"], rtol=1e-13, atol=1e-13)


def test_moe_block_is_the_weighted_sum_of_the_chosen_experts():
    dt, hidden, mlp, E = "f16", 256, 384, 8
    cfg = ol.Config(dt, hidden, 2, 2, mlp, mode=oracle.TOPK)
    experts = []
    for e in range(E):
        L = synth.layer_weights(72, e, hidden, 2, 2, mlp, dt)
        experts.append(ol.LayerWeights(None, None, L["w_gate"], L["w_up"], L["w_down"], None, None,
                                       k={"gu": 128, "down": 192}))
    x = synth.laplace_bits(72, 5, (1, hidden), dt)
    Wr = synth.weight(72, 9, hidden, E, dt, sigma=0.5)
    out = ol.moe_block(cfg, x, Wr, experts)
    # the router by plain numpy, the experts one by one
    logits = oracle.decode(x, dt).reshape(-1) @ oracle.decode(Wr, dt)
    top = np.argsort(-logits, kind="stable")[:2]
    assert out["experts"].tolist() == top.tolist()
    p = np.exp(logits[top]) / np.exp(logits[top]).sum()
    want = sum(pe * ol.mlp_block(cfg, experts[e], x)["y"] for e, pe in zip(top, p))
    assert np.allclose(out["y"], want, rtol=1e-12, atol=1e-14)
    assert np.allclose(out["logits"], logits, rtol=1e-12, atol=1e-12)
