"""Evaluation terms of Sec. 3.3 on the GPU against the checker: the missing residual (Eq. 6), the draft-expert
term and the residual loss (Eq. 7), the router-agreement divergence (Eq. 10) and the top-k set agreement."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2607_24434_b200 import synth
from tests.helpers import GATE_TOL, Y_TIGHT, check_routing, gpu_layer, row_rel_err

pytestmark = pytest.mark.gpu

SMALL = synth.LayerShape(hidden=512, n_experts=16, top_k=4, inter=64, n_shared=1, shared_inter=64, draft_inter=32,
                         score_fn=synth.SCORE_SOFTMAX, norm_topk=1, routed_scale=1.0, draft_gamma=0.75,
                         weight_dtype=synth.DTYPE_BF16)


@pytest.fixture()
def dx():
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0, act_split=True)
    yield binding, ctx
    assert ctx.device_status() == 0
    ctx.close()


def _residual_case(dx, shape, K, seed, std, zipf=False):
    binding, ctx = dx
    layer, ref = gpu_layer(shape, seed, zipf=zipf, std=std)
    L = binding.Layer.from_weights(ctx, layer)
    h = synth.hidden_block(K, shape.hidden, seed + 1, 0.3, "cuda")
    h_np = h.cpu().numpy().astype(np.float64)
    out = binding.moe_missing_residual(L, h)
    dterm = binding.moe_draft_expert_term(L, h)
    loss = binding.squared_error(ctx, dterm, out["m"])
    y_full = binding.moe_verify_block(L, h)["y"]          # the full layer afterwards: the switches must not stick
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ids = out["topk_ids"].cpu().numpy()
    _, ids_ref, _, z_ref = O.moe_target(h_np, ref)
    check_routing(shape, z_ref, ids_ref, ids)
    # Eq. 6 with the GPU's own selection replayed: y* minus the shared + top-1 path
    y_star, _, g, _ = O.moe_target(h_np, ref, forced_ids=ids)
    y_top1 = O.moe_draft(h_np, ref, gamma=0.0, forced_ids=ids)[0] if K == 1 else np.stack(
        [O.moe_draft(h_np[t:t + 1], ref, gamma=0.0, forced_ids=ids[t:t + 1])[0][0] for t in range(K)])
    m_ref = y_star - y_top1
    assert np.abs(out["topk_w"].cpu().numpy() - g).max() <= GATE_TOL * max(1.0, shape.routed_scale)
    m_gpu = out["m"].cpu().numpy()
    scale = np.abs(y_star).max(axis=1)           # rows of m can be small next to y*: bound against the layer's output
    assert (np.abs(m_gpu - m_ref).max(axis=1) / scale).max() <= Y_TIGHT
    assert row_rel_err(m_gpu, m_ref).max() <= 5 * Y_TIGHT
    # gamma * E^d(h)
    d_ref = O.draft_expert_term(h_np, ref)
    assert row_rel_err(dterm.cpu().numpy(), d_ref).max() <= Y_TIGHT
    # Eq. 7 term, from the GPU's own two operands (the reduction) and against the checker end to end
    want_red = float(((dterm.cpu().numpy().astype(np.float64) - m_gpu.astype(np.float64)) ** 2).sum())
    assert abs(float(loss.item()) - want_red) <= 1e-5 * max(want_red, 1e-30)
    want = float(((d_ref - m_ref) ** 2).sum())
    assert abs(float(loss.item()) - want) <= 2e-3 * want
    # and the ordinary verify block still gives the full layer
    assert row_rel_err(y_full.cpu().numpy(), y_star).max() <= Y_TIGHT
    L.close()


@pytest.mark.parametrize("K", [1, 4, 9])
def test_missing_residual_small(dx, K):
    _residual_case(dx, SMALL, K, seed=40 + K, std=0.08)


def test_missing_residual_tiny_fp32(dx):
    _residual_case(dx, synth.shape_tiny(), 4, seed=45, std=0.05)


def test_missing_residual_v2lite(dx):
    _residual_case(dx, synth.shape_v2lite(), 4, seed=46, std=0.02, zipf=True)


@pytest.mark.parametrize("shape,K", [(SMALL, 5), (dataclasses.replace(SMALL, score_fn=synth.SCORE_SIGMOID, n_experts=130,
                                                                      top_k=8, routed_scale=2.446), 3),
                                     (synth.shape_tiny(), 4), (synth.shape_v2lite(), 4)])
def test_router_agreement(dx, shape, K):
    binding, ctx = dx
    layer, ref = gpu_layer(shape, 50, zipf=True, std=0.05)
    L = binding.Layer.from_weights(ctx, layer)
    hs = synth.hidden_block(K, shape.hidden, 51, 0.0, "cuda")
    hd = (hs + 0.35 * synth.hidden_block(K, shape.hidden, 52, 0.0, "cuda")).contiguous()
    hd[0] = hs[0]                                   # one row where the drafter has not drifted at all
    kl, agree = binding.moe_router_agreement(L, hs, hd)
    torch.cuda.synchronize()
    kl_ref, ag_ref, ids_s, ids_d = O.router_agreement(hs.cpu().numpy().astype(np.float64),
                                                      hd.cpu().numpy().astype(np.float64), ref)
    kl_gpu = kl.cpu().numpy()
    assert abs(kl_gpu[0]) <= 1e-6 and int(agree[0].item()) == shape.top_k
    assert np.all(np.abs(kl_gpu - kl_ref) <= 1e-4 * np.maximum(1.0, kl_ref) + 1e-6)
    # the set agreement is an integer: exact wherever neither selection is near-tied
    zs = O.router_logits(hs.cpu().numpy().astype(np.float64), ref["router"], ref["bias"])
    zd = O.router_logits(hd.cpu().numpy().astype(np.float64), ref["router"], ref["bias"])
    _, gap_s = O.selection_gaps(zs, shape.top_k)
    _, gap_d = O.selection_gaps(zd, shape.top_k)
    ag_gpu = agree.cpu().numpy()
    checked = 0
    for t in range(K):
        if gap_s[t] > 1e-3 and gap_d[t] > 1e-3:
            assert ag_gpu[t] == ag_ref[t]
            checked += 1
        else:
            assert abs(int(ag_gpu[t]) - int(ag_ref[t])) <= 2
    assert checked >= 1
    L.close()
