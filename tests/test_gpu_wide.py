"""Layers packed in the wide blob layout (DX_DTYPE_BF16_WIDE): the grouped SwiGLU on tcgen05 / tensor memory with the
block rows as the 16-column operand, against the CPU checker.  Same entry points, same comparisons as the streaming
layout: routing exact outside the 1e-3 gap, gates to 1e-5, union and permutation exact, layer outputs within 2e-2 of
the row maximum (and within the bf16-activation regression bound); block lengths 1..16, ragged intermediate sizes
(partial macro-units), all supported hidden sizes, the drafter, the residual forms, cache waves, and the full
DeepSeek-V2-Lite-shaped layer at K = 4, 8 and 16."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from oracle.cache_oracle import ExpertCacheModel
from paper_2607_24434_b200 import synth
from tests.helpers import Y_BF16, check_union, gpu_layer, row_rel_err
from tests.test_gpu_parity import _draft_case, _verify_case

pytestmark = pytest.mark.gpu

SMALL = synth.LayerShape(hidden=512, n_experts=16, top_k=3, inter=40, n_shared=2, shared_inter=24, draft_inter=56,
                         score_fn=synth.SCORE_SOFTMAX, norm_topk=1, weight_dtype=synth.DTYPE_BF16_WIDE)


@pytest.fixture(scope="module")
def dxw():
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    ctx.y_tol = Y_BF16
    yield binding, ctx
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.parametrize("K", [1, 2, 4, 7, 8, 9, 13, 16])
def test_wide_small_verify(dxw, K):
    _verify_case(dxw, SMALL, K, seed=10 + K, std=0.08)


@pytest.mark.parametrize("H", [256, 1024])
def test_wide_other_hidden_sizes(dxw, H):
    sh = dataclasses.replace(SMALL, hidden=H, n_experts=130, top_k=8, inter=16, score_fn=synth.SCORE_SIGMOID,
                             routed_scale=2.446)
    _verify_case(dxw, sh, 6, seed=20, std=0.08)
    _verify_case(dxw, sh, 12, seed=21, std=0.08, zipf=True)
    _draft_case(dxw, sh, seed=22, std=0.08)


def test_wide_macro_unit_edges(dxw):
    """Intermediate sizes around the 64-wide macro-unit: one short unit, exactly one, one and a bit, several."""
    for inter in (8, 64, 72, 200):
        sh = dataclasses.replace(SMALL, inter=inter, shared_inter=inter + 8, draft_inter=inter)
        _verify_case(dxw, sh, 11, seed=40 + inter, std=0.08)
        _draft_case(dxw, sh, seed=41 + inter, std=0.08)


def test_wide_draft_and_no_shared(dxw):
    _draft_case(dxw, SMALL, seed=30, std=0.08)
    sh = dataclasses.replace(SMALL, n_shared=0, shared_inter=0, draft_inter=0)
    _verify_case(dxw, sh, 4, seed=31, std=0.08)
    _draft_case(dxw, sh, seed=32, std=0.08)


def test_wide_residual_forms_and_topr(dxw):
    binding, ctx = dxw
    layer, ref = gpu_layer(SMALL, 60, std=0.08)
    L = binding.Layer.from_weights(ctx, layer)
    h = synth.hidden_block(12, SMALL.hidden, 61, 0.9, "cuda") * 3.0
    h_np = h.cpu().numpy().astype(np.float64)
    out = binding.moe_verify_block_residual(L, h)
    torch.cuda.synchronize()
    ids = out["topk_ids"].cpu().numpy()
    want = O.stack_layer_target(h_np, ref, forced_ids=ids)[0]
    assert row_rel_err(out["h"].cpu().numpy(), want).max() <= Y_BF16
    outd = binding.moe_draft_step_residual(L, h[:1])
    torch.cuda.synchronize()
    wantd = O.stack_layer_draft(h_np[:1], ref, forced_ids=outd["topk_ids"].cpu().numpy()[None])[0]
    assert row_rel_err(outd["h"].cpu().numpy(), wantd).max() <= Y_BF16
    for r, use_d in [(1, False), (2, False), (2, True)]:
        o = binding.moe_draft_step_topr(L, h[:1].contiguous(), r, use_d)
        torch.cuda.synchronize()
        w = O.moe_draft(h_np[:1], ref, forced_ids=o["topk_ids"].cpu().numpy()[None], top_r=r,
                        gamma=None if use_d else 0.0)[0]
        assert row_rel_err(o["y"].cpu().numpy(), w).max() <= Y_BF16, (r, use_d)
    # Eq. 6 through the same kernel (each row's first selected expert weighted zero, shared experts skipped)
    m = binding.moe_missing_residual(L, h)
    torch.cuda.synchronize()
    ids_m = m["topk_ids"].cpu().numpy()
    y_star = O.moe_target(h_np, ref, forced_ids=ids_m)[0]
    y_top1 = np.stack([O.moe_draft(h_np[t:t + 1], ref, gamma=0.0, forced_ids=ids_m[t:t + 1])[0][0]
                       for t in range(h_np.shape[0])])
    scale = np.abs(y_star).max(axis=1)
    assert (np.abs(m["m"].cpu().numpy() - (y_star - y_top1)).max(axis=1) / scale).max() <= Y_BF16
    assert ctx.device_status() == 0
    L.close()


def test_wide_through_the_cache_in_waves(dxw):
    """Union larger than the slots: several launches, each over a subset of the routed groups."""
    binding, ctx = dxw
    layer, ref = gpu_layer(SMALL, 70, std=0.08)
    resident = binding.Layer.from_weights(ctx, layer)
    off = binding.Layer.from_weights(ctx, layer, routed_resident=False)
    torch.cuda.synchronize()
    host = off.blobs.cpu().pin_memory()
    cache = binding.ExpertCache(ctx, 1, SMALL.n_experts, 4, host.shape[1])
    for e in range(SMALL.n_experts):
        cache.register(0, e, host[e])
    cache.attach(off, 0)
    model = ExpertCacheModel(1, SMALL.n_experts, 4)
    for step, K in enumerate([6, 12, 16]):
        h = synth.hidden_block(K, SMALL.hidden, 80 + step, 0.5, "cuda")
        cache.begin_step(); model.begin_step()
        out = binding.moe_verify_block_cached(off, cache, 0, h)
        want = binding.moe_verify_block(resident, h)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        assert torch.equal(out["topk_ids"], want["topk_ids"])
        ids = out["topk_ids"].cpu().numpy()
        assert check_union(SMALL, K, ids, out) > 4
        assert row_rel_err(out["y"].cpu().numpy(), want["y"].cpu().numpy()).max() <= 1e-5
        y_ref = O.moe_target(h.cpu().numpy().astype(np.float64), ref, forced_ids=ids)[0]
        assert row_rel_err(out["y"].cpu().numpy(), y_ref).max() <= Y_BF16
        model.stage_union(0, out["union_list"])
        for e in range(SMALL.n_experts):
            assert cache.query(0, e)[0] == model.slot_of(0, e)
    cache.close(); off.close(); resident.close()


@pytest.mark.parametrize("K,zipf,rho", [(4, True, 0.0), (8, False, 0.9), (16, True, 0.9), (16, False, 0.0)])
def test_wide_v2lite_layer(dxw, K, zipf, rho):
    sh = dataclasses.replace(synth.shape_v2lite(), weight_dtype=synth.DTYPE_BF16_WIDE)
    near, n_union = _verify_case(dxw, sh, K, seed=100 + K, zipf=zipf, rho=rho)
    assert sh.top_k <= n_union <= min(sh.n_experts, K * sh.top_k)
    if K == 4:
        _draft_case(dxw, sh, seed=100, zipf=zipf)


def test_wide_refusals(dxw):
    binding, ctx = dxw
    layer, _ = gpu_layer(SMALL, 90, std=0.08)
    L = binding.Layer.from_weights(ctx, layer)
    with pytest.raises(binding.DxError) as err:
        binding.DraftStack(ctx, [L])                         # the persistent draft stack reads the streaming layout
    assert err.value.status == 8
    L.close()


def test_wide_wait_for_a_routing_kernel_that_never_runs_expires(dxw):
    """The give-up path of the tcgen05 kernel: launched alone in hand-over mode, its bounded waits run out, it frees
    its tensor memory and returns with DX_DEV_WAIT_EXPIRED; the next ordinary block on the context is correct."""
    binding, ctx = dxw
    layer, ref = gpu_layer(SMALL, 92, std=0.08)
    L = binding.Layer.from_weights(ctx, layer)
    h = synth.hidden_block(12, SMALL.hidden, 93, 0.0, "cuda")
    ctx.set_wait_limit(2000)
    binding.selftest_wait_expiry(L, h, torch.empty_like(h))
    torch.cuda.synchronize()
    assert ctx.device_status() == 2
    ctx.set_wait_limit(0)
    out = binding.moe_verify_block(L, h)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    y_ref = O.moe_target(h.cpu().numpy().astype(np.float64), ref, forced_ids=out["topk_ids"].cpu().numpy())[0]
    assert row_rel_err(out["y"].cpu().numpy(), y_ref).max() <= Y_BF16
    L.close()


def test_wide_overlapped_pairs_in_a_row(dxw):
    """Routing / expert kernel pairs back to back from a CUDA graph (stack of residual layers, verify and draft): each
    expert kernel starts beside its routing kernel and takes block, groups and pairs through the hand-over."""
    binding, ctx = dxw
    sh = dataclasses.replace(SMALL, inter=200, shared_inter=72, draft_inter=64)
    n_layers, K = 4, 11
    refs, Ls = [], []
    for l in range(n_layers):
        layer, ref = gpu_layer(sh, 700 + 10 * l, std=0.08)
        refs.append(ref); Ls.append(binding.Layer.from_weights(ctx, layer))
    hs = [torch.zeros((K, sh.hidden), device="cuda") for _ in range(n_layers + 1)]
    hd = [torch.zeros((1, sh.hidden), device="cuda") for _ in range(n_layers + 1)]
    rb = [binding._routing_buffers(sh, K, "cuda") for _ in range(n_layers)]
    db = [{"topk_ids": torch.empty((sh.top_k,), dtype=torch.int32, device="cuda"),
           "topk_w": torch.empty((sh.top_k,), device="cuda")} for _ in range(n_layers)]

    def chain():
        for l in range(n_layers):
            binding.moe_draft_step_residual(Ls[l], hd[l], hd[l + 1], db[l])
        for l in range(n_layers):
            binding.moe_verify_block_residual(Ls[l], hs[l], hs[l + 1], rb[l])

    stream = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    with torch.cuda.stream(side):
        chain()
    stream.wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        chain()
    for rep in range(3):
        hs[0].copy_(synth.hidden_block(K, sh.hidden, 710 + rep, 0.5, "cuda"))
        hd[0].copy_(hs[0][:1])
        for _ in range(20):
            g.replay()
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        for l in range(n_layers):
            ids = rb[l]["topk_ids"].cpu().numpy()
            want = O.stack_layer_target(hs[l].cpu().numpy().astype(np.float64), refs[l], forced_ids=ids)[0]
            assert row_rel_err(hs[l + 1].cpu().numpy(), want).max() <= Y_BF16, (rep, l)
            check_union(sh, K, ids, rb[l])
            wantd = O.stack_layer_draft(hd[l].cpu().numpy().astype(np.float64), refs[l],
                                        forced_ids=db[l]["topk_ids"].cpu().numpy()[None])[0]
            assert row_rel_err(hd[l + 1].cpu().numpy(), wantd).max() <= Y_BF16, (rep, l)
    for L in Ls:
        L.close()
