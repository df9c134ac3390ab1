"""Layers whose experts stay 4-bit block-quantised in HBM (the weight format of the paper's mobile runs, Sec. 4)
and are de-quantised inside the expert kernel's streaming loop: verify blocks (Eq. 4) and the draft step (Eq. 5)
against the checker evaluated on the exact values d * (code - 8) of the same bytes."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2607_24434_b200 import synth
from tests.helpers import Y_TOL, check_routing, check_union, row_rel_err

# Codes and scales are used exactly; the activations go to the tensor cores as bf16 without their low halves (with
# 4-bit weights the tensor pipe sets the pace).  That is one rounding of at most 2^-9 relative per element, twice in
# a row (the normalised hidden row, then the SwiGLU activations); on these cases it leaves up to 5e-3 of the row
# maximum, half of what is asserted here and a quarter of the stated tolerance for layer outputs.
Q4_TOL = 1e-2

pytestmark = pytest.mark.gpu

SMALL = synth.LayerShape(hidden=512, n_experts=16, top_k=3, inter=64, n_shared=2, shared_inter=32, draft_inter=64,
                         score_fn=synth.SCORE_SOFTMAX, norm_topk=1, weight_dtype=synth.DTYPE_BF16)


def _fast_dequant(blocks: np.ndarray) -> np.ndarray:
    """Vectorised restatement of the checker's loop-by-loop dequantiser (pinned against it below)."""
    d = blocks[..., :2].copy().view("<f2").astype(np.float64)
    lo = (blocks[..., 2:] & 15).astype(np.float64) - 8
    hi = (blocks[..., 2:] >> 4).astype(np.float64) - 8
    v = np.concatenate([lo, hi], axis=-1) * d
    return v.reshape(*blocks.shape[:-2], blocks.shape[-2] * 32)


def _reference(layer_q4, dequant):
    """The quantised layer as the checker sees it: every expert matrix replaced by its exact 4-bit values."""
    def m(t):
        return dequant(t.cpu().numpy())
    ref = {"shape": layer_q4["shape"], "router": synth.to_numpy_f32(layer_q4["router"]),
           "bias": None if layer_q4["bias"] is None else synth.to_numpy_f32(layer_q4["bias"])}
    ref["shared"] = [tuple(m(w) for w in tr) for tr in layer_q4["shared"]]
    ref["draft"] = None if layer_q4["draft"] is None else tuple(m(w) for w in layer_q4["draft"])
    ref["experts"] = tuple(np.stack([m(w[e]) for e in range(w.shape[0])]) for w in layer_q4["experts"])
    return ref


def _case(shape, seed, Ks, dequant, std=0.05, zipf=False):
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    layer = synth.quantize_layer(synth.make_layer(shape, seed, "cuda", std=std, zipf=zipf))
    ref = _reference(layer, dequant)
    qshape = layer["shape"]
    assert binding.expert_blob_bytes(qshape, shape.inter) * 32 < binding.expert_blob_bytes(shape, shape.inter) * 11
    L = binding.Layer.from_weights(ctx, layer)
    for K in Ks:
        h = synth.hidden_block(K, shape.hidden, seed + K, 0.5, "cuda")
        out = binding.moe_verify_block(L, h)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        ids = out["topk_ids"].cpu().numpy()
        h_np = h.cpu().numpy().astype(np.float64)
        _, ids_ref, _, z_ref = O.moe_target(h_np, ref)
        check_routing(shape, z_ref, ids_ref, ids)
        check_union(shape, K, ids, out)
        want = O.moe_target(h_np, ref, forced_ids=ids)[0]
        err = row_rel_err(out["y"].cpu().numpy(), want).max()
        assert err <= Q4_TOL and err <= Y_TOL, (K, err)
    hd = synth.hidden_block(1, shape.hidden, seed + 99, 0.0, "cuda")
    outd = binding.moe_draft_step(L, hd)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    wantd = O.moe_draft(hd.cpu().numpy().astype(np.float64), ref,
                        forced_ids=outd["topk_ids"].cpu().numpy()[None])[0]
    assert row_rel_err(outd["y"].cpu().numpy().reshape(1, -1), wantd).max() <= Q4_TOL
    L.close()
    ctx.close()


def test_fast_dequantiser_matches_the_loops():
    rng = np.random.default_rng(5)
    w = torch.from_numpy((rng.standard_normal((5, 96)) * 0.05).astype(np.float32))
    blk = synth.quantize_q4_0(w).numpy()
    assert np.array_equal(_fast_dequant(blk), O.dequantize_q4_0(blk))


def test_q4_resident_small_loops():
    """Small layer, the checker's own loop-by-loop dequantiser; K = 12 takes the two-token-tile kernel."""
    _case(SMALL, 310, [1, 4, 8, 12], O.dequantize_q4_0)


def test_q4_resident_other_hidden_sizes():
    for H in (256, 1024):
        _case(dataclasses.replace(SMALL, hidden=H, n_experts=8, top_k=2, n_shared=1), 320 + H, [3, 16], _fast_dequant)


def test_q4_resident_v2lite_layer():
    _case(dataclasses.replace(synth.shape_v2lite(), n_experts=16), 330, [4, 8, 16], _fast_dequant, std=0.02, zipf=True)


def test_q4_sizes_and_refusals():
    from paper_2607_24434_b200 import binding
    q = dataclasses.replace(SMALL, weight_dtype=synth.DTYPE_Q4)
    # 4 bits per weight plus one fp16 scale per 32: gate / up 0.5625 B per weight, and the scales of W_d are
    # stored once per unit of eight columns: 0.75 B per weight there
    assert binding.expert_blob_bytes(q, 64) == 64 * (512 // 128 * 144 + 512 // 256 * 192)
    with pytest.raises(binding.DxError):
        binding.expert_blob_bytes(q, 40)          # not a multiple of the quantisation block
    ctx = binding.Context(0)
    with pytest.raises(binding.DxError):
        binding.Layer(ctx, dataclasses.replace(q, draft_inter=24))
    ctx.close()


@pytest.mark.parametrize("shape,n_layers", [(SMALL, 5), (dataclasses.replace(synth.shape_v2lite(), n_experts=16), 3)])
def test_q4_draft_stack(shape, n_layers):
    """The persistent draft stack on layers with 4-bit experts (fp32 activations, exact codes and scales)."""
    from paper_2607_24434_b200 import binding
    from tests.helpers import Y_TIGHT
    ctx = binding.Context(0)
    refs, layers = [], []
    for l in range(n_layers):
        lq = synth.quantize_layer(synth.make_layer(shape, 340 + 10 * l, "cuda", std=0.05 if shape is SMALL else 0.02))
        refs.append(_reference(lq, _fast_dequant))
        layers.append(binding.Layer.from_weights(ctx, lq))
    stack = binding.DraftStack(ctx, layers)
    h0 = synth.hidden_block(1, shape.hidden, 350, 0.0, "cuda")
    out = binding.moe_draft_stack(stack, h0)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ids = out["topk_ids"].cpu().numpy()
    h = h0.cpu().numpy().astype(np.float64)
    near = 0
    for l in range(n_layers):
        _, ids_ref, _, z_ref = O.stack_layer_draft(h, refs[l])
        near += check_routing(shape, z_ref, ids_ref, ids[l][None])
        h = O.stack_layer_draft(h, refs[l], forced_ids=ids[l][None])[0]
    assert row_rel_err(out["h"].cpu().numpy(), h).max() <= Y_TIGHT
    # mixing 4-bit and bf16 layers in one stack is refused
    b = binding.Layer.from_weights(ctx, synth.make_layer(shape, 399, "cuda"))
    with pytest.raises(binding.DxError):
        binding.DraftStack(ctx, [layers[0], b])
    stack.close()
    ctx.close()


def test_q4_experts_through_the_cache():
    """4-bit routed experts in a pinned host pool, staged into cache slots as they are (packed 4-bit units, a third
    of the bf16 bytes per miss) and de-quantised by the expert kernel: same results as with all experts resident."""
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    lq = synth.quantize_layer(synth.make_layer(SMALL, 360, "cuda", std=0.05))
    qshape = lq["shape"]
    resident = binding.Layer.from_weights(ctx, lq)
    off = binding.Layer.from_weights(ctx, lq, routed_resident=False)
    nbytes = binding.expert_blob_bytes(qshape, qshape.inter)
    host = off.blobs.cpu().pin_memory()
    cache = binding.ExpertCache(ctx, 1, qshape.n_experts, 4, nbytes)
    for e in range(qshape.n_experts):
        cache.register(0, e, host[e])
    cache.attach(off, 0)
    for step, K in enumerate([6, 3, 8]):
        h = synth.hidden_block(K, qshape.hidden, 370 + step, 0.5, "cuda")
        cache.begin_step()
        out = binding.moe_verify_block_cached(off, cache, 0, h)
        want = binding.moe_verify_block(resident, h)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        assert torch.equal(out["topk_ids"], want["topk_ids"])
        assert row_rel_err(out["y"].cpu().numpy(), want["y"].cpu().numpy()).max() <= 1e-5
    st = cache.stats()
    loads = st["on_demand"] + st["prefetch_issued"]
    assert loads > 0 and st["bytes_h2d"] == loads * nbytes
    assert nbytes * 3 < binding.expert_blob_bytes(SMALL, SMALL.inter)
    cache.close()
    ctx.close()
