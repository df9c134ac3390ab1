"""4-bit block-quantised routed experts (the weight format of the paper's mobile runs, Sec. 4) on the GPU:
the expansion of a quantised expert into the bf16 streaming blob is compared bit for bit with the packed blob of
the checker's dequantised weights rounded to bf16, and a verify block whose routed experts come out of a quantised
host pool through the expert cache is compared with the checker evaluated on the exact quantised values."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2607_24434_b200 import synth
from tests.helpers import Y_TOL, check_union, gpu_layer, row_rel_err

pytestmark = pytest.mark.gpu

SHAPE = synth.LayerShape(hidden=512, n_experts=16, top_k=3, inter=64, n_shared=2, shared_inter=24, draft_inter=56,
                         score_fn=synth.SCORE_SOFTMAX, norm_topk=1, weight_dtype=synth.DTYPE_BF16)


def _bf16_of(values: np.ndarray) -> torch.Tensor:
    """float64 values -> bf16 tensor, rounded to nearest even once (each value is fp16 * small integer, so the
    float32 step in between is exact)."""
    return torch.from_numpy(values.astype(np.float32)).to(torch.bfloat16)


@pytest.mark.parametrize("H,I", [(512, 64), (256, 32), (2048, 1408)])
def test_expand_q4_is_pack_of_dequantised(H, I):
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0, act_split=True)
    sh = dataclasses.replace(SHAPE, hidden=H, inter=I)
    Wg = synth.normal((I, H), 0.02, 7, "q4.g", torch.float32)
    Wu = synth.normal((I, H), 0.02, 7, "q4.u", torch.float32)
    Wd = synth.normal((H, I), 0.02, 7, "q4.d", torch.float32)
    blob_q4 = synth.q4_expert_blob(Wg, Wu, Wd)
    assert blob_q4.numel() == binding.q4_expert_bytes(sh, I) == 3 * H * I * 18 // 32
    got = binding.expand_q4_expert(ctx, sh, I, blob_q4.cuda())
    # the checker's values of the same bytes, rounded to bf16, through the ordinary packer
    n_gu = I * (H // 32) * 18
    deq = [O.dequantize_q4_0(blob_q4[:n_gu].numpy().reshape(I, H // 32, 18)) if (H, I) != (2048, 1408) else None,
           None, None]
    if deq[0] is None:
        # full-size expert: the loop-by-loop dequantiser is too slow; use its vectorised restatement, which the
        # small cases of this test pin against the loops
        def fast(b, R, Ccols):
            blk = b.numpy().reshape(R, Ccols // 32, 18)
            d = blk[:, :, :2].copy().view("<f2").astype(np.float64)
            lo = (blk[:, :, 2:] & 15).astype(np.float64) - 8
            hi = (blk[:, :, 2:] >> 4).astype(np.float64) - 8
            return (np.concatenate([lo, hi], axis=2) * d).reshape(R, Ccols)
        g, u, dn = fast(blob_q4[:n_gu], I, H), fast(blob_q4[n_gu:2 * n_gu], I, H), fast(blob_q4[2 * n_gu:], H, I)
    else:
        g = deq[0]
        u = O.dequantize_q4_0(blob_q4[n_gu:2 * n_gu].numpy().reshape(I, H // 32, 18))
        dn = O.dequantize_q4_0(blob_q4[2 * n_gu:].numpy().reshape(H, I // 32, 18))
    want = binding.pack_expert(ctx, sh, _bf16_of(g).cuda(), _bf16_of(u).cuda(), _bf16_of(dn).cuda())
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    ctx.close()


def test_fast_dequantiser_used_above_matches_the_loops():
    rng = np.random.default_rng(3)
    w = torch.from_numpy((rng.standard_normal((6, 128)) * 0.05).astype(np.float32))
    blk = synth.quantize_q4_0(w).numpy()
    d = blk[:, :, :2].copy().view("<f2").astype(np.float64)
    lo = (blk[:, :, 2:] & 15).astype(np.float64) - 8
    hi = (blk[:, :, 2:] >> 4).astype(np.float64) - 8
    assert np.array_equal((np.concatenate([lo, hi], axis=2) * d).reshape(6, 128), O.dequantize_q4_0(blk))


def test_verify_block_from_quantised_host_pool():
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0, act_split=True)
    layer, ref = gpu_layer(SHAPE, 75, std=0.08)
    Wg, Wu, Wd = layer["experts"]
    E = SHAPE.n_experts
    q4 = torch.stack([synth.q4_expert_blob(Wg[e].float().cpu(), Wu[e].float().cpu(), Wd[e].float().cpu())
                      for e in range(E)])
    # the checker sees the exact quantised values (not rounded to bf16) for the routed experts
    n_gu = SHAPE.inter * (SHAPE.hidden // 32) * 18
    ref_q = dict(ref)
    ref_q["experts"] = (
        np.stack([O.dequantize_q4_0(q4[e, :n_gu].numpy().reshape(SHAPE.inter, -1, 18)) for e in range(E)]),
        np.stack([O.dequantize_q4_0(q4[e, n_gu:2 * n_gu].numpy().reshape(SHAPE.inter, -1, 18)) for e in range(E)]),
        np.stack([O.dequantize_q4_0(q4[e, 2 * n_gu:].numpy().reshape(SHAPE.hidden, -1, 18)) for e in range(E)]))
    off = binding.Layer.from_weights(ctx, layer, routed_resident=False)
    host = q4.pin_memory()
    slots = 4
    cache = binding.ExpertCache(ctx, 1, E, slots, binding.expert_blob_bytes(SHAPE, SHAPE.inter))
    cache.set_q4(SHAPE)
    for e in range(E):
        cache.register(0, e, host[e])
    cache.attach(off, 0)
    loads = 0
    for step, K in enumerate([6, 3, 8, 5, 7]):
        h = synth.hidden_block(K, SHAPE.hidden, 85 + step, 0.5, "cuda")
        cache.begin_step()
        if step >= 2:
            # copies (and their expansions, on a stream of their own) still in flight when the block asks for them
            cache.prefetch(0, [(3 * step + j) % E for j in range(3)])
        out = binding.moe_verify_block_cached(off, cache, 0, h)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        ids = out["topk_ids"].cpu().numpy()
        check_union(SHAPE, K, ids, out)
        y_ref = O.moe_target(h.cpu().numpy().astype(np.float64), ref_q, forced_ids=ids)[0]
        # on top of the bf16 path's own error every expanded weight carries one rounding to bf16: at most 2^-9
        # relative per weight, through three matrices in a row; 2^-8 of the row maximum bounds what is left of it
        assert row_rel_err(out["y"].cpu().numpy(), y_ref).max() <= Y_TOL
        assert row_rel_err(out["y"].cpu().numpy(), y_ref).max() <= 2.0 ** -8
    st = cache.stats()
    loads = st["on_demand"] + st["prefetch_issued"]
    assert loads > 0 and st["bytes_h2d"] == loads * host.shape[1]       # only the quantised bytes cross the link
    # the pool's format cannot change once experts are registered, and sizes are checked
    with pytest.raises(binding.DxError):
        cache.set_q4(SHAPE)
    other = binding.ExpertCache(ctx, 1, E, slots, binding.expert_blob_bytes(SHAPE, SHAPE.inter))
    with pytest.raises(binding.DxError):
        other.set_q4(dataclasses.replace(SHAPE, inter=96))
    other.close(); cache.close(); ctx.close()
