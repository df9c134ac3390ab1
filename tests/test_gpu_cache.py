"""GPU parity of the offloaded path: routed experts in pinned host memory, staged through the HBM expert cache
(Sec. 3.5, Algorithm 1) in waves, against the CPU checker and against the same layer with all experts resident.
Prefetching and caching must never change results, only where a blob sits and when it moves."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from oracle.cache_oracle import ExpertCacheModel
from paper_2607_24434_b200 import synth
from tests.helpers import Y_TIGHT, check_union, gpu_layer, row_rel_err

pytestmark = pytest.mark.gpu

SHAPE = synth.LayerShape(hidden=512, n_experts=16, top_k=3, inter=40, n_shared=2, shared_inter=24, draft_inter=56,
                         score_fn=synth.SCORE_SOFTMAX, norm_topk=1, weight_dtype=synth.DTYPE_BF16)


def _offloaded_layer(binding, ctx, seed, slots):
    layer, ref = gpu_layer(SHAPE, seed, std=0.08)
    resident = binding.Layer.from_weights(ctx, layer)
    off = binding.Layer.from_weights(ctx, layer, routed_resident=False)
    torch.cuda.synchronize()
    host = off.blobs.cpu().pin_memory()                      # the host pool: one pinned blob per routed expert
    cache = binding.ExpertCache(ctx, 1, SHAPE.n_experts, slots, host.shape[1])
    for e in range(SHAPE.n_experts):
        cache.register(0, e, host[e])
    cache.attach(off, 0)
    return ref, resident, off, cache, host


@pytest.mark.parametrize("act_split", [True, False])
def test_cached_verify_matches_resident_and_checker(act_split):
    from paper_2607_24434_b200 import binding
    from tests.helpers import Y_BF16
    ctx = binding.Context(0, act_split=act_split)
    ref, resident, off, cache, host = _offloaded_layer(binding, ctx, 70, slots=4)
    model = ExpertCacheModel(1, SHAPE.n_experts, 4)
    for step, K in enumerate([6, 6, 3, 8]):
        h = synth.hidden_block(K, SHAPE.hidden, 80 + step, 0.5, "cuda")
        cache.begin_step(); model.begin_step()
        if step >= 1:                                        # prefetch what the drafter's router predicts
            d = binding.moe_draft_step(resident, h[:1].contiguous())
            torch.cuda.synchronize()
            pred = d["topk_ids"].tolist()
            cache.prefetch(0, pred); model.prefetch(0, pred)
        out = binding.moe_verify_block_cached(off, cache, 0, h)
        want = binding.moe_verify_block(resident, h)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        assert torch.equal(out["topk_ids"], want["topk_ids"])
        ids = out["topk_ids"].cpu().numpy()
        n = check_union(SHAPE, K, ids, out)
        assert n > 4                                          # more union experts than slots: several waves
        # same arithmetic either way; only the order of the fp32 reductions into y differs between launches
        assert row_rel_err(out["y"].cpu().numpy(), want["y"].cpu().numpy()).max() <= 1e-5
        y_ref = O.moe_target(h.cpu().numpy().astype(np.float64), ref, forced_ids=ids)[0]
        assert row_rel_err(out["y"].cpu().numpy(), y_ref).max() <= (Y_TIGHT if act_split else Y_BF16)
        union = out["union_list"]
        assert union == out["union_ids"].cpu().numpy()[:n].tolist()
        model.stage_union(0, union)                          # held experts first, then the misses by ascending id
        for e in range(SHAPE.n_experts):                     # the library's slot table follows the host model
            assert cache.query(0, e)[0] == model.slot_of(0, e)
    st = cache.stats()
    for key in ("lookups", "hits", "on_demand", "prefetch_issued", "prefetch_used", "prefetch_wasted", "evictions"):
        assert st[key] == model.stats[key], key
    assert st["bytes_h2d"] == (st["on_demand"] + st["prefetch_issued"]) * host.shape[1]
    cache.close(); ctx.close()


def test_cached_draft_step_and_errors():
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0, act_split=True)
    ref, resident, off, cache, host = _offloaded_layer(binding, ctx, 71, slots=2)
    h = synth.hidden_block(1, SHAPE.hidden, 90, 0.0, "cuda")
    y = torch.empty_like(h)
    out = {"topk_ids": torch.empty((SHAPE.top_k,), dtype=torch.int32, device="cuda"),
           "topk_w": torch.empty((SHAPE.top_k,), dtype=torch.float32, device="cuda")}
    binding.moe_draft_route(off, h, y, out)
    e1 = int(out["topk_ids"][0].item())                      # the host round trip on-demand loading needs
    with pytest.raises(binding.DxError) as err:
        cache.wait(0, [e1])                                  # never prefetched: wait does not load
    assert err.value.status == 5
    cache.stage(0, [e1])
    binding.moe_draft_experts(off, h, y)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    want = O.moe_draft(h.cpu().numpy().astype(np.float64), ref, forced_ids=out["topk_ids"].cpu().numpy()[None])[0]
    assert row_rel_err(y.cpu().numpy(), want).max() <= Y_TIGHT
    cache.wait(0, [e1], timeout_s=5.0)                       # resident now: returns at once
    # the same step as one call of the library (route, read the selection on the host, stage e1, experts)
    got = binding.moe_draft_step_cached(off, h)
    torch.cuda.synchronize()
    assert got["host_ids"] == out["topk_ids"].tolist()
    assert row_rel_err(got["y"].cpu().numpy(), want).max() <= Y_TIGHT
    # ... and in the pre-norm residual form the layer stacks use
    got = binding.moe_draft_step_cached(off, h, residual=True)
    res = binding.moe_draft_step_residual(resident, h)
    torch.cuda.synchronize()
    assert got["host_ids"] == res["topk_ids"].tolist()
    assert row_rel_err(got["h"].cpu().numpy(), res["h"].cpu().numpy()).max() <= 1e-5
    # an expert that was never staged is reported through the status word, not by a fault
    other = (e1 + 1) % SHAPE.n_experts
    assert cache.query(0, other)[0] == -1
    cache.close(); ctx.close()


def test_slow_transfer_times_out_and_then_completes():
    """A transfer that is slow (made on the host: a sleeping host callback queued on the copy stream in front of the
    prefetch) makes the bounded wait of expert_cache_wait return DX_ERR_TIMEOUT; a later wait with time to spare
    succeeds, and the results equal those of the resident layer."""
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0, act_split=True)
    ref, resident, off, cache, host = _offloaded_layer(binding, ctx, 72, slots=4)
    h = synth.hidden_block(1, SHAPE.hidden, 91, 0.0, "cuda")
    want = binding.moe_draft_step(resident, h)
    torch.cuda.synchronize()
    ids = want["topk_ids"].tolist()
    cache.begin_step()
    cache.inject_transfer_delay(150)                         # the link stalls for 150 ms ...
    cache.prefetch(0, ids[:1])                               # ... with the predicted expert's copy behind it
    with pytest.raises(binding.DxError) as err:
        cache.wait(0, ids[:1], timeout_s=0.005)
    assert err.value.status == 6                             # DX_ERR_TIMEOUT
    st = cache.stats()
    assert st["waited_copies"] >= 1 and st["stall_ns"] >= 4_000_000
    cache.wait(0, ids[:1], timeout_s=10.0)                   # the copy lands once the stall is over
    y = torch.empty_like(h)
    out = {"topk_ids": torch.empty((SHAPE.top_k,), dtype=torch.int32, device="cuda"),
           "topk_w": torch.empty((SHAPE.top_k,), dtype=torch.float32, device="cuda")}
    binding.moe_draft_route(off, h, y, out)
    binding.moe_draft_experts(off, h, y)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert out["topk_ids"].tolist() == ids
    assert row_rel_err(y.cpu().numpy(), want["y"].cpu().numpy()).max() <= 1e-5
    cache.close(); ctx.close()


def test_stream_wait_for_a_slow_copy_is_timed_on_the_device():
    """A block that needs an expert whose copy is stuck behind a 60 ms stall of the link: the compute stream waits for
    it (no host wait), the result is right, and the statistics show the wait -- at least most of the stall, measured by
    events on the stream."""
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0, act_split=True)
    ref, resident, off, cache, host = _offloaded_layer(binding, ctx, 74, slots=4)
    h = synth.hidden_block(1, SHAPE.hidden, 92, 0.0, "cuda")
    want = binding.moe_draft_step(resident, h)
    torch.cuda.synchronize()
    ids = want["topk_ids"].tolist()
    cache.begin_step()
    assert cache.stats()["stream_stall_ns"] == 0
    cache.inject_transfer_delay(60)
    cache.prefetch(0, ids[:1])
    out = binding.moe_draft_step_cached(off, h)              # returns once its kernels are queued behind the copy
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert out["host_ids"] == ids
    assert row_rel_err(out["y"].cpu().numpy(), want["y"].cpu().numpy()).max() <= 1e-5
    st = cache.stats()
    assert st["waited_copies"] >= 1 and 30_000_000 <= st["stream_stall_ns"] <= 500_000_000, st
    cache.close(); ctx.close()


def test_layer_destroyed_before_its_cache():
    """Either side may go first: a destroyed layer is forgotten by its cache (no patch is sent to a freed table)."""
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    ref, resident, off, cache, host = _offloaded_layer(binding, ctx, 73, slots=4)
    cache.prefetch(0, [1, 2])
    off.close()                                              # table patches for 1 and 2 were still pending
    cache.stage(0, [3])
    torch.cuda.synchronize()
    assert cache.query(0, 3)[0] >= 0
    cache.close(); ctx.close()
