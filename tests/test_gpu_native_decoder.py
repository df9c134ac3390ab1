"""dx_decoder_step (the decode step's host loop inside the library) against the same step made call by call from
Python (paper_2607_24434_b200/decode.py, which tests/test_gpu_offload_step.py checks against the CPU checker layer by
layer): two identical set-ups -- own layers, own host pool, own cache -- stepped side by side give the same drafted
tokens, accepted lengths, emitted tokens, union sizes, slot tables and cache statistics, step after step, with the
comparison's own accepted length and with a scripted one, with bf16 and with 4-bit host pools."""
import numpy as np
import pytest
import torch

from paper_2607_24434_b200 import synth

pytestmark = pytest.mark.gpu

SHAPE = synth.LayerShape(hidden=512, n_experts=16, top_k=3, inter=64, n_shared=1, shared_inter=64, draft_inter=64,
                         score_fn=synth.SCORE_SOFTMAX, norm_topk=1, weight_dtype=synth.DTYPE_BF16)
N_LAYERS, SLOTS, VOCAB, K_MAX = 4, 5, 1031, 6


def _setup(binding, ctx, q4):
    nbytes = binding.expert_blob_bytes(SHAPE, SHAPE.inter)
    cache = binding.ExpertCache(ctx, N_LAYERS, SHAPE.n_experts, SLOTS, nbytes)
    if q4:
        cache.set_q4(SHAPE)
    layers, pools = [], []
    for l in range(N_LAYERS):
        w = synth.make_layer(SHAPE, 9100 + l, "cuda", zipf=True, std=0.08)
        L = binding.Layer.from_weights(ctx, w, routed_resident=False)
        torch.cuda.synchronize()
        if q4:
            Wg, Wu, Wd = w["experts"]
            host = torch.stack([synth.q4_expert_blob(Wg[e].float().cpu(), Wu[e].float().cpu(), Wd[e].float().cpu())
                                for e in range(SHAPE.n_experts)]).pin_memory()
        else:
            host = L.blobs.cpu().pin_memory()
        L.blobs = None
        for e in range(SHAPE.n_experts):
            cache.register(l, e, host[e])
        cache.attach(L, l)
        layers.append(L); pools.append(host)
    return layers, cache, pools


@pytest.mark.parametrize("q4", [False, True])
def test_native_step_equals_the_python_loop(q4):
    from paper_2607_24434_b200 import binding, decode
    ctx = binding.Context(0)
    emb = synth.embedding_table(VOCAB, SHAPE.hidden, 9198, "cuda")
    W_lm = synth.lm_head(VOCAB, SHAPE.hidden, 9199, torch.bfloat16, "cuda")
    twins = []
    for native in (False, True):
        layers, cache, pools = _setup(binding, ctx, q4)
        dec = decode.OffloadedDecoder(ctx, layers, cache, emb, W_lm, k_max=K_MAX, tau=0.5, budget="cache", native=native)
        twins.append((dec, layers, cache, pools))
    rng = np.random.default_rng(3)
    t0 = 11
    for step in range(8):
        scripted = None if step % 3 == 0 else int(rng.integers(0, K_MAX + 1))
        res = [tw[0].step(t0, scripted_accept=scripted) for tw in twins]
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        for key in ("drafted", "n_accept", "emitted", "next", "block_rows", "union_sizes"):
            assert res[0][key] == res[1][key], (step, key, res[0][key], res[1][key])
        assert list(res[0]["target"][:res[0]["block_rows"]]) == list(res[1]["target"])
        for l in range(N_LAYERS):
            for e in range(SHAPE.n_experts):
                assert twins[0][2].query(l, e)[0] == twins[1][2].query(l, e)[0], (step, l, e)
        s0, s1 = twins[0][2].stats(), twins[1][2].stats()
        for key in ("lookups", "hits", "on_demand", "prefetch_issued", "prefetch_used", "prefetch_wasted", "evictions",
                    "bytes_h2d"):
            assert s0[key] == s1[key], (step, key)
        t0 = res[0]["next"]
    assert s0["on_demand"] > 0 and s0["prefetch_issued"] > 0 and s0["hits"] > 0
    for dec, layers, cache, _ in twins:
        dec.close(); cache.close()
        for L in layers:
            L.close()
    ctx.close()


def test_native_decoder_refuses_what_it_cannot_run():
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    layers, cache, pools = _setup(binding, ctx, False)
    emb = synth.embedding_table(VOCAB, SHAPE.hidden, 9198, "cuda")
    W_lm = synth.lm_head(VOCAB, SHAPE.hidden, 9199, torch.bfloat16, "cuda")
    with pytest.raises(binding.DxError) as err:                       # layers out of cache order
        binding.Decoder(ctx, layers[::-1], cache, emb, W_lm)
    assert err.value.status == 1
    with pytest.raises(binding.DxError) as err:                       # more draft tokens than a block holds
        binding.Decoder(ctx, layers, cache, emb, W_lm, k_max=17)
    assert err.value.status == 1
    with pytest.raises(ValueError):
        binding.Decoder(ctx, layers, cache, emb.float(), W_lm)
    cache.close()
    for L in layers:
        L.close()
    ctx.close()
