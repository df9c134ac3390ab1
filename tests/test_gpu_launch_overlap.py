"""Context settings that move work in time or in the memory hierarchy, never what is computed.

Every setting of the launch-overlap mask (dx_set_launch_overlap: which kernels are launched with programmatic stream
serialization) gives the same results.  The default (routing + expert kernels) is what all other tests run; here the
verify block, the draft step, the residual chain and the greedy accept are compared with the CPU checker under no
overlap at all, each kernel kind alone, and all three.  Likewise dx_set_accept_l2_keep (cache hints of the LM head)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2607_24434_b200 import synth
from tests.helpers import Y_BF16, gpu_layer, row_rel_err
from tests.test_gpu_parity import SMALL, _accept_case, _draft_case, _verify_case

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=[0, 1, 2, 4, 7])
def dxm(request):
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    ctx.set_launch_overlap(request.param)
    ctx.y_tol = Y_BF16
    yield binding, ctx
    assert ctx.device_status() == 0
    ctx.close()


def test_refused_masks():
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    for bad in (-1, 8):
        with pytest.raises(binding.DxError) as err:
            ctx.set_launch_overlap(bad)
        assert err.value.status == 1
    ctx.close()


def test_block_draft_and_accept_under_the_mask(dxm):
    for K in (1, 4, 11):
        _verify_case(dxm, SMALL, K, seed=300 + K, std=0.08)
    _draft_case(dxm, SMALL, seed=310, std=0.08)
    wide = dataclasses.replace(SMALL, weight_dtype=synth.DTYPE_BF16_WIDE)
    _verify_case(dxm, wide, 9, seed=320, std=0.08)
    _draft_case(dxm, wide, seed=321, std=0.08)
    assert _accept_case(dxm, 5, 4, 4099, 256, torch.bfloat16, 330, rms=True, mode="mid") == 2
    assert _accept_case(dxm, 5, 4, 4099, 2048, torch.bfloat16, 331, rms=True, mode="mid") == 2   # (ring variant)


def test_back_to_back_steps_under_the_mask(dxm):
    """Draft step -> verify block -> accept, three times in a row on one stream without a host wait in between (the
    arrangement in which the overlap matters), on a DeepSeek-V2-Lite-shaped layer; every result against the checker."""
    binding, ctx = dxm
    shape = synth.shape_v2lite()
    layer, ref = gpu_layer(shape, 340, zipf=True)
    L = binding.Layer.from_weights(ctx, layer)
    V, K = 4099, 4
    W = synth.lm_head(V, shape.hidden, 341, torch.bfloat16, "cuda")
    W_np = synth.to_numpy_f32(W).astype(np.float64)
    blocks = [synth.hidden_block(K, shape.hidden, 342 + i, 0.5, "cuda") for i in range(3)]
    draft = torch.zeros((K,), dtype=torch.int32, device="cuda")
    outs = []
    for h in blocks:
        d = binding.moe_draft_step(L, h[:1])
        v = binding.moe_verify_block_residual(L, h)
        a = binding.spec_accept(ctx, v["h"], W, draft, rms_norm=True)
        outs.append((d, v, a))
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    for h, (d, v, a) in zip(blocks, outs):
        h_np = h.cpu().numpy().astype(np.float64)
        y_d = O.moe_draft(h_np[:1], ref, forced_ids=d["topk_ids"].cpu().numpy()[None])[0]
        assert row_rel_err(d["y"].cpu().numpy(), y_d).max() <= Y_BF16
        want = O.stack_layer_target(h_np, ref, forced_ids=v["topk_ids"].cpu().numpy())[0]
        assert row_rel_err(v["h"].cpu().numpy(), want).max() <= Y_BF16
        hn = O.rmsnorm(v["h"].cpu().numpy().astype(np.float64))
        t_ref, n_ref, next_ref, lg = O.greedy_accept_fast(hn, W_np, draft.cpu().numpy())
        srt = np.sort(lg, axis=1)
        clear = (srt[:, -1] - srt[:, -2]) > 1e-3
        assert np.array_equal(a["target"].cpu().numpy()[clear], t_ref[clear])
        if clear.all():
            assert int(a["n_accept"].item()) == n_ref and int(a["next_token"].item()) == next_ref
    L.close()


@pytest.mark.parametrize("keep_bytes", [1 << 20, 5 << 20, 1 << 30])
def test_accept_with_part_of_the_head_kept_in_l2(keep_bytes):
    """dx_set_accept_l2_keep only changes the cache hints of the loads: part of the matrix, a boundary inside it, and
    more than the whole matrix give the checker's tokens, repeatedly (the second and third calls are the ones that
    find lines in L2)."""
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    ctx.set_accept_l2_keep(keep_bytes)
    ctx.y_tol = Y_BF16
    for rep in range(3):
        assert _accept_case((binding, ctx), 9, 8, 3001, 1024, torch.bfloat16, 350, rms=True, mode="mid") == 4
    _accept_case((binding, ctx), 4, 4, 4099, 256, torch.bfloat16, 351, mode="geometric")
    # (blocks of at most eight rows at H = 2048 go through the ring variant of the kernel: hints on its bulk copies)
    for rep in range(2):
        assert _accept_case((binding, ctx), 5, 4, 148 * 16 * 3 + 9, 2048, torch.bfloat16, 352, rms=True, mode="mid") == 2
    assert ctx.device_status() == 0
    ctx.close()


def test_stage_block_and_results_written_to_the_host():
    """dx_stage_block moves pinned host bytes to the device (kernel path for small aligned sizes, copy engine
    otherwise, a page-able source refused), and the accept kernel may write its result words straight into pinned
    host memory: same tokens as with device outputs."""
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    for nbytes, offset in [(16, 0), (4 * 2048 * 4 + 16, 0), (1000, 0), (37, 0), (4096, 8), (3 << 20, 0)]:
        host = torch.empty((nbytes + offset,), dtype=torch.uint8).pin_memory()
        host.copy_(torch.randint(0, 256, (nbytes + offset,), dtype=torch.uint8))
        dst = torch.zeros((nbytes + 64,), dtype=torch.uint8, device="cuda")
        binding.stage_block(ctx, dst[:nbytes], host[offset:])
        torch.cuda.synchronize()
        assert torch.equal(dst[:nbytes].cpu(), host[offset:]) and int(dst[nbytes:].sum().item()) == 0, (nbytes, offset)
        # the host rewrites the buffer: the next transfer sees the new bytes
        host.add_(1)
        binding.stage_block(ctx, dst[:nbytes], host[offset:])
        torch.cuda.synchronize()
        assert torch.equal(dst[:nbytes].cpu(), host[offset:])
    with pytest.raises(binding.DxError) as err:
        binding.stage_block(ctx, torch.zeros((64,), dtype=torch.uint8, device="cuda"), torch.zeros((64,), dtype=torch.uint8))
    assert err.value.status == 1
    # greedy accept with its three outputs in pinned host memory
    M, K, V, H = 5, 4, 4099, 512
    W = synth.lm_head(V, H, 360, torch.bfloat16, "cuda")
    h = synth.hidden_block(M, H, 361, 0.5, "cuda")
    dev = binding.spec_accept(ctx, h, W, torch.zeros((K,), dtype=torch.int32, device="cuda"), rms_norm=True)
    torch.cuda.synchronize()
    draft = dev["target"][:K].clone()
    draft[2] = (draft[2] + 1) % V
    dev = binding.spec_accept(ctx, h, W, draft, rms_norm=True)
    res = torch.full((M + 2,), -7, dtype=torch.int32).pin_memory()
    out = {"target": res[:M], "n_accept": res[M:M + 1], "next_token": res[M + 1:M + 2]}
    binding.spec_accept(ctx, h, W, draft, rms_norm=True, out=out)
    torch.cuda.synchronize()
    assert torch.equal(res[:M], dev["target"].cpu())
    assert int(res[M]) == int(dev["n_accept"].item()) == 2 and int(res[M + 1]) == int(dev["next_token"].item())
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.parametrize("mask", [3, 7])
def test_step_graph_replays_are_stable(mask):
    """The benchmark's arrangement — draft step, verify block and greedy accept over the full 102 400-row vocabulary,
    captured once in a CUDA graph and replayed — gives, on every one of several hundred replays, the results of the
    first eager run (integer outputs bit for bit), and that run's target tokens are the checker's.  A race in one of
    the hand-overs between neighbouring kernels would show up as an occasional odd replay."""
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    ctx.set_launch_overlap(mask)
    shape = synth.shape_v2lite()
    K, V, NL = 4, 102400, 2
    layers = []
    for l in range(NL):
        w = synth.make_layer(shape, 380 + l, "cuda", zipf=True)
        layers.append(binding.Layer.from_weights(ctx, w))
        del w
    W = synth.lm_head(V, shape.hidden, 383, torch.bfloat16, "cuda")
    blocks = [synth.hidden_block(K, shape.hidden, 384 + l, 0.0, "cuda") for l in range(NL)]
    rb = [binding._routing_buffers(shape, K, "cuda") for _ in range(NL)]
    ys = [torch.empty((K, shape.hidden), device="cuda") for _ in range(NL)]
    yd = torch.empty((1, shape.hidden), device="cuda")
    dbuf = {"topk_ids": torch.empty((shape.top_k,), dtype=torch.int32, device="cuda"),
            "topk_w": torch.empty((shape.top_k,), device="cuda")}
    res = [torch.zeros((K + 2,), dtype=torch.int32, device="cuda") for _ in range(NL)]
    draft = torch.zeros((K,), dtype=torch.int32, device="cuda")

    def step(li):
        binding.moe_draft_step(layers[li], blocks[li][:1], yd, dbuf)
        binding.moe_verify_block(layers[li], blocks[li], ys[li], rb[li])
        binding.spec_accept(ctx, ys[li], W, draft, True,
                            {"target": res[li][:K], "n_accept": res[li][K:K + 1], "next_token": res[li][K + 1:K + 2]})

    for li in range(NL):
        step(li)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    want_res, want_y = [r.clone() for r in res], [y.clone() for y in ys]
    W_np = synth.to_numpy_f32(W).astype(np.float64)
    for li in range(NL):
        hn = O.rmsnorm(ys[li].cpu().numpy().astype(np.float64))
        t_ref, _, _, lg = O.greedy_accept_fast(hn, W_np, np.zeros(0, np.int32))
        srt = np.sort(lg, axis=1)
        clear = (srt[:, -1] - srt[:, -2]) > 1e-3
        assert np.array_equal(res[li][:K].cpu().numpy()[clear], t_ref[clear])
    stream = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for li in range(NL):
                step(li)
    stream.wait_stream(side)
    for it in range(300):
        for r in res:
            r.fill_(-9)
        g.replay()
        torch.cuda.synchronize()
        for li in range(NL):
            assert torch.equal(res[li], want_res[li]), (it, li)
            assert (ys[li] - want_y[li]).abs().max().item() <= 1e-4 * want_y[li].abs().max().item(), (it, li)
    assert ctx.device_status() == 0
    for L in layers:
        L.close()
    ctx.close()
