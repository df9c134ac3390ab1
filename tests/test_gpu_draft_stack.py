"""The drafter through a whole stack in one persistent launch (Eq. 5 per layer, pre-norm residual form): checked
layer by layer against the checker -- routing on the checker's own hidden row (exact outside near-ties), then the
checker advanced with the selection the kernel reported -- and against the chain of per-layer launches."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2607_24434_b200 import synth
from tests.helpers import Y_TIGHT, check_routing, row_rel_err

pytestmark = pytest.mark.gpu


def _stack_case(shape, n_layers, seed, zipf=False, reps=1):
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0, act_split=True)
    refs, layers = [], []
    for l in range(n_layers):
        w = synth.make_layer(shape, seed + 10 * l, "cuda", zipf=zipf)
        refs.append(synth.layer_to_numpy(w))
        layers.append(binding.Layer.from_weights(ctx, w))
        del w
    stack = binding.DraftStack(ctx, layers)
    for rep in range(reps):
        h0 = synth.hidden_block(1, shape.hidden, seed + 77 * rep, 0.0, "cuda")
        out = binding.moe_draft_stack(stack, h0)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        ids = out["topk_ids"].cpu().numpy()
        gates = out["topk_w"].cpu().numpy()
        # the checker, advanced with the kernel's own selection
        h = h0.cpu().numpy().astype(np.float64)
        near = 0
        for l in range(n_layers):
            _, ids_ref, _, z_ref = O.stack_layer_draft(h, refs[l])
            near += check_routing(shape, z_ref, ids_ref, ids[l][None])
            h, _, g_ref, _ = O.stack_layer_draft(h, refs[l], forced_ids=ids[l][None])
            assert np.allclose(gates[l], g_ref[0], rtol=2e-3, atol=1e-6), l
        assert near <= max(1, n_layers // 4)
        assert row_rel_err(out["h"].cpu().numpy(), h).max() <= Y_TIGHT
        # the chain of per-layer launches takes the same path (same selection => same row up to summation order)
        hc = h0
        same = True
        for l in range(n_layers):
            o = binding.moe_draft_step_residual(layers[l], hc)
            same = same and np.array_equal(o["topk_ids"].cpu().numpy(), ids[l])
            hc = o["h"]
        torch.cuda.synchronize()
        if same:
            assert row_rel_err(out["h"].cpu().numpy(), hc.cpu().numpy().astype(np.float64)).max() <= 2e-3
    stack.close()
    for L in layers:
        L.close()
    ctx.close()


def test_draft_stack_small_bf16():
    sh = dataclasses.replace(synth.shape_tiny(), weight_dtype=synth.DTYPE_BF16, n_experts=16, top_k=3)
    _stack_case(sh, 7, seed=910, reps=3)


def test_draft_stack_single_layer():
    sh = dataclasses.replace(synth.shape_tiny(), weight_dtype=synth.DTYPE_BF16, hidden=512, inter=256, shared_inter=256)
    _stack_case(sh, 1, seed=920)


def test_draft_stack_v2lite():
    _stack_case(synth.shape_v2lite(), 4, seed=930, reps=2)


def test_draft_stack_moonlight_zipf():
    _stack_case(synth.shape_moonlight(), 3, seed=940, zipf=True)


def test_draft_stack_wide_sigmoid_router_no_shared():
    """256 experts (eight logit words per lane), top-8, sigmoid scores with a routed scale, no shared expert."""
    sh = dataclasses.replace(synth.shape_tiny(), weight_dtype=synth.DTYPE_BF16, hidden=1024, n_experts=256, top_k=8,
                             n_shared=0, shared_inter=0, score_fn=synth.SCORE_SIGMOID, routed_scale=2.5)
    _stack_case(sh, 3, seed=950, zipf=True)


def test_draft_stack_graph_replay():
    """The launch (scratch clear + cooperative kernel) captured in a CUDA graph and replayed on new inputs."""
    from paper_2607_24434_b200 import binding
    sh = dataclasses.replace(synth.shape_tiny(), weight_dtype=synth.DTYPE_BF16, hidden=512, n_experts=32, top_k=4)
    ctx = binding.Context(0, act_split=True)
    refs, layers = [], []
    for l in range(5):
        w = synth.make_layer(sh, 960 + l, "cuda")
        refs.append(synth.layer_to_numpy(w))
        layers.append(binding.Layer.from_weights(ctx, w))
    stack = binding.DraftStack(ctx, layers)
    h_in = synth.hidden_block(1, sh.hidden, 1, 0.0, "cuda")
    out = binding.moe_draft_stack(stack, h_in)           # warm-up outside the capture (descriptor upload)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        binding.moe_draft_stack(stack, h_in, out["h"], out)
    for rep in range(3):
        h_in.copy_(synth.hidden_block(1, sh.hidden, 970 + rep, 0.0, "cuda"))
        g.replay()
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        ids = out["topk_ids"].cpu().numpy()
        h = h_in.cpu().numpy().astype(np.float64)
        for l in range(5):
            h = O.stack_layer_draft(h, refs[l], forced_ids=ids[l][None])[0]
        assert row_rel_err(out["h"].cpu().numpy(), h).max() <= Y_TIGHT, rep
    stack.close()
    ctx.close()


def test_draft_stack_refuses_mixed_shapes_and_fp32():
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0, act_split=True)
    a = binding.Layer.from_weights(ctx, synth.make_layer(synth.shape_tiny(), 1, "cuda"))
    with pytest.raises(binding.DxError):
        binding.DraftStack(ctx, [a])          # fp32 weights
    shb = dataclasses.replace(synth.shape_tiny(), weight_dtype=synth.DTYPE_BF16)
    b = binding.Layer.from_weights(ctx, synth.make_layer(shb, 2, "cuda"))
    c = binding.Layer.from_weights(ctx, synth.make_layer(dataclasses.replace(shb, n_experts=16), 3, "cuda"))
    with pytest.raises(binding.DxError):
        binding.DraftStack(ctx, [b, c])
    # routed experts not resident: the call (not the kernel) reports it
    d = binding.Layer.from_weights(ctx, synth.make_layer(shb, 4, "cuda"), routed_resident=False)
    st = binding.DraftStack(ctx, [b, d])
    with pytest.raises(binding.DxError):
        binding.moe_draft_stack(st, synth.hidden_block(1, shb.hidden, 5, 0.0, "cuda"))
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    st.close()
    for L in (a, b, c, d):
        L.close()
    ctx.close()


def test_draft_stack_many_launches_in_a_row():
    """Hundreds of persistent launches back to back (eager and from a CUDA graph): the scratch of one launch (delta
    rows, logit words, arrival counters) is cleared in stream order before the next; no wait may expire and every
    launch must leave the same row and the same selection."""
    from paper_2607_24434_b200 import binding
    sh = dataclasses.replace(synth.shape_v2lite(), n_experts=16)
    ctx = binding.Context(0)
    layers = [binding.Layer.from_weights(ctx, synth.make_layer(sh, 980 + l, "cuda")) for l in range(6)]
    stack = binding.DraftStack(ctx, layers)
    h0 = synth.hidden_block(1, sh.hidden, 990, 0.0, "cuda")
    first = binding.moe_draft_stack(stack, h0)
    torch.cuda.synchronize()
    want_h, want_ids = first["h"].clone(), first["topk_ids"].clone()
    out = {"topk_ids": torch.empty_like(want_ids), "topk_w": torch.empty_like(first["topk_w"])}
    h_out = torch.empty_like(want_h)
    for _ in range(200):
        binding.moe_draft_stack(stack, h0, h_out, out)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert torch.equal(out["topk_ids"], want_ids)
    assert row_rel_err(h_out.cpu().numpy(), want_h.cpu().numpy().astype(np.float64)).max() <= 1e-5
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        for _ in range(4):
            binding.moe_draft_stack(stack, h0, h_out, out)
    for _ in range(100):
        g.replay()
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert torch.equal(out["topk_ids"], want_ids)
    assert row_rel_err(h_out.cpu().numpy(), want_h.cpu().numpy().astype(np.float64)).max() <= 1e-5
    stack.close()
    ctx.close()
