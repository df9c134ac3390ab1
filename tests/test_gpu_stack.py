"""Layer stacks (attention stubbed out, pre-norm residual MoE sub-layers): DeepSeek-V2-Lite-shaped and
Moonlight-shaped stacks, teacher-forced per layer -- the checker evaluates layer l on the GPU's own layer-l input
with the GPU's routing replayed, so one near-tie early on cannot turn the rest into a meaningless comparison --
followed by greedy verification on the normalised final hidden states."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2607_24434_b200 import synth
from tests.helpers import GAP, Y_BF16, Y_TIGHT, check_routing, check_union, row_rel_err

pytestmark = pytest.mark.gpu


def _run_stack(shape, n_layers, K, seed, zipf, vocab, act_split=True):
    """act_split False is the library's default (plain bf16 activations on the tensor cores): the verify block is then
    held to the bf16 bound; the single-token draft step runs the same kernel with one row."""
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0, act_split=act_split)
    tol = Y_TIGHT if act_split else Y_BF16
    h = synth.hidden_block(K, shape.hidden, seed, 0.9, "cuda")
    hd = h[:1].clone()
    unions, near_total = [], 0
    for l in range(n_layers):
        layer = synth.make_layer(shape, seed + 10 * l, "cuda", zipf=zipf)
        ref = synth.layer_to_numpy(layer)
        L = binding.Layer.from_weights(ctx, layer)
        del layer
        out = binding.moe_verify_block_residual(L, h)
        outd = binding.moe_draft_step_residual(L, hd)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        ids = out["topk_ids"].cpu().numpy()
        h_np = h.cpu().numpy().astype(np.float64)
        want, ids_ref, _, z_ref = O.stack_layer_target(h_np, ref)
        near_total += check_routing(shape, z_ref, ids_ref, ids)
        want = O.stack_layer_target(h_np, ref, forced_ids=ids)[0]
        assert row_rel_err(out["h"].cpu().numpy(), want).max() <= tol, l
        unions.append(check_union(shape, K, ids, out))
        wantd = O.stack_layer_draft(hd.cpu().numpy().astype(np.float64), ref,
                                    forced_ids=outd["topk_ids"].cpu().numpy()[None])[0]
        assert row_rel_err(outd["h"].cpu().numpy(), wantd).max() <= tol, l
        h, hd = out["h"], outd["h"]           # the stack alternates buffers: each layer's output feeds the next
        L.close()
    W = synth.lm_head(vocab, shape.hidden, seed + 999, torch.bfloat16, "cuda")
    hn = O.rmsnorm(h.cpu().numpy().astype(np.float64))
    tgt_ref, _, _, lg = O.greedy_accept_fast(hn, synth.to_numpy_f32(W).astype(np.float64), np.zeros(0, np.int32))
    draft = synth.draft_tokens_from_target(tgt_ref, vocab, seed)
    acc = binding.spec_accept(ctx, h, W, torch.from_numpy(draft).cuda(), rms_norm=True)
    torch.cuda.synchronize()
    tgt = acc["target"].cpu().numpy()
    srt = np.sort(lg, axis=1)
    for i in range(K):
        if srt[i, -1] - srt[i, -2] > GAP:
            assert tgt[i] == tgt_ref[i]
    n = 0
    while n < K and draft[n] == tgt[n]:
        n += 1
    assert int(acc["n_accept"].item()) == n
    ctx.close()
    return unions, near_total


@pytest.mark.parametrize("act_split", [True, False])
def test_v2lite_stack_correlated_block(act_split):
    sh = synth.shape_v2lite()
    unions, near = _run_stack(sh, 4, 8, seed=500, zipf=False, vocab=102400, act_split=act_split)
    # correlated block rows (rho = 0.9) share experts: unions grow sublinearly, far below the 48 pairs of K = 8
    assert all(sh.top_k <= u < 8 * sh.top_k for u in unions)
    assert np.mean(unions) < 30


def test_moonlight_stack_sigmoid_scaled():
    unions, near = _run_stack(synth.shape_moonlight(), 3, 4, seed=600, zipf=True, vocab=163840)
    assert all(6 <= u <= 24 for u in unions)


@pytest.mark.parametrize("act_split", [True, False])
def test_stack_graph_replay_handover(act_split):
    """Back-to-back launches from a CUDA graph: each expert kernel starts while the previous layer is still running
    and picks its block input and its routed groups up through the device-side hand-over.  Every replay gets a new
    input block; each layer's output is checked against the checker on that layer's own input and routing, so a
    kernel that ran ahead with the previous layer's work list or a half-written input fails."""
    from paper_2607_24434_b200 import binding
    sh = synth.shape_v2lite()
    n_layers, K = 4, 4
    ctx = binding.Context(0, act_split=act_split)
    tol = Y_TIGHT if act_split else Y_BF16
    refs, Ls = [], []
    for l in range(n_layers):
        layer = synth.make_layer(sh, 700 + 10 * l, "cuda", zipf=True)
        refs.append(synth.layer_to_numpy(layer))
        Ls.append(binding.Layer.from_weights(ctx, layer))
        del layer
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
        g.replay()
        g.replay()          # two replays in a row: the second must not be confused by what the first left behind
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        for l in range(n_layers):
            h_np = hs[l].cpu().numpy().astype(np.float64)
            ids = rb[l]["topk_ids"].cpu().numpy()
            want = O.stack_layer_target(h_np, refs[l], forced_ids=ids)[0]
            assert row_rel_err(hs[l + 1].cpu().numpy(), want).max() <= tol, (rep, l)
            check_union(sh, K, ids, rb[l])
            wantd = O.stack_layer_draft(hd[l].cpu().numpy().astype(np.float64), refs[l],
                                        forced_ids=db[l]["topk_ids"].cpu().numpy()[None])[0]
            assert row_rel_err(hd[l + 1].cpu().numpy(), wantd).max() <= tol, (rep, l)
    for L in Ls:
        L.close()
    ctx.close()


@pytest.mark.parametrize("K", [8, 3])
def test_many_overlapped_pairs_in_a_row(K):
    """Hundreds of routing / expert kernel pairs back to back from a CUDA graph with nothing in between (draft step,
    verify block and greedy accept on independent layers, as the benchmark's step): every pair's expert kernel lets
    the next routing kernel start while it is still working, so anything of the hand-over that is read after that
    point can be wiped under it (such a window is narrow: this is a soak, not a guaranteed catch).  No wait may
    expire, and what the last replay leaves behind must be what the same calls give when each one is synchronised."""
    from paper_2607_24434_b200 import binding
    sh = synth.shape_v2lite()
    n_layers = 3
    ctx = binding.Context(0)
    Ls, hs = [], []
    for l in range(n_layers):
        layer = synth.make_layer(sh, 800 + 10 * l, "cuda", zipf=True)
        Ls.append(binding.Layer.from_weights(ctx, layer))
        del layer
        hs.append(synth.hidden_block(K, sh.hidden, 810 + l, 0.0, "cuda"))
    W = synth.lm_head(4096, sh.hidden, 820, torch.bfloat16, "cuda")
    rb = [binding._routing_buffers(sh, K, "cuda") for _ in range(n_layers)]
    ys = [torch.empty((K, sh.hidden), device="cuda") for _ in range(n_layers)]
    yd = torch.empty((1, sh.hidden), device="cuda")
    db = {"topk_ids": torch.empty((sh.top_k,), dtype=torch.int32, device="cuda"),
          "topk_w": torch.empty((sh.top_k,), device="cuda")}
    dtok = torch.zeros((K,), dtype=torch.int32, device="cuda")
    ab = {"target": torch.empty((K,), dtype=torch.int32, device="cuda"),
          "n_accept": torch.empty((1,), dtype=torch.int32, device="cuda"),
          "next_token": torch.empty((1,), dtype=torch.int32, device="cuda")}

    def steps():
        # verify blocks directly one after the other (the tightest overlap: routing kernel N + 1 starts the moment
        # expert kernel N allows it), then the benchmark's step order
        for rep in range(4):
            for l in range(n_layers):
                binding.moe_verify_block(Ls[l], hs[l], ys[l], rb[l])
        for l in range(n_layers):
            binding.moe_draft_step(Ls[l], hs[l][:1], yd, db)
            binding.moe_verify_block(Ls[l], hs[l], ys[l], rb[l])
            binding.spec_accept(ctx, ys[l], W, dtok, True, ab)

    # reference: the same calls, one at a time
    want = []
    for l in range(n_layers):
        o = binding.moe_verify_block(Ls[l], hs[l])
        torch.cuda.synchronize()
        want.append((o["y"].clone(), o["topk_ids"].clone()))
    stream = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    with torch.cuda.stream(side):
        steps()
    stream.wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        steps()
    for _ in range(1000):
        g.replay()
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    for l in range(n_layers):
        assert torch.equal(rb[l]["topk_ids"], want[l][1])
        assert row_rel_err(ys[l].cpu().numpy(), want[l][0].cpu().numpy()).max() <= 1e-5
    ctx.close()
