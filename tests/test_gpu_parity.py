"""GPU parity: the CUDA library, called through its C ABI, against the CPU checker on the same seeded
inputs.  Integer outputs (top-k ids, union, offsets, permutation, target tokens, accepted length) must be
bit-exact wherever the checker's logit gap exceeds 1e-3; gate weights within 1e-5 * scale; layer outputs within
a max relative error of 2e-2 per row (and, for this implementation, within the much tighter regression bound)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2607_24434_b200 import synth
from tests.helpers import (GAP, GATE_TOL, Y_BF16, Y_TIGHT, Y_TOL, check_routing, check_union, gpu_layer, row_rel_err)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=["bf16_activations", "split_activations"])
def dx(request):
    """Every case runs in both evaluation modes of the bf16 expert kernel: the default (activations as plain bf16
    on the tensor cores, the mode the benchmark times) and the high + residual split.  ``ctx.y_tol`` is the bound
    on layer outputs that goes with the mode; fp32 layers are exact in both."""
    from paper_2607_24434_b200 import binding
    split = request.param == "split_activations"
    ctx = binding.Context(0, act_split=split)
    ctx.y_tol = Y_TIGHT if split else Y_BF16
    yield binding, ctx
    assert ctx.device_status() == 0
    ctx.close()


def _verify_case(dx, shape, K, seed, zipf=False, std=0.02, rho=0.0):
    binding, ctx = dx
    layer, ref = gpu_layer(shape, seed, zipf=zipf, std=std)
    L = binding.Layer.from_weights(ctx, layer)
    h = synth.hidden_block(K, shape.hidden, seed + 1, rho, "cuda")
    out = binding.moe_verify_block(L, h)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ids_gpu = out["topk_ids"].cpu().numpy()
    h_np = h.cpu().numpy().astype(np.float64)
    y_free, ids_ref, g_ref, z_ref = O.moe_target(h_np, ref)
    near = check_routing(shape, z_ref, ids_ref, ids_gpu)
    # downstream of routing everything is compared with the checker replaying the GPU's selection
    y_ref, _, g_forced, _ = O.moe_target(h_np, ref, forced_ids=ids_gpu)
    assert np.abs(out["topk_w"].cpu().numpy() - g_forced).max() <= GATE_TOL * max(1.0, shape.routed_scale)
    n_union = check_union(shape, K, ids_gpu, out)
    err = row_rel_err(out["y"].cpu().numpy(), y_ref)
    assert err.max() <= Y_TOL, err
    assert err.max() <= ctx.y_tol, err
    # run-to-run: integer outputs identical, float outputs differ only by reduction order
    out2 = binding.moe_verify_block(L, h)
    torch.cuda.synchronize()
    assert torch.equal(out2["topk_ids"], out["topk_ids"]) and torch.equal(out2["perm"], out["perm"])
    assert row_rel_err(out2["y"].cpu().numpy(), out["y"].cpu().numpy()).max() <= 1e-5
    L.close()
    return near, n_union


def _draft_case(dx, shape, seed, zipf=False, std=0.02):
    binding, ctx = dx
    layer, ref = gpu_layer(shape, seed, zipf=zipf, std=std)
    L = binding.Layer.from_weights(ctx, layer)
    h = synth.hidden_block(1, shape.hidden, seed + 2, 0.0, "cuda")
    out = binding.moe_draft_step(L, h)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ids_gpu = out["topk_ids"].cpu().numpy()[None]
    h_np = h.cpu().numpy().astype(np.float64)
    _, ids_ref, _, z_ref = O.moe_draft(h_np, ref)
    check_routing(shape, z_ref, ids_ref, ids_gpu)
    y_ref, _, g_forced, _ = O.moe_draft(h_np, ref, forced_ids=ids_gpu)
    assert np.abs(out["topk_w"].cpu().numpy()[None] - g_forced).max() <= GATE_TOL * max(1.0, shape.routed_scale)
    err = row_rel_err(out["y"].cpu().numpy(), y_ref)
    assert err.max() <= Y_TOL and err.max() <= ctx.y_tol, err
    L.close()


# ------------------------------------------------------------------ tiny fp32 layer (config 0)
def test_tiny_fp32_verify_and_draft(dx):
    sh = synth.shape_tiny()
    near, n_union = _verify_case(dx, sh, 4, seed=0)
    assert 2 <= n_union <= 8
    _draft_case(dx, sh, seed=0)
    _verify_case(dx, sh, 1, seed=3)
    _verify_case(dx, sh, 16, seed=4, std=0.1)


def test_tiny_fp32_sigmoid_unnormalised(dx):
    sh = dataclasses.replace(synth.shape_tiny(), score_fn=synth.SCORE_SIGMOID, norm_topk=0, routed_scale=2.5,
                             draft_gamma=0.5, top_k=3)
    _verify_case(dx, sh, 5, seed=5, std=0.1)
    _draft_case(dx, sh, seed=5, std=0.1)


# ------------------------------------------------------------------ small bf16 layers: several tiles + ragged sizes
SMALL = synth.LayerShape(hidden=512, n_experts=16, top_k=3, inter=40, n_shared=2, shared_inter=24, draft_inter=56,
                         score_fn=synth.SCORE_SOFTMAX, norm_topk=1, weight_dtype=synth.DTYPE_BF16)


@pytest.mark.parametrize("K", [1, 2, 4, 7, 8, 9, 16])
def test_small_bf16_verify(dx, K):
    _verify_case(dx, SMALL, K, seed=10 + K, std=0.08)


@pytest.mark.parametrize("H", [256, 1024])
def test_small_bf16_other_hidden(dx, H):
    sh = dataclasses.replace(SMALL, hidden=H, n_experts=130, top_k=8, inter=16, score_fn=synth.SCORE_SIGMOID,
                             routed_scale=2.446)
    _verify_case(dx, sh, 6, seed=20, std=0.08)
    _verify_case(dx, sh, 12, seed=21, std=0.08, zipf=True)
    _draft_case(dx, sh, seed=22, std=0.08)


def test_small_bf16_draft_and_no_shared(dx):
    _draft_case(dx, SMALL, seed=30, std=0.08)
    sh = dataclasses.replace(SMALL, n_shared=0, shared_inter=0, draft_inter=0)
    _verify_case(dx, sh, 4, seed=31, std=0.08)
    _draft_case(dx, sh, seed=32, std=0.08)


def test_duplicate_rows_and_degenerate_blocks(dx):
    binding, ctx = dx
    layer, ref = gpu_layer(SMALL, 40, std=0.08)
    L = binding.Layer.from_weights(ctx, layer)
    h1 = synth.hidden_block(1, SMALL.hidden, 41, 0.0, "cuda")
    h = h1.repeat(8, 1).contiguous()
    out = binding.moe_verify_block(L, h)
    torch.cuda.synchronize()
    assert int(out["union_count"].item()) == SMALL.top_k          # identical rows: the union does not grow
    y = out["y"].cpu().numpy()
    assert row_rel_err(y[1:], np.repeat(y[:1], 7, 0)).max() <= 1e-5
    z = torch.zeros_like(h)
    out0 = binding.moe_verify_block(L, z)
    torch.cuda.synchronize()
    assert float(out0["y"].abs().max()) == 0.0                     # h = 0 -> y = 0
    assert ctx.device_status() == 0
    L.close()


def test_detached_expert_is_reported_not_trapped(dx):
    binding, ctx = dx
    layer, ref = gpu_layer(SMALL, 50, std=0.08)
    L = binding.Layer.from_weights(ctx, layer)
    h = synth.hidden_block(4, SMALL.hidden, 51, 0.0, "cuda")
    out = binding.moe_verify_block(L, h)
    torch.cuda.synchronize()
    victim = int(out["union_ids"][0].item())
    L.set_expert(victim, None)
    out2 = binding.moe_verify_block(L, h)
    torch.cuda.synchronize()
    assert ctx.device_status() == 1                                # DX_DEV_BAD_EXPERT_ID, and the context still works
    ids = out2["topk_ids"].cpu().numpy()
    y_ref = O.moe_target(h.cpu().numpy().astype(np.float64), ref, forced_ids=ids)[0]
    rows = [t for t in range(4) if victim not in ids[t]]
    if rows:
        assert row_rel_err(out2["y"].cpu().numpy()[rows], y_ref[rows]).max() <= ctx.y_tol
    assert ctx.device_status() == 0
    L.close()


def test_shared_plus_top_r_drafter(dx):
    """The training-free shared + top-r drafter of Sec. 2.2 (r = 1..3) and r = k, which is the target layer."""
    binding, ctx = dx
    for shape, std in ((SMALL, 0.08), (synth.shape_tiny(), 0.1)):
        layer, ref = gpu_layer(shape, 33, std=std)
        L = binding.Layer.from_weights(ctx, layer)
        h = synth.hidden_block(1, shape.hidden, 34, 0.0, "cuda")
        h_np = h.cpu().numpy().astype(np.float64)
        for r, use_d in [(1, False), (2, False), (shape.top_k, False), (2, True)]:
            out = binding.moe_draft_step_topr(L, h, r, use_d)
            torch.cuda.synchronize()
            ids = out["topk_ids"].cpu().numpy()[None]
            want = O.moe_draft(h_np, ref, forced_ids=ids, top_r=r, gamma=None if use_d else 0.0)[0]
            assert row_rel_err(out["y"].cpu().numpy(), want).max() <= ctx.y_tol, (r, use_d)
            if r == shape.top_k and not use_d:
                target = O.moe_target(h_np, ref, forced_ids=ids)[0]
                assert row_rel_err(out["y"].cpu().numpy(), target).max() <= ctx.y_tol
        assert ctx.device_status() == 0
        L.close()


# ------------------------------------------------------------------ residual (stack) forms
def test_residual_forms(dx):
    binding, ctx = dx
    layer, ref = gpu_layer(SMALL, 60, std=0.08)
    L = binding.Layer.from_weights(ctx, layer)
    h = synth.hidden_block(6, SMALL.hidden, 61, 0.9, "cuda") * 3.0
    h_np = h.cpu().numpy().astype(np.float64)
    out = binding.moe_verify_block_residual(L, h)
    torch.cuda.synchronize()
    ids = out["topk_ids"].cpu().numpy()
    want = O.stack_layer_target(h_np, ref, forced_ids=ids)[0]
    assert row_rel_err(out["h"].cpu().numpy(), want).max() <= ctx.y_tol
    assert torch.equal(h.cpu(), torch.from_numpy(h_np.astype(np.float32)))      # the input block is untouched
    outd = binding.moe_draft_step_residual(L, h[:1])
    torch.cuda.synchronize()
    wantd = O.stack_layer_draft(h_np[:1], ref, forced_ids=outd["topk_ids"].cpu().numpy()[None])[0]
    assert row_rel_err(outd["h"].cpu().numpy(), wantd).max() <= ctx.y_tol
    # the shared + top-r self-drafter in the same form: h + drafter(RMSNorm(h)), r = 2, without the draft expert
    buf = {"topk_ids": torch.empty((SMALL.top_k,), dtype=torch.int32, device="cuda"),
           "topk_w": torch.empty((SMALL.top_k,), dtype=torch.float32, device="cuda")}
    h1, h2 = h[:1].contiguous(), torch.empty((1, SMALL.hidden), device="cuda")
    binding.moe_draft_step_topr_residual(L, h1, h2, 2, False, buf)
    torch.cuda.synchronize()
    y_r = O.moe_draft(O.rmsnorm(h_np[:1]), ref, forced_ids=buf["topk_ids"].cpu().numpy()[None], top_r=2, gamma=0.0)[0]
    assert row_rel_err(h2.cpu().numpy(), h_np[:1] + y_r).max() <= ctx.y_tol
    assert ctx.device_status() == 0
    L.close()


# ------------------------------------------------------------------ full DeepSeek-V2-Lite-shaped layer (config 1)
@pytest.mark.parametrize("K,zipf,rho", [(4, True, 0.0), (8, False, 0.9), (16, True, 0.9)])
def test_v2lite_layer_verify_and_draft(dx, K, zipf, rho):
    sh = synth.shape_v2lite()
    near, n_union = _verify_case(dx, sh, K, seed=100 + K, zipf=zipf, rho=rho)
    assert sh.top_k <= n_union <= min(sh.n_experts, K * sh.top_k)
    if K == 4:
        _draft_case(dx, sh, seed=100, zipf=zipf)


def test_moonlight_layer_sigmoid_scaled(dx):
    _verify_case(dx, synth.shape_moonlight(), 8, seed=200, rho=0.9)


# ------------------------------------------------------------------ greedy verification
def _accept_case(dx, M, K, V, H, dtype, seed, rms=False, mode="match"):
    binding, ctx = dx
    W = synth.lm_head(V, H, seed, dtype, "cuda")
    h = synth.hidden_block(M, H, seed + 1, 0.5, "cuda")
    W_np = synth.to_numpy_f32(W).astype(np.float64)
    h_np = h.cpu().numpy().astype(np.float64)
    hn = O.rmsnorm(h_np) if rms else h_np
    target_ref, _, _, lg = O.greedy_accept_fast(hn, W_np, np.zeros(0, np.int32))
    draft = target_ref[:K].copy()
    if mode == "first":
        draft[0] = (draft[0] + 1) % V
    elif mode == "mid":
        draft[K // 2] = (draft[K // 2] + 1) % V
    elif mode == "geometric":
        draft = synth.draft_tokens_from_target(target_ref[:K], V, seed)
    out = binding.spec_accept(ctx, h, W, torch.from_numpy(draft).cuda(), rms_norm=rms)
    torch.cuda.synchronize()
    tgt = out["target"].cpu().numpy()
    srt = np.sort(lg, axis=1)
    gap = srt[:, -1] - srt[:, -2]
    for i in range(M):
        if gap[i] > GAP:
            assert tgt[i] == target_ref[i], (i, tgt[i], target_ref[i], gap[i])
        else:
            assert lg[i, tgt[i]] >= srt[i, -1] - GAP
    # accepted length and next token: the checker's own (n, next) for this draft wherever no row is near-tied ...
    _, n_ref, next_ref, _ = O.greedy_accept(hn, W_np, draft, logits=lg) if V <= 8192 else \
        O.greedy_accept_fast(hn, W_np, draft)
    if (gap > GAP).all():
        assert int(out["n_accept"].item()) == n_ref
        assert int(out["next_token"].item()) == next_ref
    # ... and in every case what the GPU's own target tokens imply (prefix rule restated on the device's tokens)
    n = 0
    while n < K and n < M and draft[n] == tgt[n]:
        n += 1
    assert int(out["n_accept"].item()) == n
    assert int(out["next_token"].item()) == (int(tgt[n]) if n < M else -1)
    return n


def test_accept_tiny_fp32(dx):
    assert _accept_case(dx, 4, 4, 1024, 256, torch.float32, 0, mode="match") == 4
    assert _accept_case(dx, 4, 4, 1024, 256, torch.float32, 0, mode="first") == 0
    assert _accept_case(dx, 4, 4, 1024, 256, torch.float32, 0, mode="mid") == 2
    assert _accept_case(dx, 5, 4, 1024, 256, torch.float32, 1, mode="match", rms=True) == 4


@pytest.mark.parametrize("M,K,V,H", [(4, 4, 1000, 512), (5, 4, 4099, 256), (9, 8, 3001, 1024), (16, 16, 2048, 512),
                                     (1, 1, 17, 256)])
def test_accept_small_bf16(dx, M, K, V, H):
    assert _accept_case(dx, M, K, V, H, torch.bfloat16, 300 + M, mode="match") == K
    _accept_case(dx, M, K, V, H, torch.bfloat16, 310 + M, mode="geometric", rms=True)
    if K > 1:
        assert _accept_case(dx, M, K, V, H, torch.bfloat16, 320 + M, mode="first") == 0


def test_accept_ties_take_lowest_index(dx):
    binding, ctx = dx
    V, H = 512, 256
    W = torch.zeros((V, H), dtype=torch.bfloat16, device="cuda")
    W[37, 0] = 1.0
    W[300, 0] = 1.0           # exact duplicate rows in different warps / CTAs
    W[301, 1] = 2.0
    W[5, 1] = 2.0
    h = torch.zeros((2, H), device="cuda")
    h[0, 0] = 1.5
    h[1, 1] = 0.75
    out = binding.spec_accept(ctx, h, W, torch.tensor([37, 5], dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert out["target"].tolist() == [37, 5] and int(out["n_accept"].item()) == 2
    assert int(out["next_token"].item()) == -1


@pytest.mark.parametrize("M,K,V,H", [(5, 4, 4099, 2048), (8, 8, 3001, 1024), (1, 1, 17, 2048), (3, 2, 2367 * 16 + 5, 1024),
                                     (8, 7, 148 * 16 * 3 + 16, 2048), (16, 16, 148 * 16 * 2 + 1, 2048),
                                     (9, 8, 5003, 2048), (13, 12, 4099, 1024)])
def test_accept_ring_bf16(dx, M, K, V, H):
    """H = 1024 / 2048 take the shared-memory ring variant of the accept kernel (one or two tiles of eight block
    rows): ragged last tile, fewer tiles than CTAs, several rounds of the three-slot ring."""
    assert _accept_case(dx, M, K, V, H, torch.bfloat16, 500 + M, mode="match") == K
    _accept_case(dx, M, K, V, H, torch.bfloat16, 510 + M, mode="geometric", rms=True)
    if K > 1:
        assert _accept_case(dx, M, K, V, H, torch.bfloat16, 520 + M, mode="mid", rms=True) == K // 2


def test_accept_ring_ties_take_lowest_index(dx):
    binding, ctx = dx
    V, H = 148 * 16 * 2 + 40, 2048
    W = torch.zeros((V, H), dtype=torch.bfloat16, device="cuda")
    W[37, 0] = 1.0
    W[4000, 0] = 1.0          # exact duplicate rows in different tiles / CTAs
    W[V - 1, 1900] = 2.0      # in the ragged last tile, in the last warp's columns
    W[5, 1900] = 2.0
    h = torch.zeros((2, H), device="cuda")
    h[0, 0] = 1.5
    h[1, 1900] = 0.75
    out = binding.spec_accept(ctx, h, W, torch.tensor([37, 5], dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert out["target"].tolist() == [37, 5] and int(out["n_accept"].item()) == 2
    assert int(out["next_token"].item()) == -1


def test_accept_full_vocab_bf16(dx):
    _accept_case(dx, 5, 4, 102400, 2048, torch.bfloat16, 400, mode="geometric", rms=True)
    _accept_case(dx, 9, 8, 163840, 2048, torch.bfloat16, 401, mode="geometric", rms=True)


# ------------------------------------------------------------------ draft token + confidence (Sec. 3.4, q_i)
@pytest.mark.parametrize("M,V,H,dtype", [(1, 1000, 512, torch.bfloat16), (4, 4099, 256, torch.bfloat16),
                                         (9, 3001, 1024, torch.bfloat16), (3, 1024, 256, torch.float32),
                                         (1, 102400, 2048, torch.bfloat16), (8, 4099, 2048, torch.bfloat16),
                                         (5, 148 * 16 + 7, 1024, torch.bfloat16), (11, 4099, 2048, torch.bfloat16)])
def test_draft_token_confidence(dx, M, V, H, dtype):
    binding, ctx = dx
    W = synth.lm_head(V, H, 700 + M, dtype, "cuda", std=0.05)
    h = synth.hidden_block(M, H, 701 + M, 0.3, "cuda") * 2.0
    tok, conf = binding.spec_draft_token(ctx, h, W, rms_norm=True)
    torch.cuda.synchronize()
    hn = O.rmsnorm(h.cpu().numpy().astype(np.float64))
    tok_ref, q_ref, lg = O.draft_confidence(hn, synth.to_numpy_f32(W).astype(np.float64))
    srt = np.sort(lg, axis=1)
    for i in range(M):
        if srt[i, -1] - srt[i, -2] > GAP:
            assert int(tok[i]) == int(tok_ref[i])
    # q = 1 / sum exp(l - l_max): fp32 logits and hardware exp, compared with the fp64 checker
    assert np.abs(conf.cpu().numpy() - q_ref).max() <= 1e-4 * max(1.0, q_ref.max()) + 2e-3 * q_ref.max()
    assert np.all(conf.cpu().numpy() > 0) and np.all(conf.cpu().numpy() <= 1.0 + 1e-6)
    # the plain accept kernel is unchanged by the confidence variant
    acc = binding.spec_accept(ctx, h, W, tok, rms_norm=True)
    torch.cuda.synchronize()
    assert torch.equal(acc["target"], tok) and int(acc["n_accept"].item()) == M
