"""The give-up path of the kernels' bounded waits, exercised without faulting or hanging the GPU: a wait for a word
that nothing sets runs out after the context's poll limit, the kernel records DX_DEV_WAIT_EXPIRED and returns, and the
context goes on working."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2607_24434_b200 import synth
from tests.helpers import Y_BF16, gpu_layer, row_rel_err

pytestmark = pytest.mark.gpu

SHAPE = synth.LayerShape(hidden=512, n_experts=16, top_k=3, inter=40, n_shared=2, shared_inter=24, draft_inter=56,
                         score_fn=synth.SCORE_SOFTMAX, norm_topk=1, weight_dtype=synth.DTYPE_BF16)
DX_DEV_WAIT_EXPIRED = 2


def test_wait_for_a_routing_kernel_that_never_runs_expires():
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    layer, ref = gpu_layer(SHAPE, 60, std=0.08)
    L = binding.Layer.from_weights(ctx, layer)
    h = synth.hidden_block(4, SHAPE.hidden, 61, 0.0, "cuda")
    y = torch.empty_like(h)
    # refused while the limit is the default one (the give-up would take seconds)
    with pytest.raises(binding.DxError) as err:
        binding.selftest_wait_expiry(L, h, y)
    assert err.value.status == 1
    ctx.set_wait_limit(2000)
    binding.selftest_wait_expiry(L, h, y)                    # the call returns; the kernel gives up and ends
    torch.cuda.synchronize()
    assert ctx.device_status() == DX_DEV_WAIT_EXPIRED
    assert ctx.device_status() == 0                          # reading clears the word
    # the context is intact: an ordinary verify block on it is correct, with a limit of 2^16 polls in force ...
    ctx.set_wait_limit(1 << 16)
    out = binding.moe_verify_block(L, h)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ids = out["topk_ids"].cpu().numpy()
    y_ref = O.moe_target(h.cpu().numpy().astype(np.float64), ref, forced_ids=ids)[0]
    assert row_rel_err(out["y"].cpu().numpy(), y_ref).max() <= Y_BF16
    # ... and after the default limit is restored
    ctx.set_wait_limit(0)
    out = binding.moe_verify_block(L, h)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert row_rel_err(out["y"].cpu().numpy(), y_ref).max() <= Y_BF16
    L.close(); ctx.close()


def test_accept_ring_gives_up_when_its_waits_are_cut_short():
    """The ring variant of the accept kernel (blocks of at most eight rows, H = 2048) waits on mbarriers for its bulk
    copies.  With a limit of a single poll those waits run out before the first tile has landed: the kernel records
    DX_DEV_WAIT_EXPIRED, stops copying, waits (bounded) for what is still in flight and returns; with the default limit
    restored the same call gives the checker's tokens."""
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0)
    M, K, V, H = 5, 4, 148 * 16 * 4 + 3, 2048
    W = synth.lm_head(V, H, 70, torch.bfloat16, "cuda")
    h = synth.hidden_block(M, H, 71, 0.5, "cuda")
    draft = torch.zeros((K,), dtype=torch.int32, device="cuda")
    ctx.set_wait_limit(1)
    binding.spec_accept(ctx, h, W, draft, rms_norm=True)
    torch.cuda.synchronize()
    assert ctx.device_status() == DX_DEV_WAIT_EXPIRED
    assert ctx.device_status() == 0
    ctx.set_wait_limit(0)
    out = binding.spec_accept(ctx, h, W, draft, rms_norm=True)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    hn = O.rmsnorm(h.cpu().numpy().astype(np.float64))
    t_ref, _, _, lg = O.greedy_accept_fast(hn, synth.to_numpy_f32(W).astype(np.float64), np.zeros(0, np.int32))
    srt = np.sort(lg, axis=1)
    clear = (srt[:, -1] - srt[:, -2]) > 1e-3
    assert np.array_equal(out["target"].cpu().numpy()[clear], t_ref[clear])
    ctx.close()
