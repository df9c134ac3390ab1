"""The allocation-free greedy-verification entry point (``spec_accept_noalloc``) against the regular one.

Some users of the library cannot allocate device memory at the point where they verify a block -- they run
under a memory pool that was sized once at start-up, or are handed buffers and a stream but no allocator -- so
they cannot create a context (``dx_create`` allocates).  The extra entry point keeps its scratch in a static device array
instead.  This test calls it through the C ABI twice in a row (the array is shared and keeps the previous
call's contents, so the second call is the one that would expose stale state) and checks every output against
``spec_accept`` on the same inputs: token ids, accepted length and next token are integers, so they must be
identical.  The outputs are also compared with the CPU checker (rows whose two best logits are closer than 1e-3 may
resolve either way).  That the call allocates nothing is checked twice: torch's allocator count must not move (the
wrapper), and the driver's free-memory figure must not move across the second call (the library itself; the first
call loads the kernels' module, which the driver accounts for).  The file is named to be collected last; it passes
alone in a fresh process and after the others."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2607_24434_b200 import synth

pytestmark = pytest.mark.gpu


def _outputs(M, device):
    return {"target": torch.full((M,), -7, dtype=torch.int32, device=device),
            "n_accept": torch.full((1,), -7, dtype=torch.int32, device=device),
            "next_token": torch.full((1,), -7, dtype=torch.int32, device=device)}


@pytest.mark.parametrize("M,K,V,H,dtype", [(5, 4, 4099, 512, torch.bfloat16), (16, 16, 3001, 256, torch.bfloat16),
                                           (4, 4, 1024, 256, torch.float32)])
def test_noalloc_matches_regular_entry_point_twice(M, K, V, H, dtype):
    from paper_2607_24434_b200 import binding
    ctx = binding.Context(0, act_split=True)
    W = synth.lm_head(V, H, 900 + M, dtype, "cuda")
    results = []
    for call in range(2):                       # two calls in a row on different inputs
        h = synth.hidden_block(M, H, 910 + 10 * call + M, 0.5, "cuda")
        ref = binding.spec_accept(ctx, h, W, torch.zeros((K,), dtype=torch.int32, device="cuda"), rms_norm=True)
        torch.cuda.synchronize()
        draft = ref["target"][:K].clone()
        if call == 1 and K > 1:
            draft[K // 2] = (draft[K // 2] + 1) % V          # mismatch in the middle on the second call
        ref = binding.spec_accept(ctx, h, W, draft, rms_norm=True)
        outs = _outputs(M, "cuda")
        torch.cuda.synchronize()
        n_allocs = torch.cuda.memory_stats()["allocation.all.allocated"]
        free_before = torch.cuda.mem_get_info()[0]
        got = binding.spec_accept_noalloc(h, W, draft, outs, rms_norm=True)
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == n_allocs   # the wrapper allocates nothing
        torch.cuda.synchronize()
        if call == 1:                                        # ... and neither does the library (driver-level figure)
            assert torch.cuda.mem_get_info()[0] == free_before
        for key in ("target", "n_accept", "next_token"):
            assert torch.equal(got[key], ref[key]), (call, key, got[key], ref[key])
        # against the CPU checker, outside the tie gap
        h_np = O.rmsnorm(h.cpu().numpy().astype(np.float64))
        t_ref, n_ref, next_ref, lg = O.greedy_accept_fast(h_np, synth.to_numpy_f32(W).astype(np.float64),
                                                          draft.cpu().numpy())
        srt = np.sort(lg, axis=1)
        clear = (srt[:, -1] - srt[:, -2]) > 1e-3
        assert np.array_equal(got["target"].cpu().numpy()[clear], t_ref[clear])
        if clear.all():
            assert int(got["n_accept"].item()) == n_ref and int(got["next_token"].item()) == next_ref
        results.append(int(got["n_accept"].item()))
    assert results[0] == K and (K == 1 or results[1] == K // 2)
    ctx.close()


def test_noalloc_rejects_sizes_beyond_its_scratch():
    from paper_2607_24434_b200 import binding
    H, V = 256, 64
    W = synth.lm_head(V, H, 950, torch.bfloat16, "cuda")
    h = torch.zeros((17, H), device="cuda")
    with pytest.raises(binding.DxError) as err:
        binding.spec_accept_noalloc(h, W, torch.zeros((4,), dtype=torch.int32, device="cuda"), _outputs(17, "cuda"))
    assert err.value.status == 8                             # DX_ERR_UNSUPPORTED, a clear refusal
