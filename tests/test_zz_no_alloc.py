"""rlkv_decode_attention_static_scratch: the decode call for hosts that must not allocate.

Some users of this library cannot call cudaMalloc when a decode step runs: a serving engine that
gave every free byte to its own KV pool at start-up, a plugin under a framework whose allocator owns
the device, a step in which an allocation would stall the whole GPU.  For them the library offers a
variant of rlkv_decode_attention whose split-KV work area is a fixed array inside the library image.
This test calls the variant through the C ABI, twice in a row (the array keeps the previous call's
contents, so the second call proves the call cleans up after the first), and compares each result
with the ordinary entry point on the same cache and query within the bounds the parity tests use.
It also checks that the call itself leaves the device's free memory where it was, and that a launch
too large for the array is refused before anything runs.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 1e-2, 1e-3


def rand_bf16(shape, seed, device):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32).to(torch.bfloat16).to(device)


def test_static_scratch_variant_matches_the_ordinary_call(cuda_device):
    import paper_2510_08525_b200.binding as rl

    # long rows on few units: most work items begin or end inside a unit, so counters, tickets and
    # partials are all in use
    layers, Hkv, Hq, D, B, S, W, n = 2, 4, 32, 128, 16, 16, 112, 6000
    mask = [1, 0, 1, 1, 1, 1, 1, 1]
    handle = rl.rlkv_cache_create(layers, Hkv, Hq, D, B, n + 8, mask, S, W)
    try:
        for layer in range(layers):
            k = rand_bf16((n, B, Hkv, D), 10 + layer, cuda_device)
            v = rand_bf16((n, B, Hkv, D), 20 + layer, cuda_device)
            rl.rlkv_prefill(handle, layer, k, v, n)
        want, got = [], []
        qs = [rand_bf16((B, Hq, D), 30 + i, cuda_device) for i in range(2)]
        for layer, q in enumerate(qs):
            out = torch.empty((B, Hq, D), dtype=torch.float32, device=cuda_device)
            rl.rlkv_decode_attention(handle, layer, q, out)
            want.append(out)
        outs = [torch.full((B, Hq, D), float("nan"), dtype=torch.float32, device=cuda_device) for _ in qs]
        # The first call on a device asks the runtime for the array's address; with lazy module
        # loading that is also the moment the driver gives the array its 4 MiB.  Do it once here,
        # as a host would at start-up, so that the measurement below sees only the calls themselves.
        first = torch.empty((B, Hq, D), dtype=torch.float32, device=cuda_device)
        rl.rlkv_decode_attention_static_scratch(handle, 0, qs[0], first)
        torch.cuda.synchronize()
        assert torch.equal(first, want[0])                  # same kernel, same split: same bits
        free_before, _ = torch.cuda.mem_get_info()          # every buffer of the test exists by now
        for layer, q in enumerate(qs):                      # two calls in a row, nothing in between
            rl.rlkv_decode_attention_static_scratch(handle, layer, q, outs[layer])
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before                    # the calls allocated nothing
        for w_, g_ in zip(want, outs):
            w_, g_ = w_.cpu().numpy().astype(np.float64), g_.cpu().numpy().astype(np.float64)
            assert np.isfinite(g_).all()
            err = np.abs(g_ - w_)
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (err.max(), err.mean())
        assert rl.rlkv_kernel_status(handle) == 0

        # the ordinary call still works on the same cache afterwards
        out = torch.empty((B, Hq, D), dtype=torch.float32, device=cuda_device)
        rl.rlkv_decode_attention(handle, 0, qs[0], out)
        assert torch.equal(out, want[0])

        # argument checks are those of the ordinary call
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_decode_attention_static_scratch(handle, layers, qs[0], out)
        assert e.value.code == rl.RLKV_EINVAL

        # cut into work items of 2 tiles, layer 1 (4 full heads x 16 rows of 94 tiles) may write over
        # 1000 partial records of 4 KiB, more than the array holds: refused, and the output buffer
        # is not touched
        assert rl.rlkv_static_scratch_bytes() == 4 << 20
        rl.rlkv_set_decode_config(handle, 0, 0, 0, 2)
        marker = torch.full((B, Hq, D), 123.0, dtype=torch.float32, device=cuda_device)
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_decode_attention_static_scratch(handle, 1, qs[1], marker)
        assert e.value.code == rl.RLKV_ESCRATCH
        torch.cuda.synchronize()
        assert (marker == 123.0).all()
    finally:
        rl.rlkv_cache_destroy(handle)
