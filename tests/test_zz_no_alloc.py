"""rlkv_decode_attention_static_scratch: the decode call for hosts that must not allocate.

Some users of this library cannot call cudaMalloc when a decode step runs: a serving engine that
gave every free byte to its own KV pool at start-up, a plugin under a framework whose allocator owns
the device, a step in which an allocation would stall the whole GPU.  For them the library offers a
variant of rlkv_decode_attention whose split-KV work area is a fixed array inside the library image.
This test calls the variant through the C ABI, twice in a row (the array keeps the previous call's
contents, so the second call proves the call cleans up after the first), and compares each result
with the ordinary entry point on the same cache and query within the bounds the parity tests use.
Both are also compared with the CPU oracle at this shape.  It also checks that the call itself leaves
the device's free memory where it was, and that a launch too large for the array is refused before
anything runs.  A second test runs other shapes (head_dim 64, groups of 4 and of 1, a layer whose
heads are all compressed, so that only the tickets' corner of the array is in use) against the oracle.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from oracle.rlkv_oracle import Oracle

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 1e-2, 1e-3


def rand_bf16(shape, seed, device):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32).to(torch.bfloat16).to(device)


def against_oracle(got, want):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    err = np.abs(got - want)
    rms = np.sqrt((want ** 2).mean(axis=-1, keepdims=True))
    assert np.isfinite(got).all()
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (err.max(), err.mean())
    assert (err <= 2e-2 * rms + 1e-6).all(), float((err / (rms + 1e-30)).max())


def test_static_scratch_variant_matches_the_ordinary_call(cuda_device):
    import paper_2510_08525_b200.binding as rl

    # long rows on few units: most work items begin or end inside a unit, so counters, tickets and
    # partials are all in use
    layers, Hkv, Hq, D, B, S, W, n = 2, 4, 32, 128, 16, 16, 112, 6000
    mask = [1, 0, 1, 1, 1, 1, 1, 1]
    handle = rl.rlkv_cache_create(layers, Hkv, Hq, D, B, n + 8, mask, S, W)
    try:
        oracle = Oracle(layers, Hkv, Hq, D, B, n + 8, mask, S, W, threads=8)
        for layer in range(layers):
            k = rand_bf16((n, B, Hkv, D), 10 + layer, cuda_device)
            v = rand_bf16((n, B, Hkv, D), 20 + layer, cuda_device)
            rl.rlkv_prefill(handle, layer, k, v, n)
            kc, vc = k.cpu(), v.cpu()
            for t in range(n):
                assert oracle.append(layer, kc[t], vc[t]) == 0
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
        for layer, q in enumerate(qs):                      # and both against the oracle at this shape
            ref = oracle.decode(layer, q.cpu())
            against_oracle(outs[layer].cpu().numpy(), ref)
            against_oracle(want[layer].cpu().numpy(), ref)
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


@pytest.mark.parametrize("Hkv,Hq,D,B,S,W,n,mask", [
    (2, 8, 64, 3, 4, 60, 1500, [1, 0, 0, 0]),          # head_dim 64, groups of 4; layer 1 holds compressed heads only
    (4, 4, 128, 2, 16, 48, 900, [0, 0, 0, 0, 1, 1, 0, 1]),   # groups of 1; layer 0 all compressed
])
def test_static_scratch_variant_on_other_shapes_against_the_oracle(cuda_device, Hkv, Hq, D, B, S, W, n, mask):
    import paper_2510_08525_b200.binding as rl
    layers = len(mask) // Hkv
    handle = rl.rlkv_cache_create(layers, Hkv, Hq, D, B, n + 8, mask, S, W)
    try:
        oracle = Oracle(layers, Hkv, Hq, D, B, n + 8, mask, S, W, threads=4)
        for layer in range(layers):
            k, v = rand_bf16((n, B, Hkv, D), 40 + layer, cuda_device), rand_bf16((n, B, Hkv, D), 50 + layer, cuda_device)
            rl.rlkv_prefill(handle, layer, k, v, n)
            kc, vc = k.cpu(), v.cpu()
            for t in range(n):
                assert oracle.append(layer, kc[t], vc[t]) == 0
        for rep in range(2):                                 # the second round reuses what the first left in the array
            for layer in range(layers):
                q = rand_bf16((B, Hq, D), 60 + 7 * rep + layer, cuda_device)
                out = torch.full((B, Hq, D), float("nan"), dtype=torch.float32, device=cuda_device)
                rl.rlkv_decode_attention_static_scratch(handle, layer, q, out)
                ordinary = torch.empty_like(out)
                rl.rlkv_decode_attention(handle, layer, q, ordinary)
                torch.cuda.synchronize()
                against_oracle(out.cpu().numpy(), oracle.decode(layer, q.cpu()))
                assert torch.equal(out, ordinary)
        assert rl.rlkv_kernel_status(handle) == 0
    finally:
        rl.rlkv_cache_destroy(handle)
