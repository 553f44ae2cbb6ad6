"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the cache is
filled from the seeded generator, one whole decode step runs through rlkv_step, and sampled
(layer, batch row, KV head) units are checked one by one -- the oracle regenerates that unit's
K/V history from the addressable generator, the unit's exported rows must match bit for bit and
its G output rows within the stated bounds.
"""
import numpy as np
import pytest
import torch

import synth
from oracle.rlkv_oracle import Oracle

pytestmark = pytest.mark.gpu


def unit_oracle(w, mask, layer, b, h, n):
    full = int(mask[layer * w.kv_heads + h])
    o = Oracle(1, 1, w.group, w.head_dim, 1, n, [full], w.sink, w.window)
    K = synth.unit_rows(w.seed, synth.STREAM_K, layer, 0, n, w.batch, w.kv_heads, w.head_dim, b, h)
    V = synth.unit_rows(w.seed, synth.STREAM_V, layer, 0, n, w.batch, w.kv_heads, w.head_dim, b, h)
    kb = K.view(torch.int16).numpy().view(np.uint16)
    vb = V.view(torch.int16).numpy().view(np.uint16)
    for t in range(n):
        o.append(0, kb[t], vb[t])
    return o


@pytest.mark.parametrize("name", ["llama8b", "qwen7b"])
def test_full_size_sampled_units(cuda_device, name):
    from paper_2510_08525_b200 import binding as rl
    from paper_2510_08525_b200 import harness
    w = synth.WORKLOADS[name]
    mask = synth.workload_mask(w)
    free, _ = torch.cuda.mem_get_info()
    need = rl.rlkv_cache_size(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, w.context + 64, mask,
                              w.sink, w.window)
    if free < need + (4 << 30):
        pytest.skip("not enough free device memory for the full-size cache")
    cache = harness.make_cache(w, device=cuda_device)
    harness.fill_cache(cache, w, w.context)
    n = w.context + 1
    k, v, q = harness.step_inputs(w, w.context, cuda_device)
    out = torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=cuda_device)
    rl.rlkv_step(cache.handle, k, v, q, out)
    torch.cuda.synchronize()
    assert cache.status() == 0
    out = out.cpu().numpy()
    q = q.cpu()
    assert np.isfinite(out).all()

    # integer cost model: bytes the library says it reads == (n_full*n + n_comp*cap) rows
    n_full = int(mask.sum())
    total = sum(cache.step_bytes(l) for l in range(w.layers))
    assert total == w.batch * (n_full * n + (mask.size - n_full) * (w.sink + w.window)) * 4 * w.head_dim

    rng = np.random.default_rng(1234)
    units = set()
    comp = np.flatnonzero(mask == 0)
    full = np.flatnonzero(mask == 1)
    for flat in list(rng.choice(full, 5, replace=False)) + list(rng.choice(comp, 5, replace=False)):
        units.add((int(flat) // w.kv_heads, int(rng.integers(w.batch)), int(flat) % w.kv_heads))
    units.add((0, 0, 0))
    units.add((w.layers - 1, w.batch - 1, w.kv_heads - 1))
    G = w.group
    for layer, b, h in sorted(units):
        o = unit_oracle(w, mask, layer, b, h, n)
        for got, ref in zip(cache.export_head(layer, b, h), o.export_head(0, 0, 0)):
            np.testing.assert_array_equal(got[:len(ref)] if got.ndim == 1 else got[:ref.shape[0]], ref)
        want = o.decode(0, q[layer, b, h * G:(h + 1) * G].contiguous())[0]
        got = out[layer, b, h * G:(h + 1) * G]
        err = np.abs(got - want)
        rms = np.sqrt((want.astype(np.float64) ** 2).mean(axis=-1, keepdims=True))
        assert err.max() <= 1e-2 and err.mean() <= 1e-3
        assert (err <= 2e-2 * rms + 1e-6).all(), (layer, b, h, float((err / rms).max()))
    cache.close()
    torch.cuda.empty_cache()


def test_full_size_decode_loop_sampled_units(cuda_device):
    """The long chain-of-thought loop at its full shape (32 layers, batch 8, 40 % of the heads
    compressed, sink 16 + window 240, room for 32768 tokens): a 4096-token prompt, then 300 whole
    steps through rlkv_step, so that every ring has wrapped.  Sampled units are checked after the last
    step: exported rows bit for bit, output rows within the stated bounds."""
    from paper_2510_08525_b200 import binding as rl
    from paper_2510_08525_b200 import harness
    w = synth.WORKLOADS["cot"]
    mask = synth.workload_mask(w)
    max_len, steps = 32768, 300
    free, _ = torch.cuda.mem_get_info()
    need = rl.rlkv_cache_size(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, max_len, mask, w.sink, w.window)
    if free < need + (4 << 30):
        pytest.skip("not enough free device memory for the full-size cache")
    cache = harness.Cache(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, max_len, mask, w.sink, w.window,
                          device=cuda_device)
    harness.fill_cache(cache, w, w.context)
    out = torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=cuda_device)
    for t in range(w.context, w.context + steps):
        k, v, q = harness.step_inputs(w, t, cuda_device)
        rl.rlkv_step(cache.handle, k, v, q, out)
    torch.cuda.synchronize()
    assert cache.status() == 0
    n = w.context + steps
    assert all(cache.length(l) == n for l in range(w.layers))
    res, q = out.cpu().numpy(), q.cpu()
    assert np.isfinite(res).all()
    rng = np.random.default_rng(99)
    comp, full = np.flatnonzero(mask == 0), np.flatnonzero(mask == 1)
    picks = list(rng.choice(full, 4, replace=False)) + list(rng.choice(comp, 4, replace=False))
    G = w.group
    for flat in picks:
        layer, h, b = int(flat) // w.kv_heads, int(flat) % w.kv_heads, int(rng.integers(w.batch))
        o = unit_oracle(w, mask, layer, b, h, n)
        for got, ref in zip(cache.export_head(layer, b, h), o.export_head(0, 0, 0)):
            np.testing.assert_array_equal(got[:len(ref)] if got.ndim == 1 else got[:ref.shape[0]], ref)
        want = o.decode(0, q[layer, b, h * G:(h + 1) * G].contiguous())[0]
        err = np.abs(res[layer, b, h * G:(h + 1) * G] - want)
        rms = np.sqrt((want.astype(np.float64) ** 2).mean(axis=-1, keepdims=True))
        assert err.max() <= 1e-2 and err.mean() <= 1e-3
        assert (err <= 2e-2 * rms + 1e-6).all(), (layer, b, h, float((err / rms).max()))
    cache.close()
    torch.cuda.empty_cache()
