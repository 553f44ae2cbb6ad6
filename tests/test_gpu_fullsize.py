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


def check_unit(cache, w, mask, layer, b, h, n, q_rows, got_rows):
    """One sampled unit against an oracle of its own: the oracle regenerates the unit's n-token history
    from the addressable generator; exported rows bit for bit, the G output rows within the bounds."""
    o = unit_oracle(w, mask, layer, b, h, n)
    for got, ref in zip(cache.export_head(layer, b, h), o.export_head(0, 0, 0)):
        np.testing.assert_array_equal(got[:len(ref)] if got.ndim == 1 else got[:ref.shape[0]], ref)
    want = o.decode(0, q_rows)[0]
    err = np.abs(got_rows - want)
    rms = np.sqrt((want.astype(np.float64) ** 2).mean(axis=-1, keepdims=True))
    assert err.max() <= 1e-2 and err.mean() <= 1e-3, (layer, b, h, n, float(err.max()), float(err.mean()))
    assert (err <= 2e-2 * rms + 1e-6).all(), (layer, b, h, n, float((err / rms).max()))


def test_full_size_decode_loop_sampled_units(cuda_device):
    """The long chain-of-thought loop exactly as the benchmark runs it (32 layers, batch 8, 40 % of the
    heads compressed, sink 16 + window 240): a 4096-token prompt, then every one of the 28672 steps
    through rlkv_step with fresh seeded inputs, to n = 32768; the rings wrap about 136 times.  72
    sampled (step, layer, batch row, KV head) units -- at steps spread over the loop, the last one
    included -- are checked when their step has run: the unit's exported rows bit for bit against an
    oracle that regenerates its history, its output rows within the stated bounds."""
    from paper_2510_08525_b200 import binding as rl
    from paper_2510_08525_b200 import harness
    w = synth.WORKLOADS["cot"]
    mask = synth.workload_mask(w)
    steps = 28672
    n_end = w.context + steps
    free, _ = torch.cuda.mem_get_info()
    need = rl.rlkv_cache_size(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, n_end, mask, w.sink, w.window)
    if free < need + (6 << 30):
        pytest.skip("not enough free device memory for the full-size cache")
    cache = harness.Cache(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, n_end, mask, w.sink, w.window,
                          device=cuda_device)
    harness.fill_cache(cache, w, w.context)
    out = torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=cuda_device)
    rng = np.random.default_rng(99)
    comp, full = np.flatnonzero(mask == 0), np.flatnonzero(mask == 1)
    # sampled steps (token index appended): the first, the ones that fill and first wrap the ring of a
    # prompt that long, a spread over the loop, and the last 8 (steady state at n = 32768)
    sample_steps = sorted(set([w.context, w.context + 1, w.context + w.window - 1, w.context + w.window]
                              + [int(x) for x in rng.integers(w.context, n_end - 8, size=28)]
                              + list(range(n_end - 4, n_end))))
    samples = {}
    for t in sample_steps:
        picks = [rng.choice(full), rng.choice(comp)]
        samples[t] = [(int(f) // w.kv_heads, int(rng.integers(w.batch)), int(f) % w.kv_heads) for f in picks]
    assert sum(len(v) for v in samples.values()) >= 64
    G, checked = w.group, 0
    t = w.context
    while t < n_end:
        t1 = min(n_end, t + 256)
        k, v, q = harness.step_inputs_block(w, t, t1, cuda_device)
        for i in range(t1 - t):
            rl.rlkv_step(cache.handle, k[i], v[i], q[i], out)
            if t + i in samples:
                torch.cuda.synchronize()
                res, qc = out.cpu().numpy(), q[i].cpu()
                for layer, b, h in samples[t + i]:
                    check_unit(cache, w, mask, layer, b, h, t + i + 1, qc[layer, b, h * G:(h + 1) * G].contiguous(),
                               res[layer, b, h * G:(h + 1) * G])
                    checked += 1
        torch.cuda.synchronize()
        t = t1
    assert checked >= 64
    assert cache.status() == 0
    assert all(cache.length(l) == n_end for l in range(w.layers))
    assert np.isfinite(out.cpu().numpy()).all()
    with pytest.raises(rl.RlkvError) as e:                  # the cache is exactly full
        rl.rlkv_step(cache.handle, k[0], v[0], q[0], out)
    assert e.value.code == rl.RLKV_EFULL
    cache.close()
    torch.cuda.empty_cache()


# The corners of the compression x context x batch sweep the benchmark times: a few layers of each
# (the mask is drawn for all 32 layers, the first `layers` are held, as the sweep does).
CORNERS = [
    # context, batch, fraction compressed, layers held
    (65536, 8, 0.0, 3),
    (65536, 8, 0.8, 6),
    (32768, 32, 0.6, 3),
    (8192, 64, 0.2, 3),
    (65536, 1, 0.4, 8),
    (2048, 64, 0.8, 8),
]


@pytest.mark.parametrize("context,batch,frac,layers", CORNERS)
def test_sweep_corners_sampled_units(cuda_device, context, batch, frac, layers):
    from paper_2510_08525_b200 import binding as rl
    from paper_2510_08525_b200 import harness
    w32 = synth.WORKLOADS["llama8b"].with_(context=context, batch=batch, frac_compressed=frac)
    w = w32.with_(layers=layers)
    mask = synth.workload_mask(w32)[:layers * w.kv_heads]
    free, _ = torch.cuda.mem_get_info()
    need = rl.rlkv_cache_size(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, w.context + 8, mask, w.sink, w.window)
    if free < need + (6 << 30):
        pytest.skip("not enough free device memory for this corner")
    cache = harness.Cache(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, w.context + 8, mask, w.sink, w.window,
                          device=cuda_device)
    harness.fill_cache(cache, w, w.context)
    out = torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=cuda_device)
    n = w.context
    for step in range(2):                                   # two steps: n = context + 1 and context + 2
        k, v, q = harness.step_inputs(w, n, cuda_device)
        rl.rlkv_step(cache.handle, k, v, q, out)
        n += 1
    torch.cuda.synchronize()
    assert cache.status() == 0
    res, qc = out.cpu().numpy(), q.cpu()
    assert np.isfinite(res).all()
    total = sum(cache.step_bytes(l) for l in range(w.layers))
    n_full = int(mask.sum())
    assert total == w.batch * (n_full * n + (mask.size - n_full) * (w.sink + w.window)) * 4 * w.head_dim
    rng = np.random.default_rng(context + batch)
    units = {(0, 0, 0), (w.layers - 1, w.batch - 1, w.kv_heads - 1)}
    for cls in (np.flatnonzero(mask == 1), np.flatnonzero(mask == 0)):
        for flat in rng.choice(cls, min(3, len(cls)), replace=False) if len(cls) else []:
            units.add((int(flat) // w.kv_heads, int(rng.integers(w.batch)), int(flat) % w.kv_heads))
    G = w.group
    for layer, b, h in sorted(units):
        check_unit(cache, w, mask, layer, b, h, n, qc[layer, b, h * G:(h + 1) * G].contiguous(),
                   res[layer, b, h * G:(h + 1) * G])
    cache.close()
    torch.cuda.empty_cache()


def paged_unit_oracle(w, mask, seq, layer, h, n, scales):
    """Oracle of one (sequence, layer, KV head) unit of the paged batch: n tokens regenerated from the
    sequence's own generator; `scales` (k, v) puts it in 8-bit storage."""
    from paper_2510_08525_b200 import harness
    full = int(mask[layer * w.kv_heads + h])
    o = Oracle(1, 1, w.group, w.head_dim, 1, n, [full], w.sink, w.window)
    if scales is not None:
        o.set_fp8([scales[0]], [scales[1]])
    seed = harness.paged_seq_seed(w, seq)
    K = synth.unit_rows(seed, synth.STREAM_K, layer, 0, n, 1, w.kv_heads, w.head_dim, 0, h)
    V = synth.unit_rows(seed, synth.STREAM_V, layer, 0, n, 1, w.kv_heads, w.head_dim, 0, h)
    kb = K.view(torch.int16).numpy().view(np.uint16)
    vb = V.view(torch.int16).numpy().view(np.uint16)
    for t in range(n):
        o.append(0, kb[t], vb[t])
    return o


@pytest.mark.parametrize("kind,fp8", [("uniform", False), ("ragged", False), ("uniform", True)])
def test_paged_full_size_sampled_units(cuda_device, kind, fp8):
    """The paged batches bench.py times (the 32 layers of the llama8b mask, 16 sequences at 8193 tokens
    or spread from 2048 to 14338, 16-bit and 8-bit), through the two launch forms it times: one whole
    step (rlkv_paged_step: one attention launch over all layers) and one launch per layer
    (rlkv_paged_decode_attention).  Sampled (layer, sequence, KV head) units against an oracle of their
    own: stored rows (or codes) bit for bit, the G output rows within the bounds."""
    from paper_2510_08525_b200 import binding as rl
    from paper_2510_08525_b200 import harness
    w = synth.WORKLOADS["llama8b"]
    mask = synth.workload_mask(w)
    n0 = w.context
    lens = [n0] * w.batch if kind == "uniform" else harness.paged_spread_lengths(n0 + 1, w.batch)
    pages = sum((x + 1 + 63) // 64 for x in lens) + 2 + 2 * len(lens)
    scale = np.float32(1.0 / 64)
    scales = np.full(w.layers * w.kv_heads, scale, np.float32) if fp8 else None
    size = (rl.rlkv_paged_size_fp8 if fp8 else rl.rlkv_paged_size)(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, pages,
                                                                   max(lens) + 128, mask, w.sink, w.window)
    free, _ = torch.cuda.mem_get_info()
    if free < size + (4 << 30):
        pytest.skip("not enough free device memory for the full-size paged cache")
    pc = harness.PagedCache(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, pages, max(lens) + 128, mask,
                            w.sink, w.window, device=cuda_device, k_scale=scales, v_scale=scales)
    try:
        slots = [pc.open_seq() for _ in lens]
        harness.fill_paged(pc, w, slots, lens)
        k, v, q = harness.paged_step_inputs(pc, w, lens)
        out = torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=cuda_device)
        rl.rlkv_paged_step(pc.handle, slots, k, v, q, out)
        torch.cuda.synchronize()
        assert pc.status() == 0
        step_out = out.cpu().numpy()
        assert np.isfinite(step_out).all()
        # one launch per layer on the sampled layers: the state has not changed, so the same attention
        rng = np.random.default_rng(77)
        units = {(0, 0, 0), (w.layers - 1, w.batch - 1, w.kv_heads - 1)}
        full, comp = np.flatnonzero(mask == 1), np.flatnonzero(mask == 0)
        for flat in list(rng.choice(full, 4, replace=False)) + list(rng.choice(comp, 3, replace=False)):
            units.add((int(flat) // w.kv_heads, int(rng.integers(w.batch)), int(flat) % w.kv_heads))
        units.add((int(full[0]) // w.kv_heads, int(np.argmax(lens)), int(full[0]) % w.kv_heads))   # the longest sequence
        units.add((int(full[-1]) // w.kv_heads, int(np.argmin(lens)), int(full[-1]) % w.kv_heads))  # the shortest
        layer_out = {}
        for layer in sorted({u[0] for u in units}):
            o = torch.empty((w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=cuda_device)
            rl.rlkv_paged_decode_attention(pc.handle, layer, slots, q[layer], o)
            layer_out[layer] = o.cpu().numpy()
        assert pc.status() == 0
        qc = q.cpu()
        G = w.group
        unit_scales = (scale, scale) if fp8 else None
        for layer, i, h in sorted(units):
            n = lens[i] + 1
            assert pc.length(layer, slots[i]) == n
            o = paged_unit_oracle(w, mask, i, layer, h, n, unit_scales)
            gk, gv, gt = pc.export_head(layer, slots[i], h)
            ok, ov, ot = o.export_head(0, 0, 0)
            rows = len(gt)
            np.testing.assert_array_equal(gt, ot[:rows])
            np.testing.assert_array_equal(gk, ok[:rows])
            np.testing.assert_array_equal(gv, ov[:rows])
            want = o.decode(0, qc[layer, i, h * G:(h + 1) * G].contiguous())[0]
            rms = np.sqrt((want.astype(np.float64) ** 2).mean(axis=-1, keepdims=True))
            for got in (step_out[layer, i, h * G:(h + 1) * G], layer_out[layer][i, h * G:(h + 1) * G]):
                err = np.abs(got - want)
                assert err.max() <= 1e-2 and err.mean() <= 1e-3, (layer, i, h, float(err.max()), float(err.mean()))
                assert (err <= 2e-2 * rms + 1e-6).all(), (layer, i, h, float((err / rms).max()))
            o.close()
    finally:
        pc.close()
        torch.cuda.empty_cache()


def test_per_layer_chain_full_size_sampled_units(cuda_device):
    """The per-layer calls of a model forward at the headline size, issued as bench.py's per_layer_calls
    leg issues them: before every layer a stand-in kernel (a 96 MiB device copy) that writes the
    layer's k, v, q at its very end, then the attention call launched to overlap with it.  One step
    with rlkv_layer_step_overlapped (one launch per layer), one with rlkv_append_overlapped +
    rlkv_decode_attention_overlapped; after each, sampled units against an oracle of their own."""
    from paper_2510_08525_b200 import binding as rl
    from paper_2510_08525_b200 import harness
    w = synth.WORKLOADS["llama8b"]
    mask = synth.workload_mask(w)
    free, _ = torch.cuda.mem_get_info()
    need = rl.rlkv_cache_size(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, w.context + 64, mask, w.sink, w.window)
    if free < need + (4 << 30):
        pytest.skip("not enough free device memory for the full-size cache")
    cache = harness.make_cache(w, device=cuda_device)
    try:
        harness.fill_cache(cache, w, w.context)
        kv_elems, q_elems = w.batch * w.kv_heads * w.head_dim, w.batch * w.q_heads * w.head_dim
        buf = torch.zeros(2 * kv_elems + q_elems, dtype=torch.bfloat16, device=cuda_device)   # k | v | q of the current layer
        kb, vb, qb = buf[:kv_elems], buf[kv_elems:2 * kv_elems], buf[2 * kv_elems:]
        work_src = torch.ones(96 << 20, dtype=torch.uint8, device=cuda_device)
        work_dst = torch.empty_like(work_src)
        out = torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=cuda_device)
        rng = np.random.default_rng(99)
        full, comp = np.flatnonzero(mask == 1), np.flatnonzero(mask == 0)
        for step, one_launch in enumerate((True, False)):
            t = w.context + step
            k, v, q = harness.step_inputs(w, t, cuda_device)
            src = [torch.cat([k[l].reshape(-1), v[l].reshape(-1), q[l].reshape(-1)]) for l in range(w.layers)]
            torch.cuda.synchronize()
            for l in range(w.layers):
                rl.rlkv_debug_standin(work_dst, work_src, work_src.numel(), out[l - 1] if l else None, buf, src[l],
                                      buf.numel() * 2, 1)
                if one_launch:
                    rl.rlkv_layer_step_overlapped(cache.handle, l, kb, vb, qb, out[l])
                else:
                    rl.rlkv_append_overlapped(cache.handle, l, kb, vb)
                    rl.rlkv_decode_attention_overlapped(cache.handle, l, qb, out[l])
            torch.cuda.synchronize()
            assert cache.status() == 0
            got = out.cpu().numpy()
            assert np.isfinite(got).all()
            qc = q.cpu()
            units = {(0, 0, 0), (w.layers - 1, w.batch - 1, w.kv_heads - 1)}
            for flat in list(rng.choice(full, 4, replace=False)) + list(rng.choice(comp, 3, replace=False)):
                units.add((int(flat) // w.kv_heads, int(rng.integers(w.batch)), int(flat) % w.kv_heads))
            G = w.group
            for layer, b, h in sorted(units):
                check_unit(cache, w, mask, layer, b, h, t + 1, qc[layer, b, h * G:(h + 1) * G].contiguous(),
                           got[layer, b, h * G:(h + 1) * G])
    finally:
        cache.close()
        torch.cuda.empty_cache()
