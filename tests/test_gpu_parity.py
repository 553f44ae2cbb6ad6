"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.  Cache state is compared bit for bit; attention outputs within the stated bounds
(max abs error <= 1e-2, mean abs error <= 1e-3, plus max abs error <= 2e-2 * rms(out) per query
head so the check keeps its teeth at long contexts where |out| ~ 0.02).
"""
import numpy as np
import pytest
import torch

import synth
from oracle.rlkv_oracle import Oracle

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS, REL_RMS = 1e-2, 1e-3, 2e-2


@pytest.fixture(scope="module")
def rl(cuda_device):
    import paper_2510_08525_b200.binding as binding
    return binding


@pytest.fixture(scope="module")
def hz(cuda_device):
    import paper_2510_08525_b200.harness as harness
    return harness


def rand_bf16(shape, seed, device="cpu"):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32).to(torch.bfloat16).to(device)


def check_out(got, want):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    assert np.isfinite(got).all()
    err = np.abs(got - want)
    assert err.max() <= MAX_ABS, err.max()
    assert err.mean() <= MEAN_ABS, err.mean()
    rms = np.sqrt((want ** 2).mean(axis=-1, keepdims=True))
    assert (err <= REL_RMS * rms + 1e-6).all(), float((err / (rms + 1e-30)).max())


def check_state(cache, oracle, layers=None, rows=None):
    for l in (range(cache.layers) if layers is None else layers):
        assert cache.length(l) == oracle.length(l)
        for b in range(cache.batch):
            for h in range(cache.kv_heads):
                gk, gv, gt = cache.export_head(l, b, h)
                ok, ov, ot = oracle.export_head(l, b, h)
                np.testing.assert_array_equal(gt, ot)
                np.testing.assert_array_equal(gk, ok)
                np.testing.assert_array_equal(gv, ov)


def build_pair(hz, layers, Hkv, Hq, D, B, max_len, mask, S, W, dev):
    cache = hz.Cache(layers, Hkv, Hq, D, B, max_len, mask, S, W, device=dev)
    oracle = Oracle(layers, Hkv, Hq, D, B, max_len, mask, S, W, threads=8)
    return cache, oracle


def feed(cache, oracle, layer, K, V, bulk):
    """K, V: bf16 [n][B][Hkv][D] on the CPU."""
    dev = cache.device
    if bulk:
        cache.prefill(layer, K.to(dev), V.to(dev))
    else:
        for t in range(K.shape[0]):
            cache.append(layer, K[t].to(dev), V[t].to(dev))
    for t in range(K.shape[0]):
        assert oracle.append(layer, K[t], V[t]) == 0


# ------------------------------------------------------------------------------------------ tiny
@pytest.mark.parametrize("bulk", [False, True])
def test_tiny_config(rl, hz, cuda_device, bulk):
    """1 layer, batch 1, 8/2 heads, D 64, KV head 0 full, head 1 compressed 4+60; 512 cached tokens,
    one append, one decode (n = 513); also checked at n = 512."""
    w = synth.WORKLOADS["tiny"]
    mask = hz.workload_mask(w)
    cache, oracle = build_pair(hz, 1, w.kv_heads, w.q_heads, w.head_dim, 1, 520, mask, w.sink, w.window, cuda_device)
    K = synth.rows(w.seed, synth.STREAM_K, 0, 0, 513, 1, w.kv_heads, w.head_dim)
    V = synth.rows(w.seed, synth.STREAM_V, 0, 0, 513, 1, w.kv_heads, w.head_dim)
    feed(cache, oracle, 0, K[:512], V[:512], bulk)
    q512 = synth.rows(w.seed, synth.STREAM_Q, 0, 511, 512, 1, w.q_heads, w.head_dim)[0]
    check_out(cache.decode(0, q512.to(cuda_device)).cpu().numpy(), oracle.decode(0, q512))
    feed(cache, oracle, 0, K[512:], V[512:], False)
    q = synth.rows(w.seed, synth.STREAM_Q, 0, 512, 513, 1, w.q_heads, w.head_dim)[0]
    out = cache.decode(0, q.to(cuda_device))
    check_out(out.cpu().numpy(), oracle.decode(0, q))
    check_state(cache, oracle)
    assert cache.step_bytes(0) == (513 + 64) * 2 * 64 * 2
    assert cache.status() == 0
    # determinism: the same call again gives the same bits
    out2 = cache.decode(0, q.to(cuda_device))
    assert torch.equal(out, out2)


# ------------------------------------------------------------------------------------------ shapes
SHAPES = [
    # layers, Hkv, Hq, D, B, S, W, n, mask pattern
    (1, 2, 8, 64, 1, 4, 60, 1, "10"),
    (1, 2, 8, 64, 2, 4, 60, 63, "10"),
    (1, 2, 8, 64, 2, 4, 60, 64, "01"),
    (1, 2, 8, 64, 2, 4, 60, 65, "10"),
    (2, 4, 28, 128, 3, 16, 112, 300, "1001" "0110"),
    (2, 4, 28, 128, 2, 16, 112, 129, "0000" "1111"),
    (1, 8, 32, 128, 2, 16, 112, 1000, "11011011"),
    (1, 1, 8, 128, 1, 0, 5, 777, "0"),
    (1, 1, 1, 64, 5, 3, 200, 450, "1"),
    (1, 3, 15, 128, 2, 1, 1, 200, "010"),
    (1, 2, 6, 64, 1, 7, 57, 2000, "10"),
    (1, 2, 8, 128, 1, 16, 240, 5000, "11"),       # long single rows: every CTA writes partials
    (3, 2, 4, 128, 4, 130, 62, 193, "100111"),    # sink larger than the window; n == sink + window + 1
]


@pytest.mark.parametrize("bulk", [True, False])
@pytest.mark.parametrize("shape", SHAPES, ids=[f"s{i}" for i in range(len(SHAPES))])
def test_shapes_against_oracle(rl, hz, cuda_device, shape, bulk):
    layers, Hkv, Hq, D, B, S, W, n, pattern = shape
    if not bulk and n > 1000:
        pytest.skip("single appends covered at smaller n")
    mask = [int(c) for c in pattern]
    cache, oracle = build_pair(hz, layers, Hkv, Hq, D, B, n + 3, mask, S, W, cuda_device)
    for l in range(layers):
        K, V = rand_bf16((n, B, Hkv, D), 100 + l), rand_bf16((n, B, Hkv, D), 200 + l)
        feed(cache, oracle, l, K, V, bulk)
    for l in range(layers):
        q = rand_bf16((B, Hq, D), 300 + l)
        out = cache.decode(l, q.to(cuda_device))
        check_out(out.cpu().numpy(), oracle.decode(l, q))
    check_state(cache, oracle)
    assert cache.status() == 0


def test_ring_wraps_many_times_and_mixed_append_sizes(rl, hz, cuda_device):
    """Appends in chunks of 1, 7, 300 ... so the ring wraps inside and across bulk appends; state is
    compared bit for bit and outputs at several lengths."""
    layers, Hkv, Hq, D, B, S, W = 1, 2, 4, 64, 2, 16, 48
    total = 1500
    cache, oracle = build_pair(hz, layers, Hkv, Hq, D, B, total, [0, 1], S, W, cuda_device)
    K, V = rand_bf16((total, B, Hkv, D), 1), rand_bf16((total, B, Hkv, D), 2)
    t, sizes, i = 0, [1, 7, 300, 2, 64, 1, 1, 129, 48, 47, 500], 0
    while t < total:
        n = min(sizes[i % len(sizes)], total - t)
        feed(cache, oracle, 0, K[t:t + n], V[t:t + n], bulk=n > 1)
        t += n
        i += 1
        q = rand_bf16((B, Hq, D), 1000 + t)
        check_out(cache.decode(0, q.to(cuda_device)).cpu().numpy(), oracle.decode(0, q))
        check_state(cache, oracle)
    with pytest.raises(rl.RlkvError) as e:
        cache.append(0, K[0].to(cuda_device), V[0].to(cuda_device))
    assert e.value.code == rl.RLKV_EFULL
    check_state(cache, oracle)          # the refused append changed nothing


# ------------------------------------------------------------------------------------------ needles
def test_planted_needles_at_tile_and_split_boundaries(rl, hz, cuda_device):
    """One token whose key is aligned with q carries a marker value: the output must be the marker
    iff the head retains the token.  Positions sweep tile edges and the compressed head's edges."""
    D, n, S, W, B = 128, 2200, 16, 112, 1
    base_K, base_V = rand_bf16((n, B, 2, D), 5), rand_bf16((n, B, 2, D), 6)
    q = rand_bf16((B, 2, D), 7)
    marker = torch.full((D,), 7.0, dtype=torch.bfloat16)
    spots = [0, 1, S - 1, S, 63, 64, 65, 127, 128, 1023, 1024, n - W - 1, n - W, n - 2, n - 1]
    # the scan of this shape is cut into work items of 4 tiles (256 tokens): add their boundaries
    spots += [t for c in range(1, 9) for t in (c * 256 - 1, c * 256)]
    for t_star in sorted(set(spots)):
        K, V = base_K.clone(), base_V.clone()
        for h in range(2):
            qq = q[0, h].to(torch.float32)
            K[t_star, 0, h] = (qq / qq.norm() * 100.0).to(torch.bfloat16)
            V[t_star, 0, h] = marker
        cache, oracle = build_pair(hz, 1, 2, 2, D, B, n, [1, 0], S, W, cuda_device)
        feed(cache, oracle, 0, K, V, bulk=True)
        out = cache.decode(0, q.to(cuda_device)).cpu().numpy()
        want = oracle.decode(0, q)
        check_out(out, want)
        assert np.abs(out[0, 0] - 7.0).max() < 1e-2
        visible = t_star < S or t_star >= n - W
        assert (np.abs(out[0, 1] - 7.0).max() < 1e-2) == visible
        cache.close()


# ------------------------------------------------------------------------------------------ budget
def test_compressed_heads_stay_inside_their_budget(rl, hz, cuda_device):
    """Caller-provided buffer framed by sentinel guard bands; after many appends and decodes the
    guards are intact, bytes read per step stop growing with n for compressed heads, and the padding
    rows of every head are still zero."""
    layers, Hkv, Hq, D, B, S, W, max_len = 2, 2, 4, 64, 2, 4, 28, 400
    mask = [0, 1, 0, 0]
    need = rl.rlkv_cache_size(layers, Hkv, Hq, D, B, max_len, mask, S, W)
    guard = 4096
    buf = torch.full((need + 2 * guard + 1024,), 0xA5, dtype=torch.uint8, device=cuda_device)
    off = (-buf.data_ptr() - guard) % 1024 + guard
    inner = buf[off:off + need]
    assert inner.data_ptr() % 1024 == 0
    cache = hz.Cache(layers, Hkv, Hq, D, B, max_len, mask, S, W, device=cuda_device, device_buf=inner)
    oracle = Oracle(layers, Hkv, Hq, D, B, max_len, mask, S, W)
    K, V = rand_bf16((max_len, B, Hkv, D), 8), rand_bf16((max_len, B, Hkv, D), 9)
    seen = []
    for l in range(layers):
        for t0 in range(0, max_len, 50):
            feed(cache, oracle, l, K[t0:t0 + 50], V[t0:t0 + 50], bulk=(t0 % 100 == 0))
            q = rand_bf16((B, Hq, D), t0)
            check_out(cache.decode(l, q.to(cuda_device)).cpu().numpy(), oracle.decode(l, q))
            if l == 1:
                seen.append(cache.step_bytes(1))
    check_state(cache, oracle)
    torch.cuda.synchronize()
    assert (buf[:off] == 0xA5).all() and (buf[off + need:] == 0xA5).all()
    # layer 1 has only compressed heads: bytes per step are constant once n >= S + W
    assert seen[0] == B * 2 * 32 * 2 * D * 2 and len(set(seen)) == 1
    # cost model in integers: bytes == B * 2*D*2 * (n_full*n + n_comp*min(n, S+W))
    assert cache.step_bytes(0) == B * 2 * D * 2 * (1 * max_len + 1 * (S + W))
    with pytest.raises(rl.RlkvError) as e:
        cache.append(1, K[0].to(cuda_device), V[0].to(cuda_device))
    assert e.value.code == rl.RLKV_EFULL      # uniform rule, even for an all-compressed layer
    # The pool starts the buffer: per layer the full heads' region [batch][full head][K|V][rows_full][D],
    # then the compressed heads' [batch][compressed head][K|V][rows_comp][D], rows rounded up to the
    # 64-row tile.  Every row past a head's budget (rows 400.. of a full head, rows 32.. of a ring) must
    # still hold the zeros it was created with: a write that strays out of a ring lands there first.
    rows_full, rows_comp, cap = 448, 64, S + W
    pool = inner.view(torch.bfloat16)
    row = 0
    heads_seen = 0
    for l in range(layers):
        n_full = sum(mask[l * Hkv:(l + 1) * Hkv])
        for rows, count, used in ((rows_full, B * n_full, max_len), (rows_comp, B * (Hkv - n_full), cap)):
            for _ in range(2 * count):                       # K block and V block of every head
                block = pool[row * D:(row + rows) * D].view(rows, D)
                assert block[:used].any()                    # the head's own rows were written ...
                assert not block[used:].any()                # ... and nothing beyond them
                row += rows
                heads_seen += 1
    assert heads_seen == 2 * B * layers * Hkv


# ------------------------------------------------------------------------------------------ errors
def test_error_paths_leave_state_untouched(rl, hz, cuda_device):
    D, B, Hkv, Hq = 64, 1, 2, 4
    with pytest.raises(rl.RlkvError) as e:
        rl.rlkv_cache_create(1, 2, 5, D, B, 10, [1, 0], 1, 1)          # q_heads % kv_heads
    assert e.value.code == rl.RLKV_EINVAL
    for bad in (dict(head_dim=96), dict(window=0), dict(sink=-1), dict(q_heads=18)):
        args = dict(layers=1, kv_heads=2, q_heads=4, head_dim=D, batch=B, max_len=10, head_is_full=[1, 0],
                    sink=1, window=1)
        args.update(bad)
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_cache_create(**args)
        assert e.value.code == rl.RLKV_EINVAL
    cache = hz.Cache(1, Hkv, Hq, D, B, 10, [1, 0], 1, 2, device=cuda_device)
    q = rand_bf16((B, Hq, D), 1, cuda_device)
    out = torch.zeros((B, Hq, D), dtype=torch.float32, device=cuda_device)
    with pytest.raises(rl.RlkvError) as e:
        cache.decode(0, q, out)
    assert e.value.code == rl.RLKV_EEMPTY
    k = rand_bf16((B, Hkv, D), 2, cuda_device)
    for call in (lambda: rl.rlkv_append(cache.handle, 1, k, k), lambda: rl.rlkv_append(cache.handle, -1, k, k),
                 lambda: rl.rlkv_append(cache.handle, 0, 0, k), lambda: rl.rlkv_append(cache.handle, 0, k.data_ptr() + 2, k),
                 lambda: rl.rlkv_decode_attention(cache.handle, 0, q, 0),
                 lambda: rl.rlkv_prefill(cache.handle, 0, k, k, 0)):
        with pytest.raises(rl.RlkvError) as e:
            call()
        assert e.value.code == rl.RLKV_EINVAL
    big = rand_bf16((11, B, Hkv, D), 3, cuda_device)
    with pytest.raises(rl.RlkvError) as e:
        rl.rlkv_prefill(cache.handle, 0, big, big, 11)
    assert e.value.code == rl.RLKV_EFULL
    assert cache.length(0) == 0 and not out.any()
    gk, gv, gt = cache.export_head(0, 0, 0)
    assert not gk.any() and not gv.any() and (gt == -1).all()
    assert rl.rlkv_strerror(rl.RLKV_EFULL) and cache.status() == 0


# ------------------------------------------------------------------------------------------ step API
def test_step_and_step_host_equal_per_layer_calls(rl, hz, cuda_device):
    w = synth.WORKLOADS["llama8b"].with_(layers=3, batch=2, context=200)
    mask = synth.head_mask(w.seed, w.layers, w.kv_heads, 0.4)
    a = hz.Cache(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, 260, mask, w.sink, w.window, device=cuda_device)
    b = hz.Cache(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, 260, mask, w.sink, w.window, device=cuda_device)
    c = hz.Cache(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, 260, mask, w.sink, w.window, device=cuda_device)
    oracle = Oracle(w.layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, 260, mask, w.sink, w.window, threads=8)
    for cache in (a, b, c):
        hz.fill_cache(cache, w, 200)
    for l in range(w.layers):
        K = synth.rows(w.seed, synth.STREAM_K, l, 0, 200, w.batch, w.kv_heads, w.head_dim)
        V = synth.rows(w.seed, synth.STREAM_V, l, 0, 200, w.batch, w.kv_heads, w.head_dim)
        for t in range(200):
            oracle.append(l, K[t], V[t])
    for t in range(200, 203):
        k, v, q = hz.step_inputs(w, t, cuda_device)
        out_a = torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=torch.float32, device=cuda_device)
        for l in range(w.layers):
            a.append(l, k[l], v[l])
            a.decode(l, q[l], out_a[l])
        out_b = torch.empty_like(out_a)
        rl.rlkv_step(b.handle, k, v, q, out_b)
        kh, vh, qh = (x.cpu().pin_memory() for x in (k, v, q))
        out_c = torch.empty(out_a.shape, dtype=torch.float32).pin_memory()
        rl.rlkv_step_host(c.handle, kh, vh, qh, out_c)
        torch.cuda.synchronize()
        # the step and the per-layer calls may cut the work differently: same values up to summation order
        assert torch.allclose(out_a, out_b, atol=1e-4, rtol=0) and torch.equal(out_b.cpu(), out_c)
        for l in range(w.layers):
            oracle.append(l, k[l].cpu(), v[l].cpu())
            check_out(out_a[l].cpu().numpy(), oracle.decode(l, q[l].cpu()))
    check_state(b, oracle)
    check_state(c, oracle)
    assert rl.rlkv_launch_count(b.handle) > 0


def test_reset_and_config_knobs(rl, hz, cuda_device):
    D, B, Hkv, Hq, n = 128, 2, 2, 8, 700
    cache, oracle = build_pair(hz, 1, Hkv, Hq, D, B, n, [1, 0], 16, 112, cuda_device)
    K, V, q = rand_bf16((n, B, Hkv, D), 1), rand_bf16((n, B, Hkv, D), 2), rand_bf16((B, Hq, D), 3)
    feed(cache, oracle, 0, K, V, True)
    want = oracle.decode(0, q)
    outs = []
    for cps, st, ng, it in ((1, 6, 1, 0), (1, 2, 2, 2), (2, 2, 1, 3), (1, 3, 3, 2), (2, 2, 2, 5), (1, 4, 2, 16),
                            (1, 0, 3, 7), (1, 5, 1, 1024), (1, 3, 3, 4), (1, 4, 2, 4)):
        rl.rlkv_set_decode_config(cache.handle, cps, st, ng, it)
        outs.append(cache.decode(0, q.to(cuda_device)).cpu().numpy())
        check_out(outs[-1], want)
        again = cache.decode(0, q.to(cuda_device)).cpu().numpy()
        assert np.array_equal(outs[-1], again)      # which CTA claims which item must not matter
    for bad in ((2, 6, 1),      # does not fit in shared memory twice
                (1, 5, 2), (1, 4, 3),    # stages must be a multiple of the consumer groups
                (1, 6, 2, 1)):           # work items have at least 2 tiles
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_set_decode_config(cache.handle, *bad)
        assert e.value.code == rl.RLKV_EINVAL
    rl.rlkv_cache_reset(cache.handle)
    assert cache.length(0) == 0
    gk, gv, gt = cache.export_head(0, 0, 1)
    assert not gk.any() and not gv.any() and (gt == -1).all()
    feed(cache, Oracle(1, Hkv, Hq, D, B, n, [1, 0], 16, 112), 0, K[:100], V[:100], True)
    o2 = Oracle(1, Hkv, Hq, D, B, n, [1, 0], 16, 112)
    for t in range(100):
        o2.append(0, K[t], V[t])
    check_out(cache.decode(0, q.to(cuda_device)).cpu().numpy(), o2.decode(0, q))


# ------------------------------------------------------------------------------------------ work claims
def test_dynamic_work_claims_do_not_change_bits(rl, hz, cuda_device):
    """A shape with a few hundred work items over all SMs: the items a CTA gets beyond its first are
    claimed at run time, so repeated calls distribute them differently -- the output bits must not
    move, and every unit that is split over items must still match the oracle."""
    layers, Hkv, Hq, D, B, S, W, n = 1, 8, 32, 128, 4, 16, 112, 3001
    mask = [1, 1, 0, 1, 1, 0, 1, 1]
    cache, oracle = build_pair(hz, layers, Hkv, Hq, D, B, n + 1, mask, S, W, cuda_device)
    K, V, q = rand_bf16((n, B, Hkv, D), 41), rand_bf16((n, B, Hkv, D), 42), rand_bf16((B, Hq, D), 43)
    feed(cache, oracle, 0, K, V, True)
    want = oracle.decode(0, q)
    qd = q.to(cuda_device)
    first = cache.decode(0, qd).clone()
    check_out(first.cpu().numpy(), want)
    for it in (4, 2, 9):
        rl.rlkv_set_decode_config(cache.handle, 0, 0, 0, it)
        ref = cache.decode(0, qd).clone()
        check_out(ref.cpu().numpy(), want)
        for _ in range(4):
            assert torch.equal(cache.decode(0, qd), ref)
    assert cache.status() == 0
    # the trace counts what the launch did: every tile was consumed exactly once
    rl.rlkv_debug_trace(cache.handle, 1)
    cache.decode(0, qd)
    words = rl.rlkv_debug_trace(cache.handle, 0, read=True)
    tiles = B * (6 * ((n + 63) // 64) + 2 * 2)
    assert int(words[:, 5].sum()) == tiles


# ------------------------------------------------------------------------------------------ decode loop
@pytest.mark.parametrize("step_mode", [1, 2], ids=["launch_per_layer", "one_launch"])
@pytest.mark.parametrize("layers", [1, 2])
def test_long_decode_loop_through_rlkv_step(rl, hz, cuda_device, layers, step_mode):
    """A reduced chain-of-thought loop: prompt of 300 tokens, then 700 whole steps through rlkv_step
    (whose launches overlap one another on the device), sink 16 + window 240 so the ring wraps several
    times.  Outputs are compared with the oracle every 50 steps and at the end, cache state bit for bit
    at the end.  One layer is the case where an append may not run beside the decode before it."""
    Hkv, Hq, D, B, S, W, prompt, steps = 2, 8, 128, 2, 16, 240, 300, 700
    mask = ([1, 0] + [0, 1])[:2 * layers]
    cache, oracle = build_pair(hz, layers, Hkv, Hq, D, B, prompt + steps, mask, S, W, cuda_device)
    rl.rlkv_set_step_mode(cache.handle, step_mode)
    for l in range(layers):
        feed(cache, oracle, l, rand_bf16((prompt, B, Hkv, D), 50 + l), rand_bf16((prompt, B, Hkv, D), 60 + l), True)
    out = torch.empty((layers, B, Hq, D), dtype=torch.float32, device=cuda_device)
    K = rand_bf16((steps, layers, B, Hkv, D), 70)
    V = rand_bf16((steps, layers, B, Hkv, D), 71)
    Q = rand_bf16((steps, layers, B, Hq, D), 72)
    Kd, Vd, Qd = K.to(cuda_device), V.to(cuda_device), Q.to(cuda_device)
    for t in range(steps):
        rl.rlkv_step(cache.handle, Kd[t], Vd[t], Qd[t], out)
        for l in range(layers):
            assert oracle.append(l, K[t, l], V[t, l]) == 0
        if t % 50 == 49 or t == steps - 1:
            got = out.cpu().numpy()
            for l in range(layers):
                check_out(got[l], oracle.decode(l, Q[t, l]))
    check_state(cache, oracle)
    assert cache.status() == 0
    with pytest.raises(rl.RlkvError) as e:
        rl.rlkv_step(cache.handle, Kd[0], Vd[0], Qd[0], out)
    assert e.value.code == rl.RLKV_EFULL


def test_reduced_loop_of_4000_steps_checked_at_every_step(rl, hz, cuda_device):
    """The long decode loop at a reduced shape (2 layers, batch 2, 8/2 heads, prompt 300, sink 16 +
    window 240, 4000 steps: the rings wrap 16 times).  At EVERY step the outputs of both layers are
    compared with the oracle and the rings of the compressed heads bit for bit; the whole cache state
    every 250 steps and at the end."""
    layers, Hkv, Hq, D, B, S, W, prompt, steps = 2, 2, 8, 128, 2, 16, 240, 300, 4000
    mask = [1, 0, 0, 1]
    cache, oracle = build_pair(hz, layers, Hkv, Hq, D, B, prompt + steps, mask, S, W, cuda_device)
    for l in range(layers):
        feed(cache, oracle, l, rand_bf16((prompt, B, Hkv, D), 250 + l), rand_bf16((prompt, B, Hkv, D), 260 + l), True)
    out = torch.empty((layers, B, Hq, D), dtype=torch.float32, device=cuda_device)
    block = 500
    for t0 in range(0, steps, block):
        K = rand_bf16((block, layers, B, Hkv, D), 270 + t0)
        V = rand_bf16((block, layers, B, Hkv, D), 271 + t0)
        Q = rand_bf16((block, layers, B, Hq, D), 272 + t0)
        Kd, Vd, Qd = K.to(cuda_device), V.to(cuda_device), Q.to(cuda_device)
        for i in range(block):
            rl.rlkv_step(cache.handle, Kd[i], Vd[i], Qd[i], out)
            got = out.cpu().numpy()
            for l in range(layers):
                assert oracle.append(l, K[i, l], V[i, l]) == 0
                check_out(got[l], oracle.decode(l, Q[i, l]))
                h = mask[l * Hkv:(l + 1) * Hkv].index(0)     # the layer's compressed head
                for b in range(B):
                    for g_, o_ in zip(cache.export_head(l, b, h), oracle.export_head(l, b, h)):
                        np.testing.assert_array_equal(g_, o_)
            if (t0 + i) % 250 == 249:
                check_state(cache, oracle)
    check_state(cache, oracle)
    assert cache.length(0) == prompt + steps and cache.status() == 0


@pytest.mark.parametrize("step_mode", [1, 2], ids=["launch_per_layer", "one_launch"])
def test_step_mixes_tiny_and_gpu_filling_launches(rl, hz, cuda_device, step_mode):
    """Seven layers that alternate between a few work items and more than one per SM (all heads
    compressed, one full head, all full).  With one launch per layer every launch of the step starts
    beside its predecessor and holds its own successor back until that predecessor has completed; with
    one launch for the step the layers' units share one flat tile space.  60 consecutive steps, every
    layer against the oracle at several of them, and the step's results equal to the per-layer calls on
    a twin cache."""
    Hkv, Hq, D, B, S, W, prompt, steps = 4, 16, 128, 6, 8, 56, 3000, 60
    mask = [0, 0, 0, 0,  1, 1, 1, 1,  0, 1, 0, 0,  0, 0, 0, 0,  0, 0, 0, 0,  1, 1, 1, 1,  1, 0, 0, 1]
    layers = len(mask) // Hkv
    cache, oracle = build_pair(hz, layers, Hkv, Hq, D, B, prompt + steps, mask, S, W, cuda_device)
    rl.rlkv_set_step_mode(cache.handle, step_mode)
    twin = hz.Cache(layers, Hkv, Hq, D, B, prompt + steps, mask, S, W, device=cuda_device)
    for l in range(layers):
        K, V = rand_bf16((prompt, B, Hkv, D), 150 + l), rand_bf16((prompt, B, Hkv, D), 160 + l)
        feed(cache, oracle, l, K, V, True)
        twin.prefill(l, K.to(cuda_device), V.to(cuda_device))
    out = torch.empty((layers, B, Hq, D), dtype=torch.float32, device=cuda_device)
    K, V = rand_bf16((steps, layers, B, Hkv, D), 170), rand_bf16((steps, layers, B, Hkv, D), 171)
    Q = rand_bf16((steps, layers, B, Hq, D), 172)
    Kd, Vd, Qd = K.to(cuda_device), V.to(cuda_device), Q.to(cuda_device)
    for t in range(steps):
        rl.rlkv_step(cache.handle, Kd[t], Vd[t], Qd[t], out)
        for l in range(layers):
            assert oracle.append(l, K[t, l], V[t, l]) == 0
            twin.append(l, Kd[t, l], Vd[t, l])
        if t in (0, 1, 2, 31, steps - 1):
            got = out.cpu().numpy()
            for l in range(layers):
                check_out(got[l], oracle.decode(l, Q[t, l]))
                # the two cut the rows differently, so P is rounded to bf16 against different running
                # maxima: the difference is rounding noise (a few 1e-5 per element at this length)
                np.testing.assert_allclose(got[l], twin.decode(l, Qd[t, l]).cpu().numpy(), atol=5e-4, rtol=0)
    check_state(cache, oracle)
    assert cache.status() == 0 and twin.status() == 0


def test_one_launch_step_against_launch_per_layer_and_oracle(rl, hz, cuda_device):
    """rlkv_step as one attention launch over all layers against the same step with one launch per layer
    and against the oracle, on shapes where the whole-step schedule has a prefix of whole units (many
    units), where it has none (few tiles), with layers that hold no full or no compressed head, and
    with head_dim 64.  A step whose layers hold different numbers of tokens falls back to one launch per
    layer and is still right.  Planted needles: in every layer one batch row's newest token (written by
    the step's own append launch, which the attention launch may start beside) and its first token carry
    markers that must show in the output."""
    cases = [
        # layers, Hkv, Hq, D, B, S, W, n, fraction compressed
        (6, 4, 16, 128, 8, 16, 48, 3000, 0.4),
        (5, 2, 8, 64, 2, 4, 60, 150, 0.5),
        (3, 8, 32, 128, 1, 16, 112, 5000, 0.8),
        (4, 4, 4, 128, 3, 8, 24, 700, 0.0),
        (4, 4, 28, 128, 3, 8, 24, 700, 1.0),
    ]
    for ci, (layers, Hkv, Hq, D, B, S, W, n, frac) in enumerate(cases):
        mask = synth.head_mask(40 + ci, layers, Hkv, frac)
        a, oracle = build_pair(hz, layers, Hkv, Hq, D, B, n + 8, mask, S, W, cuda_device)
        b = hz.Cache(layers, Hkv, Hq, D, B, n + 8, mask, S, W, device=cuda_device)
        rl.rlkv_set_step_mode(a.handle, 2)
        rl.rlkv_set_step_mode(b.handle, 1)
        for l in range(layers):
            K, V = rand_bf16((n, B, Hkv, D), 500 + 10 * ci + l), rand_bf16((n, B, Hkv, D), 600 + 10 * ci + l)
            feed(a, oracle, l, K, V, True)
            b.prefill(l, K.to(cuda_device), V.to(cuda_device))
        out_a = torch.empty((layers, B, Hq, D), dtype=torch.float32, device=cuda_device)
        out_b = torch.empty_like(out_a)
        for t in range(3):
            k, v = rand_bf16((layers, B, Hkv, D), 700 + t), rand_bf16((layers, B, Hkv, D), 710 + t)
            q = rand_bf16((layers, B, Hq, D), 720 + t)
            if t == 1:                                       # needles: the token appended now, row 0 of every layer
                for l in range(layers):
                    for h in range(Hkv):
                        qq = q[l, 0, h * (Hq // Hkv)].to(torch.float32)
                        k[l, 0, h] = (qq / qq.norm() * 100.0).to(torch.bfloat16)
                        v[l, 0, h] = 5.0
            kd, vd, qd = k.to(cuda_device), v.to(cuda_device), q.to(cuda_device)
            rl.rlkv_step(a.handle, kd, vd, qd, out_a)
            rl.rlkv_step(b.handle, kd, vd, qd, out_b)
            got = out_a.cpu().numpy()
            assert torch.allclose(out_a, out_b, atol=5e-4, rtol=0)   # different cuts: rounding noise only
            for l in range(layers):
                assert oracle.append(l, k[l], v[l]) == 0
                check_out(got[l], oracle.decode(l, q[l]))
            if t == 1:
                G = Hq // Hkv
                assert np.abs(got[:, 0, ::G] - 5.0).max() < 1e-2     # the first query head of every group saw its needle
        check_state(a, oracle)
        # different lengths: one more token for layer 0 only, then a step
        k1, v1 = rand_bf16((B, Hkv, D), 800), rand_bf16((B, Hkv, D), 801)
        a.append(0, k1.to(cuda_device), v1.to(cuda_device))
        oracle.append(0, k1, v1)
        k, v, q = rand_bf16((layers, B, Hkv, D), 802), rand_bf16((layers, B, Hkv, D), 803), rand_bf16((layers, B, Hq, D), 804)
        rl.rlkv_step(a.handle, k.to(cuda_device), v.to(cuda_device), q.to(cuda_device), out_a)
        got = out_a.cpu().numpy()
        for l in range(layers):
            assert oracle.append(l, k[l], v[l]) == 0
            check_out(got[l], oracle.decode(l, q[l]))
        check_state(a, oracle)
        assert a.status() == 0 and b.status() == 0
        a.close()
        b.close()


@pytest.mark.parametrize("one_launch", [0, 1], ids=["append_then_attend", "layer_step"])
@pytest.mark.parametrize("overlap", [1, 0], ids=["neighbours_overlap", "ordinary_neighbours"])
@pytest.mark.parametrize("shape", [(4, 4, 16, 128, 8, 16, 48, 3000), (3, 2, 8, 64, 2, 4, 60, 100), (2, 8, 32, 128, 16, 16, 112, 1500),
                                   (2, 2, 4, 128, 3, 130, 62, 190)],
                         ids=["many_items", "shorter_than_the_ring", "wide", "ring_just_filling"])
def test_overlapped_per_layer_calls_wait_for_their_inputs(rl, hz, cuda_device, shape, overlap, one_launch):
    """The chain of a model forward: before every layer's attention a stand-in kernel copies that layer's
    k, v and q into the buffers the calls read -- at the very end of the kernel -- and
    rlkv_append_overlapped / rlkv_decode_attention_overlapped are launched right behind it so that they
    may start while it still runs.  Until the stand-in has finished, the buffers hold the previous
    layer's values: a call that read its inputs too early would append wrong rows (the state check is
    bit for bit) or attend with the wrong query.  Six steps over all layers, outputs against the
    oracle at every step, the state at the end; the same with ordinary launches around the calls, and
    with rlkv_layer_step_overlapped, whose one launch writes the token's rows itself."""
    layers, Hkv, Hq, D, B, S, W, n = shape
    mask = synth.head_mask(77, layers, Hkv, 0.4)
    cache, oracle = build_pair(hz, layers, Hkv, Hq, D, B, n + 8, mask, S, W, cuda_device)
    for l in range(layers):
        feed(cache, oracle, l, rand_bf16((n, B, Hkv, D), 900 + l), rand_bf16((n, B, Hkv, D), 910 + l), True)
    kv_elems, q_elems = B * Hkv * D, B * Hq * D
    buf = torch.zeros(2 * kv_elems + q_elems, dtype=torch.bfloat16, device=cuda_device)   # k | v | q of the current layer
    kb, vb, qb = buf[:kv_elems], buf[kv_elems:2 * kv_elems], buf[2 * kv_elems:]
    work_src = torch.ones(32 << 20, dtype=torch.uint8, device=cuda_device)                # the stand-in's own traffic
    work_dst = torch.empty_like(work_src)
    out = torch.empty((layers, B, Hq, D), dtype=torch.float32, device=cuda_device)
    for t in range(6):
        K, V, Q = rand_bf16((layers, B, Hkv, D), 920 + t), rand_bf16((layers, B, Hkv, D), 930 + t), rand_bf16((layers, B, Hq, D), 940 + t)
        src = [torch.cat([K[l].reshape(-1), V[l].reshape(-1), Q[l].reshape(-1)]).to(cuda_device) for l in range(layers)]
        torch.cuda.synchronize()
        for l in range(layers):
            rl.rlkv_debug_standin(work_dst, work_src, work_src.numel(), out[l - 1] if l else None, buf, src[l],
                                  buf.numel() * 2, overlap)
            if one_launch:
                rl.rlkv_layer_step_overlapped(cache.handle, l, kb, vb, qb, out[l])
            else:
                rl.rlkv_append_overlapped(cache.handle, l, kb, vb)
                rl.rlkv_decode_attention_overlapped(cache.handle, l, qb, out[l])
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        for l in range(layers):
            assert oracle.append(l, K[l], V[l]) == 0
            check_out(got[l], oracle.decode(l, Q[l]))
    check_state(cache, oracle)
    # the overlapped call and the ordinary one cut the work alike: the same bits
    ref = cache.decode(0, qb)
    again = torch.empty_like(ref)
    rl.rlkv_decode_attention_overlapped(cache.handle, 0, qb, again)
    assert torch.equal(ref, again)
    assert cache.status() == 0


def test_step_host_in_chunks_over_several_steps(rl, hz, cuda_device):
    """Nine layers, so that rlkv_step_host brings inputs in and takes results out in chunks on its side
    streams, and consecutive calls alternate between its two input staging areas: five steps in a row
    without synchronising in between, every result compared with rlkv_step on a twin cache and with
    the oracle."""
    layers, Hkv, Hq, D, B, S, W, n0, steps = 9, 2, 4, 64, 2, 4, 28, 150, 5
    mask = [1, 0] * layers
    a = hz.Cache(layers, Hkv, Hq, D, B, n0 + steps, mask, S, W, device=cuda_device)
    b, oracle = build_pair(hz, layers, Hkv, Hq, D, B, n0 + steps, mask, S, W, cuda_device)
    for l in range(layers):
        K, V = rand_bf16((n0, B, Hkv, D), 80 + l), rand_bf16((n0, B, Hkv, D), 90 + l)
        a.prefill(l, K.to(cuda_device), V.to(cuda_device))
        feed(b, oracle, l, K, V, True)
    ins = [(rand_bf16((layers, B, Hkv, D), 100 + t).pin_memory(), rand_bf16((layers, B, Hkv, D), 110 + t).pin_memory(),
            rand_bf16((layers, B, Hq, D), 120 + t).pin_memory()) for t in range(steps)]
    outs = [torch.empty((layers, B, Hq, D), dtype=torch.float32).pin_memory() for _ in range(steps)]
    for t in range(steps):                                   # back to back: copies and kernels of
        rl.rlkv_step_host(a.handle, *ins[t], outs[t])        # neighbouring calls overlap
    torch.cuda.synchronize()
    for t in range(steps):
        k, v, q = (x.to(cuda_device) for x in ins[t])
        ref = torch.empty((layers, B, Hq, D), dtype=torch.float32, device=cuda_device)
        rl.rlkv_step(b.handle, k, v, q, ref)
        assert torch.allclose(ref.cpu(), outs[t], atol=5e-4, rtol=0)   # cut differently: rounding noise only
        for l in range(layers):
            oracle.append(l, ins[t][0][l], ins[t][1][l])
            check_out(outs[t][l].numpy(), oracle.decode(l, ins[t][2][l]))
    check_state(a, oracle)
    assert a.status() == 0 and b.status() == 0


# ------------------------------------------------------------------------------------------ bf16 output
def test_bf16_output_is_the_rounded_fp32_output(rl, hz, cuda_device):
    """rlkv_set_output_bf16: the same arithmetic, results rounded to nearest even when stored -- so
    the bf16 result must equal the fp32 result of the same call converted by torch, bit for bit, for
    the per-layer call, the whole step on device buffers and the step on host buffers."""
    layers, Hkv, Hq, D, B, S, W, n = 8, 4, 16, 128, 3, 16, 48, 700
    mask = synth.head_mask(5, layers, Hkv, 0.4)
    caches = []
    for _ in range(2):
        c = hz.Cache(layers, Hkv, Hq, D, B, n + 8, mask, S, W, device=cuda_device)
        for l in range(layers):
            c.prefill(l, rand_bf16((n, B, Hkv, D), 10 + l, cuda_device), rand_bf16((n, B, Hkv, D), 50 + l, cuda_device))
        caches.append(c)
    f32, b16 = caches
    oracle = Oracle(layers, Hkv, Hq, D, B, n + 8, mask, S, W, threads=8)
    for l in range(layers):
        Kc, Vc = rand_bf16((n, B, Hkv, D), 10 + l), rand_bf16((n, B, Hkv, D), 50 + l)
        for t in range(n):
            assert oracle.append(l, Kc[t], Vc[t]) == 0
    rl.rlkv_set_output_bf16(b16.handle, 1)
    q = rand_bf16((layers, B, Hq, D), 90, cuda_device)

    def check_bf16(got, want):
        """bf16 results against the oracle's fp32 ones: the usual bounds, widened by the half ulp that
        the final rounding to bf16 may add (2^-9 of the value)."""
        got, want = got.float().cpu().numpy().astype(np.float64), np.asarray(want, np.float64)
        err = np.abs(got - want)
        half_ulp = np.abs(want) * 2.0 ** -8
        rms = np.sqrt((want ** 2).mean(axis=-1, keepdims=True))
        assert np.isfinite(got).all()
        assert (err <= MAX_ABS + half_ulp).all() and err.mean() <= MEAN_ABS + half_ulp.mean()
        assert (err <= REL_RMS * rms + half_ulp + 1e-6).all()

    # per-layer call
    want = f32.decode(0, q[0])
    got = torch.empty((B, Hq, D), dtype=torch.bfloat16, device=cuda_device)
    rl.rlkv_decode_attention(b16.handle, 0, q[0], got)
    assert torch.equal(got, want.to(torch.bfloat16))
    ref0 = oracle.decode(0, q[0].cpu())
    check_out(want.cpu().numpy(), ref0)
    check_bf16(got, ref0)
    # whole step, device buffers
    k, v = rand_bf16((layers, B, Hkv, D), 91, cuda_device), rand_bf16((layers, B, Hkv, D), 92, cuda_device)
    want = torch.empty((layers, B, Hq, D), dtype=torch.float32, device=cuda_device)
    got = torch.zeros((layers, B, Hq, D), dtype=torch.bfloat16, device=cuda_device)
    rl.rlkv_step(f32.handle, k, v, q, want)
    rl.rlkv_step(b16.handle, k, v, q, got)
    assert torch.equal(got, want.to(torch.bfloat16))
    for l in range(layers):                                  # both against the oracle, every layer
        assert oracle.append(l, k[l].cpu(), v[l].cpu()) == 0
        ref = oracle.decode(l, q[l].cpu())
        check_out(want[l].cpu().numpy(), ref)
        check_bf16(got[l], ref)
    # whole step, host buffers
    kh, vh, qh = (x.cpu().pin_memory() for x in (k, v, q))
    want_h = torch.empty((layers, B, Hq, D), dtype=torch.float32).pin_memory()
    got_h = torch.zeros((layers, B, Hq, D), dtype=torch.bfloat16).pin_memory()
    rl.rlkv_step_host(f32.handle, kh, vh, qh, want_h)
    rl.rlkv_step_host(b16.handle, kh, vh, qh, got_h)
    torch.cuda.synchronize()
    assert torch.equal(got_h, want_h.to(torch.bfloat16))
    # mixed attention writes its rows once, so it can round them as well; back to fp32, the cache works as before
    allf = hz.Cache(1, Hkv, Hq, D, B, 400, np.ones(Hkv, np.uint8), S, W, device=cuda_device)
    allf.prefill(0, rand_bf16((300, B, Hkv, D), 93, cuda_device), rand_bf16((300, B, Hkv, D), 94, cuda_device))
    gates = torch.rand(Hkv, device=cuda_device)
    mixed32 = allf.decode_mixed(0, q[0], gates)
    rl.rlkv_set_output_bf16(allf.handle, 1)
    mixed16 = torch.empty((B, Hq, D), dtype=torch.bfloat16, device=cuda_device)
    rl.rlkv_decode_mixed_attention(allf.handle, 0, q[0], gates, mixed16)
    assert torch.equal(mixed16, mixed32.to(torch.bfloat16))
    rl.rlkv_set_output_bf16(b16.handle, 0)
    assert torch.equal(b16.decode(1, q[1]), f32.decode(1, q[1]))
    assert f32.status() == 0 and b16.status() == 0
    for c in caches + [allf]:
        c.close()
