"""GPU parity of the paged, ragged cache (rlkv_paged_*): every sequence must come out exactly as a
batch row of its own would -- the oracle is one single-sequence oracle per request slot.  Cache
state is compared bit for bit (full heads gathered page by page in token order, compressed heads as
their physical ring), attention outputs within the bounds of the other parity tests.
"""
import numpy as np
import pytest
import torch

from oracle.rlkv_oracle import Oracle
from test_gpu_parity import check_out, rand_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rl(cuda_device):
    import paper_2510_08525_b200.binding as binding
    return binding


@pytest.fixture(scope="module")
def hz(cuda_device):
    import paper_2510_08525_b200.harness as harness
    return harness


class Seq:
    """One request: its slot in the cache under test and its own oracle."""

    def __init__(self, cache, seed, max_len, scales=None):
        self.cache, self.seed = cache, seed
        self.slot = cache.open_seq()
        self.oracle = Oracle(cache.layers, cache.kv_heads, cache.q_heads, cache.head_dim, 1, max_len,
                             cache.mask.reshape(-1), cache.sink, cache.window, threads=4)
        if scales is not None:                                # all heads in 8-bit storage
            self.oracle.set_fp8(*scales)
        self.n = 0

    def rows(self, layer, t0, t1, what):
        return rand_bf16((t1 - t0, self.cache.kv_heads, self.cache.head_dim),
                         (self.seed * 131 + layer) * 100003 + t0 * 7 + what)

    def prefill(self, n, dev):
        for layer in range(self.cache.layers):
            K, V = self.rows(layer, self.n, self.n + n, 0), self.rows(layer, self.n, self.n + n, 1)
            self.cache.prefill(layer, self.slot, K.to(dev), V.to(dev))
            for t in range(n):
                assert self.oracle.append(layer, K[t], V[t]) == 0
        self.n += n


def append_all(cache, seqs, dev):
    """One token for every sequence of `seqs`, every layer, in one call per layer."""
    for layer in range(cache.layers):
        ks = [s.rows(layer, s.n, s.n + 1, 0) for s in seqs]
        vs = [s.rows(layer, s.n, s.n + 1, 1) for s in seqs]
        cache.append(layer, [s.slot for s in seqs], torch.cat(ks).to(dev), torch.cat(vs).to(dev))
        for s, k, v in zip(seqs, ks, vs):
            assert s.oracle.append(layer, k[0], v[0]) == 0
    for s in seqs:
        s.n += 1


def check_decode(cache, seqs, dev, seed, layers=None):
    for layer in (range(cache.layers) if layers is None else layers):
        q = rand_bf16((len(seqs), cache.q_heads, cache.head_dim), seed + layer)
        out = cache.decode(layer, [s.slot for s in seqs], q.to(dev))
        again = cache.decode(layer, [s.slot for s in seqs], q.to(dev))
        assert torch.equal(out, again)                       # the same call, the same bits
        out = out.cpu().numpy()
        for i, s in enumerate(seqs):
            check_out(out[i], s.oracle.decode(layer, q[i:i + 1])[0])


def check_state(cache, seqs):
    for s in seqs:
        for layer in range(cache.layers):
            assert cache.length(layer, s.slot) == s.oracle.length(layer) == s.n
            for h in range(cache.kv_heads):
                gk, gv, gt = cache.export_head(layer, s.slot, h)
                ok, ov, ot = s.oracle.export_head(layer, 0, h)
                rows = s.n if cache.mask[layer, h] else cache.sink + cache.window
                assert len(gt) == rows
                np.testing.assert_array_equal(gt, ot[:rows])
                np.testing.assert_array_equal(gk, ok[:rows])
                np.testing.assert_array_equal(gv, ov[:rows])


SHAPES = [
    # layers, Hkv, Hq, D, S, W, mask, lengths
    (1, 2, 8, 64, 4, 60, "10", [1]),
    (1, 2, 8, 64, 4, 60, "01", [63, 64, 65]),
    (2, 2, 8, 64, 4, 12, "1001", [5, 200, 17, 129]),
    (1, 4, 28, 128, 16, 112, "1001", [300, 1, 128, 1000, 77]),
    (2, 8, 32, 128, 16, 112, "11011011" "00100001", [900, 64, 2500, 130]),
    (1, 1, 8, 128, 0, 5, "0", [777, 3]),
    (1, 2, 4, 128, 100, 200, "11", [1500, 299, 301]),
    (1, 4, 16, 128, 16, 64, "0000", [400, 90]),
    (1, 2, 4, 64, 16, 112, "10", [40000, 100]),   # 625 pages: the prompt goes in over two prefill launches
]


@pytest.mark.parametrize("layers,Hkv,Hq,D,S,W,mask,lens", SHAPES)
def test_ragged_batch_matches_one_oracle_per_sequence(rl, hz, cuda_device, layers, Hkv, Hq, D, S, W, mask, lens):
    mask = [int(c) for c in mask]
    max_len = max(lens) + 8
    pages = sum((n + 2 + 63) // 64 for n in lens) + 2
    cache = hz.PagedCache(layers, Hkv, Hq, D, len(lens) + 1, pages, max_len, mask, S, W, device=cuda_device)
    seqs = []
    for i, n in enumerate(lens):
        s = Seq(cache, i + 1, max_len)
        if n > 1:
            s.prefill(n - 1, cuda_device)
        seqs.append(s)
    append_all(cache, seqs, cuda_device)                     # the decode step's own token, for everyone
    check_decode(cache, seqs, cuda_device, 500)
    check_state(cache, seqs)
    # a subset, in another order, after one more token for that subset only
    sub = seqs[::-1][: max(1, len(seqs) // 2)]
    append_all(cache, sub, cuda_device)
    check_decode(cache, sub, cuda_device, 600)
    check_state(cache, seqs)
    want = sum(int(cache.mask[0].sum()) * s.n + int((1 - cache.mask[0]).sum()) * min(s.n, S + W) for s in sub) * 4 * D
    assert cache.step_bytes(0, [s.slot for s in sub]) == want
    assert cache.status() == 0
    cache.close()


def test_continuous_batching_slots_and_pages_are_reused(rl, hz, cuda_device):
    """Requests arrive, grow token by token across page boundaries, finish and hand their pages to
    newcomers; every step is checked for the sequences alive at that moment."""
    layers, Hkv, Hq, D, S, W = 2, 4, 16, 128, 8, 56
    mask = [1, 0, 1, 1, 0, 1, 0, 0]
    cache = hz.PagedCache(layers, Hkv, Hq, D, 4, 12, 400, mask, S, W, device=cuda_device)
    assert cache.pages() == (12, 12)
    a, b = Seq(cache, 1, 400), Seq(cache, 2, 400)
    a.prefill(120, cuda_device)                              # 2 pages
    b.prefill(190, cuda_device)                              # 3 pages
    assert cache.pages() == (7, 12)
    live = [a, b]
    for step in range(12):                                   # a: 120 -> 132 (3rd page at 128), b: 190 -> 202 (4th at 192)
        append_all(cache, live, cuda_device)
        if step in (0, 7, 8, 11):
            check_decode(cache, live, cuda_device, 700 + step)
    assert cache.pages() == (5, 12)
    check_state(cache, live)
    # b finishes; c takes its slot and its pages
    slot_b = b.slot
    cache.close_seq(b.slot)
    assert cache.pages() == (9, 12)
    c = Seq(cache, 3, 400)
    assert c.slot == slot_b
    c.prefill(300, cuda_device)                              # 5 pages, four of them b's old ones
    assert cache.pages() == (4, 12)
    live = [c, a]
    for step in range(5):
        append_all(cache, live, cuda_device)
    check_decode(cache, live, cuda_device, 800)
    check_state(cache, live)
    # the free list runs dry: refused, and nothing has changed for anybody
    d = Seq(cache, 4, 400)
    with pytest.raises(rl.RlkvError) as e:
        d.cache.prefill(0, d.slot, rand_bf16((4 * 64 + 1, Hkv, D), 9).to(cuda_device),
                        rand_bf16((4 * 64 + 1, Hkv, D), 10).to(cuda_device))
    assert e.value.code == rl.RLKV_EFULL
    assert cache.pages() == (4, 12) and cache.length(0, d.slot) == 0
    check_decode(cache, live, cuda_device, 900)
    assert cache.status() == 0
    cache.close()


def test_paged_argument_checks(rl, hz, cuda_device):
    Hkv, Hq, D = 2, 8, 64
    cache = hz.PagedCache(1, Hkv, Hq, D, 2, 2, 128, [1, 0], 4, 12, device=cuda_device)
    k = rand_bf16((2, Hkv, D), 1).to(cuda_device)
    q = rand_bf16((2, Hq, D), 2).to(cuda_device)
    out = torch.full((2, Hq, D), 3.0, dtype=torch.float32, device=cuda_device)
    s0, s1 = cache.open_seq(), cache.open_seq()
    with pytest.raises(rl.RlkvError) as e:                   # no third slot
        cache.open_seq()
    assert e.value.code == rl.RLKV_EFULL
    for bad in ([s0, s0], [5], [-1], []):
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_paged_append(cache.handle, 0, bad, k, k)
        assert e.value.code == rl.RLKV_EINVAL
    with pytest.raises(rl.RlkvError) as e:                   # nothing cached yet
        rl.rlkv_paged_decode_attention(cache.handle, 0, [s0, s1], q, out)
    assert e.value.code == rl.RLKV_EEMPTY
    cache.append(0, [s0, s1], k, k)
    assert cache.pages() == (0, 2)
    cache.close_seq(s1)
    with pytest.raises(rl.RlkvError) as e:                   # a closed slot
        rl.rlkv_paged_append(cache.handle, 0, [s1], k, k)
    assert e.value.code == rl.RLKV_EINVAL
    for _ in range(127):
        cache.append(0, [s0], k[:1], k[:1])
    assert cache.length(0, s0) == 128
    with pytest.raises(rl.RlkvError) as e:                   # at max_seq_len
        cache.append(0, [s0], k[:1], k[:1])
    assert e.value.code == rl.RLKV_EFULL
    assert cache.length(0, s0) == 128
    torch.cuda.synchronize()
    assert (out == 3.0).all()
    assert cache.status() == 0
    cache.close()


def test_max_seq_len_is_the_limit_even_with_pages_to_spare(rl, hz, cuda_device):
    """max_seq_len = 100 is no multiple of the page (64) nor of the table's padding (256 tokens), and
    the free list holds far more pages than one sequence can use: append, prefill and step must all
    refuse token 100 with RLKV_EFULL and leave lengths, page table and free list as they were."""
    Hkv, Hq, D = 2, 4, 64
    cache = hz.PagedCache(2, Hkv, Hq, D, 2, 16, 100, [1, 0, 0, 1], 4, 12, device=cuda_device)
    s0, s1 = cache.open_seq(), cache.open_seq()
    k = rand_bf16((100, Hkv, D), 5).to(cuda_device)
    with pytest.raises(rl.RlkvError) as e:                   # 101 tokens at once
        rl.rlkv_paged_prefill(cache.handle, 0, s0, torch.cat([k, k[:1]]), torch.cat([k, k[:1]]), 101)
    assert e.value.code == rl.RLKV_EFULL and cache.length(0, s0) == 0 and cache.pages() == (16, 16)
    for layer in range(2):
        cache.prefill(layer, s0, k[:99], k[:99])
        cache.prefill(layer, s1, k[:40], k[:40])
    assert cache.pages() == (16 - 2 - 1, 16)
    with pytest.raises(rl.RlkvError) as e:                   # 99 + 2 > 100
        rl.rlkv_paged_prefill(cache.handle, 0, s0, k[:2], k[:2], 2)
    assert e.value.code == rl.RLKV_EFULL and cache.length(0, s0) == 99
    q = rand_bf16((2, 2, Hq, D), 6).to(cuda_device)
    out = torch.empty((2, 2, Hq, D), dtype=torch.float32, device=cuda_device)
    kv = k[:4].reshape(2, 2, Hkv, D).contiguous()
    rl.rlkv_paged_step(cache.handle, [s0, s1], kv, kv, q, out)   # token 99 of s0: the last one allowed
    assert [cache.length(l, s0) for l in range(2)] == [100, 100] and cache.length(0, s1) == 41
    free = cache.pages()
    with pytest.raises(rl.RlkvError) as e:
        rl.rlkv_paged_step(cache.handle, [s0, s1], kv, kv, q, out)
    assert e.value.code == rl.RLKV_EFULL
    with pytest.raises(rl.RlkvError) as e:                   # nothing appended for s1 either
        rl.rlkv_paged_append(cache.handle, 1, [s1, s0], kv[0], kv[0])
    assert e.value.code == rl.RLKV_EFULL
    assert [cache.length(l, s) for l in range(2) for s in (s0, s1)] == [100, 41, 100, 41]
    assert cache.pages() == free
    rows = cache.export_head(0, s0, 0)                       # a buffer of max_seq_len rows is enough
    assert rows[0].shape[0] == 100
    assert cache.status() == 0
    cache.close()


def test_many_ragged_sequences_at_a_serving_shape(rl, hz, cuda_device):
    """48 requests of 40 .. 5000 tokens over 8/32 heads of 128 with a mixed mask: sampled sequences
    against their oracles (the long ones split over many work items, the short ones lie inside one)."""
    layers, Hkv, Hq, D, S, W = 1, 8, 32, 128, 16, 112
    mask = [1, 1, 0, 1, 1, 0, 1, 1]
    rng = np.random.default_rng(3)
    lens = [int(x) for x in rng.integers(40, 5000, size=48)]
    lens[5], lens[17] = 64 * 70, 1
    pages = sum((n + 63) // 64 for n in lens) + 4
    cache = hz.PagedCache(layers, Hkv, Hq, D, 64, pages, 5200, mask, S, W, device=cuda_device)
    seqs = []
    for i, n in enumerate(lens):
        s = Seq(cache, 50 + i, n + 2)
        s.prefill(n, cuda_device)
        seqs.append(s)
    q = rand_bf16((len(seqs), Hq, D), 4242)
    out = cache.decode(0, [s.slot for s in seqs], q.to(cuda_device)).cpu().numpy()
    assert np.isfinite(out).all()
    for i in [0, 5, 17, 23, 31, 47, int(np.argmax(lens)), int(np.argmin(lens))]:
        check_out(out[i], seqs[i].oracle.decode(0, q[i:i + 1])[0])
    assert cache.status() == 0
    cache.close()


def test_paged_bf16_output_is_the_rounded_fp32_output(rl, hz, cuda_device):
    Hkv, Hq, D, S, W = 4, 16, 128, 16, 48
    cache = hz.PagedCache(1, Hkv, Hq, D, 3, 40, 1000, [1, 0, 1, 1], S, W, device=cuda_device)
    seqs = [Seq(cache, i + 1, 1000) for i in range(3)]
    for s, n in zip(seqs, (900, 33, 257)):
        s.prefill(n, cuda_device)
    q = rand_bf16((3, Hq, D), 77).to(cuda_device)
    slots = [s.slot for s in seqs]
    want = cache.decode(0, slots, q)
    rl.rlkv_paged_set_output_bf16(cache.handle, 1)
    got = torch.zeros((3, Hq, D), dtype=torch.bfloat16, device=cuda_device)
    rl.rlkv_paged_decode_attention(cache.handle, 0, slots, q, got)
    assert torch.equal(got, want.to(torch.bfloat16))
    rl.rlkv_paged_set_output_bf16(cache.handle, 0)
    assert torch.equal(cache.decode(0, slots, q), want)
    assert cache.status() == 0
    cache.close()


def test_four_hundred_sequences_in_one_call(rl, hz, cuda_device):
    """More requests than the paper's largest serving batch (375, Table 3) in one append and one decode
    call: 400 sequences of 1 .. 260 tokens, one full and one compressed head."""
    Hkv, Hq, D, S, W, n = 2, 4, 64, 4, 28, 400
    rng = np.random.default_rng(8)
    lens = [int(x) for x in rng.integers(1, 261, size=n)]
    pages = sum((x + 1 + 63) // 64 for x in lens) + 1
    cache = hz.PagedCache(1, Hkv, Hq, D, n, pages, 300, [1, 0], S, W, device=cuda_device)
    seqs = []
    for i, x in enumerate(lens):
        s = Seq(cache, 1000 + i, 300)
        if x > 1:
            s.prefill(x - 1, cuda_device)
        seqs.append(s)
    append_all(cache, seqs, cuda_device)
    q = rand_bf16((n, Hq, D), 31)
    out = cache.decode(0, [s.slot for s in seqs], q.to(cuda_device)).cpu().numpy()
    for i, s in enumerate(seqs):
        check_out(out[i], s.oracle.decode(0, q[i:i + 1])[0])
    with pytest.raises(rl.RlkvError) as e:                   # 513 would be too many for one call
        rl.rlkv_paged_decode_attention(cache.handle, 0, list(range(400)) + list(range(113)), q.to(cuda_device), out)
    assert e.value.code == rl.RLKV_EINVAL
    assert cache.status() == 0
    cache.close()


@pytest.mark.parametrize("step_mode", [1, 2], ids=["launch_per_layer", "one_launch"])
@pytest.mark.parametrize("shape", ["small", "filling", "uniform"])
def test_paged_step_equals_the_per_layer_calls(rl, hz, cuda_device, shape, step_mode):
    """rlkv_paged_step (one append launch for all layers, then one attention launch over every layer, or
    the layers' attention launches overlapped) over consecutive steps that cross page boundaries: every
    sequence against its oracle, and the page accounting as the per-layer calls would leave it.
    'small': a few work items; 'filling': more than one item per SM, lengths all different (every item
    of the whole-step launch is claimed); 'uniform': equal lengths (most units whole in one item per CTA)."""
    if shape == "small":
        layers, Hkv, Hq, D, S, W, lens = 5, 2, 8, 64, 4, 28, [60, 1, 126, 200]
        mask = [1, 0, 0, 0, 1, 1, 0, 1, 1, 0]
    elif shape == "uniform":
        layers, Hkv, Hq, D, S, W, lens = 4, 4, 16, 128, 16, 48, [1530] * 12
        mask = [1, 1, 0, 1] + [0, 0, 0, 0] + [1, 1, 1, 1] + [0, 1, 1, 0]
    else:
        layers, Hkv, Hq, D, S, W, lens = 3, 8, 32, 128, 16, 112, [3000, 1500, 2900, 700, 2047, 3100, 2500, 1000]
        mask = [1] * 8 + [1, 1, 0, 1, 1, 0, 1, 1] + [0] * 8
    steps = 6
    pages = sum((n + steps + 63) // 64 for n in lens) + 1
    cache = hz.PagedCache(layers, Hkv, Hq, D, len(lens), pages, max(lens) + 64, mask, S, W, device=cuda_device)
    rl.rlkv_paged_set_step_mode(cache.handle, step_mode)
    seqs = []
    for i, n in enumerate(lens):
        s = Seq(cache, 300 + i, max(lens) + 64)
        s.prefill(n, cuda_device)
        seqs.append(s)
    slots = [s.slot for s in seqs]
    out = torch.empty((layers, len(seqs), Hq, D), dtype=torch.float32, device=cuda_device)
    for step in range(steps):
        ks = torch.stack([torch.cat([s.rows(l, s.n, s.n + 1, 0) for s in seqs]) for l in range(layers)])
        vs = torch.stack([torch.cat([s.rows(l, s.n, s.n + 1, 1) for s in seqs]) for l in range(layers)])
        q = rand_bf16((layers, len(seqs), Hq, D), 2000 + step)
        rl.rlkv_paged_step(cache.handle, slots, ks.to(cuda_device), vs.to(cuda_device), q.to(cuda_device), out)
        for i, s in enumerate(seqs):
            for l in range(layers):
                assert s.oracle.append(l, ks[l, i], vs[l, i]) == 0
            s.n += 1
        got = out.cpu().numpy()
        for l in range(layers):
            for i, s in enumerate(seqs):
                check_out(got[l, i], s.oracle.decode(l, q[l, i:i + 1])[0])
    check_state(cache, seqs)
    assert cache.pages()[0] == pages - sum((s.n + 63) // 64 for s in seqs)
    # a sequence that is ahead in one layer cannot take part in a whole step
    k1 = rand_bf16((1, Hkv, D), 5).to(cuda_device)
    cache.append(0, [slots[0]], k1, k1)
    with pytest.raises(rl.RlkvError) as e:
        rl.rlkv_paged_step(cache.handle, slots, ks.to(cuda_device), vs.to(cuda_device), q.to(cuda_device), out)
    assert e.value.code == rl.RLKV_EINVAL
    assert cache.status() == 0
    cache.close()


# ------------------------------------------------------------------------------------------ 8-bit pages
FP8_SHAPES = [
    # layers, Hkv, Hq, S, W, mask, lengths
    (1, 2, 8, 4, 60, "10", [1, 63, 64, 65]),
    (2, 4, 28, 16, 112, "1001" "0111", [300, 1, 128, 1000, 77]),
    (1, 8, 32, 16, 112, "11111111", [900, 64, 2500]),
    (1, 1, 8, 0, 5, "1", [777, 3]),
    (1, 4, 16, 16, 64, "0000", [400, 90]),
    (1, 2, 8, 16, 112, "11", [9000, 4100]),              # long rows: split over many work items
    (3, 4, 16, 16, 112, "1011" "0110" "1111", [700] * 6),    # equal lengths: the whole step's schedule has its prefix
]


@pytest.mark.parametrize("layers,Hkv,Hq,S,W,mask,lens", FP8_SHAPES)
def test_fp8_pages_match_the_quantising_oracle(rl, hz, cuda_device, layers, Hkv, Hq, S, W, mask, lens):
    """rlkv_paged_create_fp8: the codes in the pages and in the rings equal the oracle's bit for bit (K
    in row order, V transposed back), outputs within the usual bounds of the oracle's attention over
    the dequantised rows.  Scales differ per head and are no powers of two."""
    D = 128
    mask = [int(c) for c in mask]
    rng = np.random.default_rng(17)
    ks = rng.uniform(0.008, 0.05, size=layers * Hkv).astype(np.float32)      # N(0,1) inputs reach about 4.5: some saturate
    vs = rng.uniform(0.02, 1.5, size=layers * Hkv).astype(np.float32)
    max_len = max(lens) + 8
    pages = sum((n + 2 + 63) // 64 for n in lens) + 2
    cache = hz.PagedCache(layers, Hkv, Hq, D, len(lens) + 1, pages, max_len, mask, S, W, device=cuda_device,
                          k_scale=ks, v_scale=vs)
    seqs = []
    for i, n in enumerate(lens):
        s = Seq(cache, i + 1, max_len, scales=(ks, vs))
        if n > 1:
            s.prefill(n - 1, cuda_device)
        seqs.append(s)
    append_all(cache, seqs, cuda_device)
    check_decode(cache, seqs, cuda_device, 500)
    check_state(cache, seqs)
    n_full = int(cache.mask[0].sum())
    want = sum((n_full * s.n + (Hkv - n_full) * min(s.n, S + W)) * 2 * D for s in seqs)
    assert cache.step_bytes(0, [s.slot for s in seqs]) == want       # a K row and a V row of codes: 2 * D bytes
    # whole steps on the same cache
    slots = [s.slot for s in seqs]
    out = torch.empty((layers, len(seqs), Hq, D), dtype=torch.float32, device=cuda_device)
    for step in range(3):
        kk = torch.stack([torch.cat([s.rows(l, s.n, s.n + 1, 0) for s in seqs]) for l in range(layers)])
        vv = torch.stack([torch.cat([s.rows(l, s.n, s.n + 1, 1) for s in seqs]) for l in range(layers)])
        q = rand_bf16((layers, len(seqs), Hq, D), 3000 + step)
        rl.rlkv_paged_step(cache.handle, slots, kk.to(cuda_device), vv.to(cuda_device), q.to(cuda_device), out)
        for i, s in enumerate(seqs):
            for l in range(layers):
                assert s.oracle.append(l, kk[l, i], vv[l, i]) == 0
            s.n += 1
        got = out.cpu().numpy()
        for l in range(layers):
            for i, s in enumerate(seqs):
                check_out(got[l, i], s.oracle.decode(l, q[l, i:i + 1])[0])
    check_state(cache, seqs)
    assert cache.status() == 0
    cache.close()


def test_fp8_argument_checks(rl, hz, cuda_device):
    ok = dict(layers=1, kv_heads=2, q_heads=8, head_dim=128, max_seqs=2, n_pages=4, max_seq_len=128,
              head_is_full=[1, 0], sink=4, window=12, k_scale=[1.0, 1.0], v_scale=[1.0, 1.0])
    for bad in (dict(head_dim=64), dict(k_scale=[0.0, 1.0]), dict(v_scale=[1.0, -2.0]), dict(k_scale=[float("nan"), 1.0]),
                dict(v_scale=[float("inf"), 1.0])):
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_paged_create_fp8(**{**ok, **bad})
        assert e.value.code == rl.RLKV_EINVAL
    h = rl.rlkv_paged_create_fp8(**ok)
    assert rl.rlkv_paged_size_fp8(1, 2, 8, 128, 2, 4, 128, [1, 0], 4, 12) < rl.rlkv_paged_size(1, 2, 8, 128, 2, 4, 128, [1, 0], 4, 12)
    rl.rlkv_paged_destroy(h)
