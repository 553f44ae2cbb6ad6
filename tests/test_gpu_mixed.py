"""GPU parity of rlkv_decode_mixed_attention (Eq. 1 of the paper: gate * full attention +
(1 - gate) * sink+window attention) against the CPU oracle, through the C ABI, within the bounds
the other parity tests use.  Shapes span several tiles, ragged tails, windows that start in the
middle of a tile, sequences shorter than sink + window, no sink at all and sinks longer than a tile.
"""
import numpy as np
import pytest
import torch

import synth
from oracle.rlkv_oracle import Oracle
from test_gpu_parity import check_out, check_state, feed, rand_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rl(cuda_device):
    import paper_2510_08525_b200.binding as binding
    return binding


@pytest.fixture(scope="module")
def hz(cuda_device):
    import paper_2510_08525_b200.harness as harness
    return harness


def gates(Hkv, seed, dev):
    g = torch.Generator().manual_seed(seed)
    a = torch.rand(Hkv, generator=g, dtype=torch.float32)
    if Hkv >= 2:
        a[0], a[-1] = 1.0, 0.0            # the two ends of Eq. 1 always take part
    return a, a.to(dev)


SHAPES = [
    # Hkv, Hq, D, B, S, W, n
    (2, 8, 64, 1, 4, 60, 1),
    (2, 8, 64, 2, 4, 60, 3),              # shorter than the sink
    (2, 8, 64, 2, 4, 60, 64),             # exactly sink + window
    (2, 8, 64, 2, 4, 60, 65),             # the first eviction
    (2, 8, 64, 2, 4, 60, 513),
    (4, 28, 128, 3, 16, 112, 300),
    (4, 28, 128, 2, 16, 112, 129),
    (8, 32, 128, 2, 16, 112, 1000),
    (1, 8, 128, 1, 0, 5, 777),            # no sink
    (2, 4, 128, 2, 100, 200, 1500),       # sink longer than a tile, window over four tiles
    (2, 16, 64, 1, 64, 64, 4097),         # sink and window of exactly one tile
    (8, 32, 128, 4, 128, 256, 3000),      # the paper's training setting (128 sink + 256 local)
    (4, 16, 128, 16, 16, 64, 9000),       # many items per unit: split merges on both kinds of unit
]


@pytest.mark.parametrize("Hkv,Hq,D,B,S,W,n", SHAPES)
def test_mixed_attention_matches_oracle(rl, hz, cuda_device, Hkv, Hq, D, B, S, W, n):
    mask = np.ones(Hkv, np.uint8)
    cache = hz.Cache(1, Hkv, Hq, D, B, n + 3, mask, S, W, device=cuda_device)
    oracle = Oracle(1, Hkv, Hq, D, B, n + 3, mask, S, W, threads=8)
    K, V = rand_bf16((n, B, Hkv, D), 100 + n), rand_bf16((n, B, Hkv, D), 200 + n)
    feed(cache, oracle, 0, K, V, bulk=True)
    q = rand_bf16((B, Hq, D), 300 + n)
    a_cpu, a_dev = gates(Hkv, 400 + n, cuda_device)
    out = cache.decode_mixed(0, q.to(cuda_device), a_dev)
    check_out(out.cpu().numpy(), oracle.decode_mixed(0, q, a_cpu.numpy()))
    assert cache.status() == 0
    # the same call again: the same bits (two addends on zero commute)
    assert torch.equal(out, cache.decode_mixed(0, q.to(cuda_device), a_dev))
    # the ordinary call is not disturbed by the mixed one, and the gates' ends reproduce it
    plain = cache.decode(0, q.to(cuda_device))
    check_out(plain.cpu().numpy(), oracle.decode(0, q))
    ones = torch.ones(Hkv, dtype=torch.float32, device=cuda_device)
    check_out(cache.decode_mixed(0, q.to(cuda_device), ones).cpu().numpy(), oracle.decode(0, q))
    check_state(cache, oracle)
    cache.close()


def test_mixed_attention_over_a_decode_loop(rl, hz, cuda_device):
    """Append and attend token by token across the first eviction and several tile boundaries."""
    Hkv, Hq, D, B, S, W = 2, 8, 128, 2, 5, 70
    mask = np.ones(Hkv, np.uint8)
    cache = hz.Cache(1, Hkv, Hq, D, B, 400, mask, S, W, device=cuda_device)
    oracle = Oracle(1, Hkv, Hq, D, B, 400, mask, S, W, threads=8)
    a_cpu, a_dev = gates(Hkv, 7, cuda_device)
    a_cpu[:] = torch.tensor([0.35, 0.8])
    a_dev.copy_(a_cpu)
    K, V = rand_bf16((330, B, Hkv, D), 11), rand_bf16((330, B, Hkv, D), 12)
    feed(cache, oracle, 0, K[:60], V[:60], bulk=True)
    for t in range(60, 330):
        feed(cache, oracle, 0, K[t:t + 1], V[t:t + 1], bulk=False)
        if t % 7 and t not in (74, 75, 76, 127, 128, 129, 191, 192, 193):
            continue
        q = rand_bf16((B, Hq, D), 1000 + t)
        check_out(cache.decode_mixed(0, q.to(cuda_device), a_dev).cpu().numpy(),
                  oracle.decode_mixed(0, q, a_cpu.numpy()))
    assert cache.status() == 0
    cache.close()


def test_mixed_attention_argument_checks(rl, hz, cuda_device):
    Hkv, Hq, D, B = 2, 8, 64, 1
    q = rand_bf16((B, Hq, D), 1).to(cuda_device)
    out = torch.full((B, Hq, D), 5.0, dtype=torch.float32, device=cuda_device)
    alpha = torch.full((Hkv,), 0.5, dtype=torch.float32, device=cuda_device)
    cache = hz.Cache(2, Hkv, Hq, D, B, 64, [1, 1, 1, 0], 4, 12, device=cuda_device)
    with pytest.raises(rl.RlkvError) as e:                 # nothing cached yet
        rl.rlkv_decode_mixed_attention(cache.handle, 0, q, alpha, out)
    assert e.value.code == rl.RLKV_EEMPTY
    k = rand_bf16((B, Hkv, D), 2).to(cuda_device)
    cache.append(0, k, k)
    cache.append(1, k, k)
    with pytest.raises(rl.RlkvError) as e:                 # layer 1 holds a compressed head
        rl.rlkv_decode_mixed_attention(cache.handle, 1, q, alpha, out)
    assert e.value.code == rl.RLKV_EINVAL
    with pytest.raises(rl.RlkvError) as e:
        rl.rlkv_decode_mixed_attention(cache.handle, 2, q, alpha, out)
    assert e.value.code == rl.RLKV_EINVAL
    torch.cuda.synchronize()
    assert (out == 5.0).all()                              # refused calls touch nothing
    rl.rlkv_decode_mixed_attention(cache.handle, 0, q, alpha, out)
    torch.cuda.synchronize()
    # one token: softmax over one row is that row of V, whatever the gate
    np.testing.assert_allclose(out.cpu().numpy()[0, :4], np.tile(k[0, 0].float().cpu().numpy(), (4, 1)), atol=1e-6)
    cache.close()


@pytest.mark.parametrize("name,layers", [("llama8b", 3), ("qwen7b", 2)])
def test_mixed_attention_full_size_sampled_units(rl, hz, cuda_device, name, layers):
    """The benchmark's shapes (every head full, a few layers of them) with the launch the benchmark's
    side measurement times: sampled (layer, batch row, KV head) units against the oracle, which
    regenerates the unit's K/V history from the addressable generator."""
    w = synth.WORKLOADS[name].with_(layers=layers, frac_compressed=0.0)
    n = w.context + 1
    mask = np.ones(layers * w.kv_heads, np.uint8)
    cache = hz.Cache(layers, w.kv_heads, w.q_heads, w.head_dim, w.batch, n + 8, mask, w.sink, w.window,
                     device=cuda_device)
    hz.fill_cache(cache, w, n)
    g = torch.Generator().manual_seed(5)
    alpha = torch.rand((layers, w.kv_heads), generator=g, dtype=torch.float32)
    a_dev = alpha.to(cuda_device)
    q = hz.step_inputs(w, n - 1, cuda_device)[2]
    outs = [cache.decode_mixed(l, q[l], a_dev[l]) for l in range(layers)]
    torch.cuda.synchronize()
    assert cache.status() == 0
    q = q.cpu()
    rng = np.random.default_rng(77)
    G = w.group
    for _ in range(6):
        layer, b, h = int(rng.integers(layers)), int(rng.integers(w.batch)), int(rng.integers(w.kv_heads))
        o = Oracle(1, 1, G, w.head_dim, 1, n, [1], w.sink, w.window)
        K = synth.unit_rows(w.seed, synth.STREAM_K, layer, 0, n, w.batch, w.kv_heads, w.head_dim, b, h)
        V = synth.unit_rows(w.seed, synth.STREAM_V, layer, 0, n, w.batch, w.kv_heads, w.head_dim, b, h)
        kb, vb = K.view(torch.int16).numpy().view(np.uint16), V.view(torch.int16).numpy().view(np.uint16)
        for t in range(n):
            o.append(0, kb[t], vb[t])
        want = o.decode_mixed(0, q[layer, b, h * G:(h + 1) * G].contiguous(), [float(alpha[layer, h])])[0]
        check_out(outs[layer][b, h * G:(h + 1) * G].cpu().numpy(), want)
    cache.close()
    torch.cuda.empty_cache()
