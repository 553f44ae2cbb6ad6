"""GPU parity of the lock-step cache held in 8 bits (rlkv_cache_create_fp8) against the quantising
oracle: the codes in the cache equal the oracle's bit for bit, outputs are within the bounds of the
other parity tests of the oracle's attention over the dequantised rows.  The handle is used through
the ordinary rlkv_* calls only.
"""
import numpy as np
import pytest
import torch

from oracle.rlkv_oracle import Oracle
from test_gpu_parity import check_out, rand_bf16

pytestmark = pytest.mark.gpu

D = 128


@pytest.fixture(scope="module")
def rl(cuda_device):
    import paper_2510_08525_b200.binding as binding
    return binding


def scales(layers, Hkv, seed):
    rng = np.random.default_rng(seed)
    ks = rng.uniform(0.008, 0.05, size=layers * Hkv).astype(np.float32)   # N(0,1) inputs reach about 4.5: some saturate
    vs = rng.uniform(0.02, 1.5, size=layers * Hkv).astype(np.float32)
    return ks, vs


def check_state(rl, handle, oracle, layers, Hkv, B, n, max_len, mask, cap):
    for layer in range(layers):
        assert rl.rlkv_length(handle, layer) == oracle.length(layer) == n[layer]
        for b in range(B):
            for h in range(Hkv):
                gk, gv, gt = rl.rlkv_debug_export_head(handle, layer, b, h, max_len if mask[layer * Hkv + h] else cap, D)
                ok, ov, ot = oracle.export_head(layer, b, h)
                np.testing.assert_array_equal(gt, ot)
                np.testing.assert_array_equal(gk, ok)       # rows that hold no token are zero on both sides
                np.testing.assert_array_equal(gv, ov)


SHAPES = [
    # layers, Hkv, Hq, B, S, W, mask, prompt, tokens after it
    (1, 2, 8, 3, 4, 60, "10", 200, 3),
    (2, 4, 16, 5, 16, 112, "1011" "0110", 700, 2),
    (3, 8, 32, 2, 16, 112, "11011011" "00000000" "11111111", 1300, 2),
    (1, 1, 8, 1, 0, 5, "0", 1, 70),
    (2, 2, 4, 16, 16, 48, "1101", 64, 1),
]


@pytest.mark.parametrize("layers,Hkv,Hq,B,S,W,mask,prompt,more", SHAPES)
def test_fp8_cache_matches_the_quantising_oracle(rl, cuda_device, layers, Hkv, Hq, B, S, W, mask, prompt, more):
    mask = [int(c) for c in mask]
    max_len = prompt + more + 9
    ks, vs = scales(layers, Hkv, 23)
    handle = rl.rlkv_cache_create_fp8(layers, Hkv, Hq, D, B, max_len, mask, S, W, ks, vs)
    n = [0] * layers
    try:
        for cycle in range(2):                              # the second cycle runs after rlkv_cache_reset
            oracle = Oracle(layers, Hkv, Hq, D, B, max_len, mask, S, W, threads=8)
            oracle.set_fp8(ks, vs)
            for layer in range(layers):                     # the prompt: one call, all batch rows
                K, V = rand_bf16((prompt, B, Hkv, D), 100 + 7 * layer + cycle), rand_bf16((prompt, B, Hkv, D), 200 + 7 * layer + cycle)
                rl.rlkv_prefill(handle, layer, K.to(cuda_device), V.to(cuda_device), prompt)
                for t in range(prompt):
                    assert oracle.append(layer, K[t], V[t]) == 0
                n[layer] += prompt
            for t in range(more):                           # token by token, one layer at a time
                for layer in range(layers):
                    k, v = rand_bf16((B, Hkv, D), 300 + 11 * t + layer), rand_bf16((B, Hkv, D), 400 + 11 * t + layer)
                    rl.rlkv_append(handle, layer, k.to(cuda_device), v.to(cuda_device))
                    assert oracle.append(layer, k, v) == 0
                    n[layer] += 1
                    q = rand_bf16((B, Hq, D), 500 + 11 * t + layer)
                    out = torch.empty((B, Hq, D), dtype=torch.float32, device=cuda_device)
                    rl.rlkv_decode_attention(handle, layer, q.to(cuda_device), out)
                    check_out(out.cpu().numpy(), oracle.decode(layer, q))
            check_state(rl, handle, oracle, layers, Hkv, B, n, max_len, mask, S + W)
            n_full = sum(mask[:Hkv])
            want = B * (n_full * n[0] + (Hkv - n_full) * min(n[0], S + W)) * 2 * D
            assert rl.rlkv_step_bytes(handle, 0) == want

            # whole steps: device arrays, then host arrays, in both step modes
            for step, (mode, host) in enumerate([(0, False), (1, False), (0, True)]):
                rl.rlkv_set_step_mode(handle, mode)
                k, v = rand_bf16((layers, B, Hkv, D), 600 + step), rand_bf16((layers, B, Hkv, D), 700 + step)
                q = rand_bf16((layers, B, Hq, D), 800 + step)
                if host:
                    out = torch.empty((layers, B, Hq, D), dtype=torch.float32).pin_memory()
                    rl.rlkv_step_host(handle, k.pin_memory(), v.pin_memory(), q.pin_memory(), out)
                    torch.cuda.synchronize()
                else:
                    out = torch.empty((layers, B, Hq, D), dtype=torch.float32, device=cuda_device)
                    rl.rlkv_step(handle, k.to(cuda_device), v.to(cuda_device), q.to(cuda_device), out)
                got = out.cpu().numpy()
                for layer in range(layers):
                    assert oracle.append(layer, k[layer], v[layer]) == 0
                    n[layer] += 1
                    check_out(got[layer], oracle.decode(layer, q[layer]))
            rl.rlkv_set_step_mode(handle, 0)
            check_state(rl, handle, oracle, layers, Hkv, B, n, max_len, mask, S + W)
            assert rl.rlkv_kernel_status(handle) == 0
            oracle.close()
            if cycle == 0:
                rl.rlkv_cache_reset(handle)
                n = [0] * layers
    finally:
        rl.rlkv_cache_destroy(handle)


def test_fp8_cache_limits_and_calls_it_does_not_serve(rl, cuda_device):
    layers, Hkv, Hq, B, S, W = 2, 2, 8, 2, 4, 12
    mask = [1, 0, 1, 1]
    ks, vs = scales(layers, Hkv, 5)
    ok = dict(layers=layers, kv_heads=Hkv, q_heads=Hq, head_dim=D, batch=B, max_len=70, head_is_full=mask, sink=S, window=W)
    for bad in (dict(head_dim=64), dict(batch=0), dict(max_len=0)):
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_cache_create_fp8(**{**ok, **bad}, k_scale=ks, v_scale=vs)
        assert e.value.code == rl.RLKV_EINVAL
    with pytest.raises(rl.RlkvError) as e:
        rl.rlkv_cache_create_fp8(**ok, k_scale=[0.0] * 4, v_scale=vs)
    assert e.value.code == rl.RLKV_EINVAL
    # half the bytes per token: a long cache costs less than its 16-bit counterpart
    long_ = {**ok, "max_len": 64 * 400}
    assert rl.rlkv_cache_size_fp8(**long_) < 0.6 * rl.rlkv_cache_size(**long_)

    # in a buffer of the caller
    need = rl.rlkv_cache_size_fp8(**ok)
    buf = torch.empty(need + 1024, dtype=torch.uint8, device=cuda_device)
    base = (buf.data_ptr() + 1023) // 1024 * 1024
    with pytest.raises(rl.RlkvError) as e:
        rl.rlkv_cache_create_fp8(**ok, k_scale=ks, v_scale=vs, device_buf=base, device_buf_bytes=need - 1)
    assert e.value.code == rl.RLKV_ENOMEM
    handle = rl.rlkv_cache_create_fp8(**ok, k_scale=ks, v_scale=vs, device_buf=base, device_buf_bytes=need)
    oracle = Oracle(layers, Hkv, Hq, D, B, 70, mask, S, W, threads=2)
    oracle.set_fp8(ks, vs)
    try:
        q = rand_bf16((B, Hq, D), 1).to(cuda_device)
        out = torch.empty((B, Hq, D), dtype=torch.float32, device=cuda_device)
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_decode_attention(handle, 0, q, out)
        assert e.value.code == rl.RLKV_EEMPTY
        K, V = rand_bf16((70, B, Hkv, D), 2), rand_bf16((70, B, Hkv, D), 3)
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_prefill(handle, 0, K.to(cuda_device), V.to(cuda_device), 71)
        assert e.value.code == rl.RLKV_EFULL
        assert rl.rlkv_length(handle, 0) == 0
        for layer in range(layers):
            rl.rlkv_prefill(handle, layer, K.to(cuda_device), V.to(cuda_device), 70)
            for t in range(70):
                assert oracle.append(layer, K[t], V[t]) == 0
        launches = rl.rlkv_launch_count(handle)
        assert launches >= 2
        k1 = rand_bf16((B, Hkv, D), 4).to(cuda_device)
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_append(handle, 1, k1, k1)
        assert e.value.code == rl.RLKV_EFULL
        kk = rand_bf16((layers, B, Hkv, D), 5).to(cuda_device)
        qq = rand_bf16((layers, B, Hq, D), 6).to(cuda_device)
        oo = torch.empty((layers, B, Hq, D), dtype=torch.float32, device=cuda_device)
        with pytest.raises(rl.RlkvError) as e:
            rl.rlkv_step(handle, kk, kk, qq, oo)
        assert e.value.code == rl.RLKV_EFULL
        assert rl.rlkv_launch_count(handle) == launches     # the refused calls launched nothing
        for layer in range(layers):
            rl.rlkv_decode_attention(handle, layer, q, out)
            check_out(out.cpu().numpy(), oracle.decode(layer, q.cpu()))
        # bf16 results
        rl.rlkv_set_output_bf16(handle, 1)
        out16 = torch.empty((B, Hq, D), dtype=torch.bfloat16, device=cuda_device)
        rl.rlkv_decode_attention(handle, 1, q, out16)
        want = oracle.decode(1, q.cpu())
        assert np.abs(out16.float().cpu().numpy() - want).max() <= 1e-2 + np.abs(want).max() / 128
        rl.rlkv_set_output_bf16(handle, 0)
        # calls this kind of handle does not serve
        alpha = torch.full((Hkv,), 0.5, dtype=torch.float32, device=cuda_device)
        for call in (lambda: rl.rlkv_set_decode_config(handle, 0, 0, 0, 8),
                     lambda: rl.rlkv_decode_attention_static_scratch(handle, 0, q, out),
                     lambda: rl.rlkv_decode_attention_overlapped(handle, 0, q, out),
                     lambda: rl.rlkv_append_overlapped(handle, 0, k1, k1),
                     lambda: rl.rlkv_layer_step_overlapped(handle, 0, k1, k1, q, out),
                     lambda: rl.rlkv_decode_mixed_attention(handle, 1, q, alpha, out)):
            with pytest.raises(rl.RlkvError) as e:
                call()
            assert e.value.code == rl.RLKV_EINVAL
        assert rl.rlkv_kernel_status(handle) == 0
    finally:
        rl.rlkv_cache_destroy(handle)
