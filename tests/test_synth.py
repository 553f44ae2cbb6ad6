"""The seeded input generator: addressable, device-independent, N(0,1)-like, right head counts."""
import numpy as np
import torch

import synth


def test_unit_rows_match_full_rows():
    full = synth.rows(5, synth.STREAM_K, 3, 10, 30, 2, 3, 16)
    assert full.dtype == torch.bfloat16 and full.shape == (20, 2, 3, 16)
    for b in range(2):
        for h in range(3):
            one = synth.unit_rows(5, synth.STREAM_K, 3, 10, 30, 2, 3, 16, b, h)
            assert torch.equal(one.view(torch.int16), full[:, b, h].contiguous().view(torch.int16))
    # token ranges compose
    a = synth.rows(5, synth.STREAM_K, 3, 10, 20, 2, 3, 16)
    assert torch.equal(a.view(torch.int16), full[:10].contiguous().view(torch.int16))


def test_streams_layers_seeds_differ():
    base = synth.rows(0, synth.STREAM_K, 0, 0, 8, 1, 2, 64).view(torch.int16)
    for other in (synth.rows(0, synth.STREAM_V, 0, 0, 8, 1, 2, 64),
                  synth.rows(0, synth.STREAM_K, 1, 0, 8, 1, 2, 64),
                  synth.rows(1, synth.STREAM_K, 0, 0, 8, 1, 2, 64)):
        assert (other.view(torch.int16) != base).float().mean() > 0.9


def test_values_look_standard_normal():
    x = synth.rows(7, synth.STREAM_V, 0, 0, 256, 4, 4, 64).to(torch.float64)
    assert abs(x.mean().item()) < 0.01 and abs(x.std().item() - 1.0) < 0.01
    assert torch.isfinite(x).all() and x.abs().max() < 6.0
    table = synth.normal_table()
    t = synth.bf16_bits_to_float(table.numpy())
    assert np.all(np.diff(t) >= 0) and abs(t[32768]) < 1e-4


def test_head_mask_counts_and_order():
    for name, want in (("llama8b", 51), ("qwen7b", 67), ("cot", 102)):
        w = synth.WORKLOADS[name]
        m = synth.head_mask(w.seed, w.layers, w.kv_heads, w.frac_compressed)
        assert m.shape == (w.layers * w.kv_heads,) and int((m == 0).sum()) == want
        u = synth.head_scores(w.seed, w.layers, w.kv_heads)
        assert u.min() >= 0 and u.max() < 1
        assert u[m == 0].max() <= u[m == 1].min()          # lowest scores are the compressed ones
    assert synth.head_mask(0, 4, 4, 0.0).all() and not synth.head_mask(0, 4, 4, 1.0).any()
