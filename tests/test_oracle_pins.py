"""Pins for the CPU oracle: each test checks it against something other than itself.

The oracle is the plain definition of decode attention over a head-mixed KV cache
(Section 3.3 last paragraph; Section 4.3; Appendix B of the paper).  The paper prints
no numeric attention values, so the pins are: a library routine (all-full == causal
attention's last row), reductions, brute force with an explicit mask written here in
numpy, ring-buffer invariants, closed forms, planted needles, and the paper's printed
"theoretical speedup" column for the retained-token count.
"""
import itertools
import os

import numpy as np
import pytest
import torch

import synth
from oracle.rlkv_oracle import Oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f32(x):
    """bf16 torch tensor -> float32 numpy."""
    return x.to(torch.float32).numpy()


def rand_bf16(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32).to(torch.bfloat16)


def fill(oracle, layer, K, V):
    """K, V: bf16 [n][B][Hkv][D] appended token by token."""
    for t in range(K.shape[0]):
        assert oracle.append(layer, K[t], V[t]) == 0


def brute_force(q, K, V, keep):
    """Masked softmax attention written from the definition, float64 numpy.

    q [D], K [n][D], V [n][D] float arrays, keep bool[n]."""
    q, K, V = q.astype(np.float64), K.astype(np.float64), V.astype(np.float64)
    s = K @ q / np.sqrt(q.shape[0])
    s = np.where(keep, s, -np.inf)
    p = np.exp(s - s[keep].max())
    p = np.where(keep, p, 0.0)
    return (p / p.sum()) @ V


# ---------------------------------------------------------------------------- I1
@pytest.mark.parametrize("acc", ["f32", "f64"])
@pytest.mark.parametrize("Hq,Hkv,D,B,n", [(8, 2, 64, 2, 97), (6, 6, 32, 1, 33), (28, 4, 128, 1, 70)])
def test_all_full_equals_library_causal_attention(acc, Hq, Hkv, D, B, n):
    """With every head full the method is ordinary causal attention; the decode step is its
    last row.  Compared against torch's scaled_dot_product_attention (is_causal=True)."""
    K = rand_bf16((n, B, Hkv, D), 1)
    V = rand_bf16((n, B, Hkv, D), 2)
    Q = rand_bf16((n, B, Hq, D), 3)          # queries for every position; the last one is the decode
    o = Oracle(1, Hkv, Hq, D, B, n, np.ones(Hkv, np.uint8), 4, 8, acc=acc)
    fill(o, 0, K, V)
    out = o.decode(0, Q[-1])
    G = Hq // Hkv
    q4 = Q.permute(1, 2, 0, 3).to(torch.float64)                                  # [B][Hq][n][D]
    k4 = K.permute(1, 2, 0, 3).to(torch.float64).repeat_interleave(G, dim=1)      # head j reads j//G
    v4 = V.permute(1, 2, 0, 3).to(torch.float64).repeat_interleave(G, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(q4, k4, v4, is_causal=True)[:, :, -1, :]
    tol = 2e-5 if acc == "f32" else 2e-7      # the output array itself is float32
    np.testing.assert_allclose(out, ref.numpy(), atol=tol, rtol=0)


# ---------------------------------------------------------------------------- I2
@pytest.mark.parametrize("S,W,n", [(4, 60, 64), (4, 60, 10), (0, 50, 50), (16, 112, 100), (3, 5, 8)])
def test_compressed_with_budget_at_least_n_equals_full(S, W, n):
    Hq, Hkv, D, B = 4, 2, 32, 2
    K, V, q = rand_bf16((n, B, Hkv, D), 4), rand_bf16((n, B, Hkv, D), 5), rand_bf16((B, Hq, D), 6)
    a = Oracle(1, Hkv, Hq, D, B, n, [1, 1], S, W)
    b = Oracle(1, Hkv, Hq, D, B, n, [0, 0], S, W)
    fill(a, 0, K, V)
    fill(b, 0, K, V)
    np.testing.assert_array_equal(a.decode(0, q), b.decode(0, q))


# ---------------------------------------------------------------------------- I3
def test_compressed_head_equals_bruteforce_mask_exhaustive():
    """keep[t] = (t < S) or (t >= n - W), for every small (S, W, n)."""
    D, Hq, Hkv = 8, 4, 2
    nmax = 24
    K, V = rand_bf16((nmax, 1, Hkv, D), 7), rand_bf16((nmax, 1, Hkv, D), 8)
    checked = 0
    for S, W in itertools.product([0, 1, 2, 5], [1, 2, 3, 7]):
        o = Oracle(1, Hkv, Hq, D, 1, nmax, [1, 0], S, W, acc="f64")
        for n in range(1, nmax + 1):
            o.append(0, K[n - 1], V[n - 1])
            q = rand_bf16((1, Hq, D), 100 + n)
            out = o.decode(0, q)
            t = np.arange(n)
            for j in range(Hq):
                h = j // (Hq // Hkv)
                keep = np.ones(n, bool) if h == 0 else ((t < S) | (t >= n - W))
                ref = brute_force(f32(q[0, j]), f32(K[:n, 0, h]), f32(V[:n, 0, h]), keep)
                np.testing.assert_allclose(out[0, j], ref, atol=1e-6, rtol=0)
                checked += 1
    assert checked == 16 * nmax * Hq


def test_current_token_is_inside_the_window():
    """W = 1, S = 0: the head sees only the token appended in this very step."""
    D = 8
    K, V = rand_bf16((9, 1, 1, D), 9), rand_bf16((9, 1, 1, D), 10)
    o = Oracle(1, 1, 1, D, 1, 9, [0], 0, 1)
    for t in range(9):
        o.append(0, K[t], V[t])
        out = o.decode(0, rand_bf16((1, 1, D), t))
        np.testing.assert_allclose(out[0, 0], f32(V[t, 0, 0]), atol=1e-6)


# ---------------------------------------------------------------------------- I4
@pytest.mark.parametrize("S,W", [(4, 60), (0, 7), (16, 240), (3, 1)])
def test_ring_holds_sinks_and_last_window_tokens(S, W):
    D, B, Hkv = 16, 2, 2
    steps = max(5 * W + S + 3, 40)
    K, V = rand_bf16((steps, B, Hkv, D), 11), rand_bf16((steps, B, Hkv, D), 12)
    o = Oracle(1, Hkv, Hkv, D, B, steps, [0, 1], S, W)
    kb, vb = K.view(torch.int16).numpy().view(np.uint16), V.view(torch.int16).numpy().view(np.uint16)
    for t in range(steps):
        assert o.append(0, K[t], V[t]) == 0
        n = t + 1
        if n in (1, S, S + 1, S + W, S + W + 1) or n % 17 == 0 or n == steps:
            for b in range(B):
                k, v, tok = o.export_head(0, b, 0)
                want = set(range(min(S, n))) | set(range(max(S, n - W), n))
                assert set(tok[tok >= 0].tolist()) == want
                assert len(tok) == S + W
                for s, tt in enumerate(tok):
                    if tt >= 0:
                        assert s == (tt if tt < S else S + (tt - S) % W)
                        np.testing.assert_array_equal(k[s], kb[tt, b, 0])
                        np.testing.assert_array_equal(v[s], vb[tt, b, 0])
                    else:
                        assert not k[s].any() and not v[s].any()
                kf, vf, tokf = o.export_head(0, b, 1)
                np.testing.assert_array_equal(kf[:n], kb[:n, b, 1])
                np.testing.assert_array_equal(vf[:n], vb[:n, b, 1])
                assert tokf[:n].tolist() == list(range(n)) and (tokf[n:] == -1).all()
    assert o.append(0, K[0], V[0]) == -1 and o.length(0) == steps   # full: state unchanged


# ---------------------------------------------------------------------------- I5
@pytest.mark.parametrize("mask", [[1, 1], [0, 0], [1, 0]])
def test_closed_forms(mask):
    D, B, Hq, Hkv, n, S, W = 16, 2, 4, 2, 50, 3, 9
    K, V, q = rand_bf16((n, B, Hkv, D), 13), rand_bf16((n, B, Hkv, D), 14), rand_bf16((B, Hq, D), 15)
    t = np.arange(n)
    keep_c = (t < S) | (t >= n - W)
    # (a) all V rows equal -> out equals that row, whatever the scores
    vrow = rand_bf16((D,), 16)
    o = Oracle(1, Hkv, Hq, D, B, n, mask, S, W)
    fill(o, 0, K, vrow.expand(n, B, Hkv, D).contiguous())
    np.testing.assert_allclose(o.decode(0, q), np.broadcast_to(f32(vrow), (B, Hq, D)), atol=2e-6)
    # (b) K = 0 -> arithmetic mean of the retained V rows; (c) q = 0 -> the same mean
    for kk, qq in ((torch.zeros_like(K), q), (K, torch.zeros_like(q))):
        o = Oracle(1, Hkv, Hq, D, B, n, mask, S, W)
        fill(o, 0, kk, V)
        out = o.decode(0, qq)
        for j in range(Hq):
            h = j // 2
            keep = np.ones(n, bool) if mask[h] else keep_c
            want = f32(V[:, :, h]).astype(np.float64)[keep].mean(axis=0)          # [B][D]
            np.testing.assert_allclose(out[:, j], want, atol=2e-6)


# ---------------------------------------------------------------------------- I6
def test_planted_needle_visibility():
    """A token whose key is strongly aligned with q dominates iff the head retains it."""
    D, n, S, W = 32, 200, 4, 20
    base_K, base_V = rand_bf16((n, 1, 2, D), 17), rand_bf16((n, 1, 2, D), 18)
    q = rand_bf16((1, 2, D), 19)
    marker = torch.full((D,), 7.0, dtype=torch.bfloat16)
    for t_star in [0, S - 1, S, n - W - 1, n - W, n - 1, 63, 64, 65, 127, 128]:
        K, V = base_K.clone(), base_V.clone()
        for h in range(2):
            qq = q[0, h].to(torch.float32)
            K[t_star, 0, h] = (qq / qq.norm() * 60.0).to(torch.bfloat16)   # score ~ 60*|q|/sqrt(D) >> others
            V[t_star, 0, h] = marker
        o = Oracle(1, 2, 2, D, 1, n, [1, 0], S, W)
        fill(o, 0, K, V)
        out = o.decode(0, q)
        assert np.abs(out[0, 0] - 7.0).max() < 1e-3                       # full head always sees it
        visible = t_star < S or t_star >= n - W
        if visible:
            assert np.abs(out[0, 1] - 7.0).max() < 1e-3
        else:
            assert np.abs(out[0, 1]).max() < 4.0                           # needle evicted: nowhere near 7


# ---------------------------------------------------------------------------- I7
def test_group_and_batch_symmetries():
    D, B, Hq, Hkv, n = 16, 3, 6, 2, 40
    K, V = rand_bf16((n, B, Hkv, D), 20), rand_bf16((n, B, Hkv, D), 21)
    qh = rand_bf16((B, Hkv, 1, D), 22)
    q = qh.expand(B, Hkv, Hq // Hkv, D).reshape(B, Hq, D).contiguous()     # same q within a group
    o = Oracle(1, Hkv, Hq, D, B, n, [1, 0], 2, 6)
    fill(o, 0, K, V)
    out = o.decode(0, q)
    for h in range(Hkv):
        for g in range(1, Hq // Hkv):
            np.testing.assert_array_equal(out[:, h * 3], out[:, h * 3 + g])
    # distinct q per head must give distinct outputs (catches a collapsed head index)
    q2 = rand_bf16((B, Hq, D), 23)
    out2 = o.decode(0, q2)
    assert np.abs(out2[:, 0] - out2[:, 1]).max() > 1e-3
    perm = [2, 0, 1]
    o2 = Oracle(1, Hkv, Hq, D, B, n, [1, 0], 2, 6)
    fill(o2, 0, K[:, perm].contiguous(), V[:, perm].contiguous())
    np.testing.assert_array_equal(o2.decode(0, q2[perm].contiguous()), out2[perm])


# ---------------------------------------------------------------------------- I8
def test_evicted_tokens_do_not_matter():
    D, n, S, W = 16, 90, 3, 10
    K, V = rand_bf16((n, 1, 1, D), 24), rand_bf16((n, 1, 1, D), 25)
    K2, V2 = K.clone(), V.clone()
    K2[S:n - W] = rand_bf16((n - W - S, 1, 1, D), 26)
    V2[S:n - W] = rand_bf16((n - W - S, 1, 1, D), 27)
    q = rand_bf16((1, 1, D), 28)
    a, b = Oracle(1, 1, 1, D, 1, n, [0], S, W), Oracle(1, 1, 1, D, 1, n, [0], S, W)
    fill(a, 0, K, V)
    fill(b, 0, K2, V2)
    np.testing.assert_array_equal(a.decode(0, q), b.decode(0, q))
    for x, y in zip(a.export_head(0, 0, 0), b.export_head(0, 0, 0)):
        np.testing.assert_array_equal(x, y)


# ---------------------------------------------------------------------------- cost model
def test_retained_tokens_reproduce_printed_theoretical_speedups():
    """Table 3 prints 1/((1-s) + s*W/L); with W = 16 + 64 and L = 3019 (the Math500 mean length
    the paper quotes) the oracle's retained-token counts reproduce the printed column."""
    rows = [tuple(map(float, ln.split())) for ln in open(os.path.join(GOLDEN, "table3_theoretical.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 4
    L, S, W, heads = 3019, 16, 64, 10
    z = torch.zeros((1, heads, 1), dtype=torch.bfloat16)
    for s, printed in rows:
        n_comp = int(round(s * heads))
        mask = [1] * (heads - n_comp) + [0] * n_comp
        o = Oracle(1, heads, heads, 1, 1, L, mask, S, W)
        for _ in range(L):
            o.append(0, z, z)
        kept = sum(o.retained(0, h) for h in range(heads))
        assert o.retained(0, heads - 1) == (S + W if n_comp else L)
        speedup = heads * L / kept
        assert abs(round(speedup, 2) - printed) < 1e-9, (s, speedup, printed)


# ---------------------------------------------------------------------------- self-check
def test_f32_build_close_to_f64_build():
    D, B, Hq, Hkv, n = 128, 1, 8, 2, 3000
    K, V, q = rand_bf16((n, B, Hkv, D), 29), rand_bf16((n, B, Hkv, D), 30), rand_bf16((B, Hq, D), 31)
    a = Oracle(1, Hkv, Hq, D, B, n, [1, 0], 16, 112, acc="f32")
    b = Oracle(1, Hkv, Hq, D, B, n, [1, 0], 16, 112, acc="f64")
    fill(a, 0, K, V)
    fill(b, 0, K, V)
    assert np.abs(a.decode(0, q) - b.decode(0, q)).max() < 2e-6


def test_threads_do_not_change_results():
    D, B, Hq, Hkv, n = 32, 3, 4, 2, 77
    K, V, q = rand_bf16((n, B, Hkv, D), 32), rand_bf16((n, B, Hkv, D), 33), rand_bf16((B, Hq, D), 34)
    o = Oracle(1, Hkv, Hq, D, B, n, [1, 0], 4, 9)
    fill(o, 0, K, V)
    one = o.decode(0, q)
    o.set_threads(4)
    np.testing.assert_array_equal(one, o.decode(0, q))


def test_layers_keep_separate_lengths_and_masks():
    D = 8
    o = Oracle(2, 2, 2, D, 1, 10, [1, 0, 0, 1], 1, 2)
    K, V = rand_bf16((6, 1, 2, D), 35), rand_bf16((6, 1, 2, D), 36)
    for t in range(6):
        o.append(0, K[t], V[t])
    for t in range(3):
        o.append(1, K[t], V[t])
    assert (o.length(0), o.length(1)) == (6, 3)
    assert [o.retained(0, 0), o.retained(0, 1), o.retained(1, 0), o.retained(1, 1)] == [6, 3, 3, 3]
    with pytest.raises(RuntimeError):
        Oracle(1, 1, 1, D, 1, 4, [1], 0, 1).decode(0, rand_bf16((1, 1, D), 1))   # empty layer


# ---------------------------------------------------------------------------- mixed attention, Eq. 1
def mask_matrices(n, S, W):
    """M_causal and M_local of Section 3.1 as boolean [n][n] matrices (row = query position):
    causal = every earlier token and the query's own; local = causal AND (one of the first S tokens
    OR one of the W most recent, the query's own included)."""
    i, j = np.arange(n)[:, None], np.arange(n)[None, :]
    causal = j <= i
    local = causal & ((j < S) | (j > i - W))
    return causal, local


@pytest.mark.parametrize("acc", ["f32", "f64"])
@pytest.mark.parametrize("S,W,n", [(4, 8, 40), (0, 5, 23), (3, 1, 17), (16, 64, 200)])
def test_mixed_equals_masked_softmax_with_mask_matrices(acc, S, W, n):
    """Eq. 1 computed for EVERY position with explicit mask matrices in float64 numpy; the decode
    step is the last row."""
    Hq, Hkv, D, B = 6, 2, 16, 2
    G = Hq // Hkv
    K, V, Q = rand_bf16((n, B, Hkv, D), 71), rand_bf16((n, B, Hkv, D), 72), rand_bf16((n, B, Hq, D), 73)
    alpha = np.array([0.3, 0.85], np.float32)
    o = Oracle(1, Hkv, Hq, D, B, n, [1, 1], S, W, acc=acc)
    fill(o, 0, K, V)
    out = o.decode_mixed(0, Q[-1], alpha)
    causal, local = mask_matrices(n, S, W)
    for b in range(B):
        for j in range(Hq):
            h = j // G
            q2, k2, v2 = (f32(Q[:, b, j]).astype(np.float64), f32(K[:, b, h]).astype(np.float64),
                          f32(V[:, b, h]).astype(np.float64))
            s = q2 @ k2.T / np.sqrt(D)                               # [n][n]
            rows = []
            for m in (causal, local):
                sm = np.where(m, s, -np.inf)
                p = np.exp(sm - sm.max(axis=1, keepdims=True))
                rows.append(((p / p.sum(axis=1, keepdims=True)) @ v2)[-1])
            want = float(alpha[h]) * rows[0] + (1.0 - float(alpha[h])) * rows[1]
            np.testing.assert_allclose(out[b, j], want, atol=2e-5 if acc == "f32" else 3e-7, rtol=0)


def test_mixed_gate_one_is_full_attention_and_gate_zero_is_the_compressed_head():
    """alpha = 1 must give what a full head gives and alpha = 0 what a compressed head gives
    (Section 3.3: at inference the gate picks one branch) -- through rlkv_oracle_decode, whose own
    pins are above.  A swapped gate or a window off by one fails here."""
    Hq, Hkv, D, B, S, W, n = 8, 2, 32, 2, 4, 12, 61
    K, V, q = rand_bf16((n, B, Hkv, D), 74), rand_bf16((n, B, Hkv, D), 75), rand_bf16((B, Hq, D), 76)
    full = Oracle(1, Hkv, Hq, D, B, n, [1, 1], S, W)
    comp = Oracle(1, Hkv, Hq, D, B, n, [0, 0], S, W)
    fill(full, 0, K, V)
    fill(comp, 0, K, V)
    np.testing.assert_allclose(full.decode_mixed(0, q, [1.0, 1.0]), full.decode(0, q), atol=1e-6, rtol=0)
    np.testing.assert_allclose(full.decode_mixed(0, q, [0.0, 0.0]), comp.decode(0, q), atol=1e-6, rtol=0)
    mixed = full.decode_mixed(0, q, [1.0, 0.0])                     # head 0 full, head 1 local
    G = Hq // Hkv
    np.testing.assert_allclose(mixed[:, :G], full.decode(0, q)[:, :G], atol=1e-6, rtol=0)
    np.testing.assert_allclose(mixed[:, G:], comp.decode(0, q)[:, G:], atol=1e-6, rtol=0)
    # the two branches differ here, so the checks above can tell them apart
    assert np.abs(full.decode(0, q) - comp.decode(0, q)).max() > 1e-2
    # in between: the straight line between the two branches, gate by gate
    a = np.array([0.25, 0.6], np.float32)
    want = np.repeat(a, G)[None, :, None] * full.decode(0, q) + np.repeat(1 - a, G)[None, :, None] * comp.decode(0, q)
    np.testing.assert_allclose(full.decode_mixed(0, q, a), want, atol=2e-6, rtol=0)


def test_mixed_short_sequence_does_not_depend_on_the_gate():
    """While n <= sink + window the local mask hides nothing, both branches agree and the gate
    drops out of Eq. 1."""
    Hq, Hkv, D, B, S, W = 4, 2, 32, 1, 4, 28
    for n in (1, 3, 4, 5, 32):
        K, V, q = rand_bf16((n, B, Hkv, D), 77), rand_bf16((n, B, Hkv, D), 78), rand_bf16((B, Hq, D), 79)
        o = Oracle(1, Hkv, Hq, D, B, 64, [1, 1], S, W)
        fill(o, 0, K, V)
        ref = o.decode(0, q)
        for a in ([0.0, 1.0], [0.5, 0.123]):
            np.testing.assert_allclose(o.decode_mixed(0, q, a), ref, atol=1e-6, rtol=0)


def test_mixed_planted_needle_is_seen_only_through_the_full_branch():
    """One token in the evicted middle carries a key aligned with the query and a marker value: the
    full branch returns (almost exactly) the marker, the local branch cannot see it, so the output
    is alpha * marker + (1 - alpha) * local."""
    Hq, Hkv, D, B, S, W, n = 2, 1, 32, 1, 2, 6, 50
    K, V = rand_bf16((n, B, Hkv, D), 80) * 0.1, rand_bf16((n, B, Hkv, D), 81)
    q = torch.zeros((B, Hq, D), dtype=torch.bfloat16)
    q[..., 0] = 16.0
    K[20, 0, 0, :] = 0
    K[20, 0, 0, 0] = 64.0                                     # score 16*64/sqrt(32) = 181 above the rest
    V[20, 0, 0, :] = 7.0
    o = Oracle(1, Hkv, Hq, D, B, n, [1], S, W)
    c = Oracle(1, Hkv, Hq, D, B, n, [0], S, W)
    fill(o, 0, K, V)
    fill(c, 0, K, V)
    local = c.decode(0, q)
    assert np.abs(local - 7.0).min() > 1.0
    out = o.decode_mixed(0, q, [0.75])
    np.testing.assert_allclose(out, 0.75 * 7.0 + 0.25 * local, atol=1e-5, rtol=0)


def test_mixed_refuses_compressed_heads_and_gates_outside_the_unit_interval():
    Hq, Hkv, D, B = 4, 2, 16, 1
    K, V, q = rand_bf16((9, B, Hkv, D), 82), rand_bf16((9, B, Hkv, D), 83), rand_bf16((B, Hq, D), 84)
    o = Oracle(1, Hkv, Hq, D, B, 16, [1, 0], 2, 3)
    fill(o, 0, K, V)
    with pytest.raises(RuntimeError, match="-5"):
        o.decode_mixed(0, q, [0.5, 0.5])
    o = Oracle(1, Hkv, Hq, D, B, 16, [1, 1], 2, 3)
    with pytest.raises(RuntimeError, match="-3"):
        o.decode_mixed(0, q, [0.5, 0.5])
    fill(o, 0, K, V)
    for bad in ([1.5, 0.5], [0.5, -0.1], [float("nan"), 0.5]):
        with pytest.raises(RuntimeError, match="-6"):
            o.decode_mixed(0, q, bad)


# ---------------------------------------------------------------------------- 8-bit K/V (E4M3)
def test_e4m3_values_of_all_codes_match_the_library_type():
    from oracle.rlkv_oracle import e4m3_value
    codes = torch.arange(256, dtype=torch.uint8)
    want = codes.view(torch.float8_e4m3fn).to(torch.float32).numpy()
    got = np.array([e4m3_value(int(c)) for c in codes], dtype=np.float32)
    assert np.isnan(got[[0x7f, 0xff]]).all() and np.isnan(want[[0x7f, 0xff]]).all()
    ok = ~np.isnan(want)
    np.testing.assert_array_equal(got[ok], want[ok])
    # what the format's definition fixes, written out: largest finite, smallest normal, smallest subnormal
    assert e4m3_value(0x7e) == 448.0 and e4m3_value(0x08) == 2.0 ** -6 and e4m3_value(0x01) == 2.0 ** -9
    assert e4m3_value(0x38) == 1.0 and e4m3_value(0xb8) == -1.0 and e4m3_value(0x80) == 0.0


def test_e4m3_encoder_matches_the_library_cast_on_every_code_midpoint_and_neighbour():
    """Every representable value, every midpoint between neighbours (the ties) and points just beside
    them, both signs, against torch's float32 -> float8_e4m3fn cast, which rounds to nearest even.
    Above 464 torch's cast gives NaN where this format's users saturate: there the reading (448) is
    checked as such."""
    from oracle.rlkv_oracle import e4m3_encode, e4m3_value
    vals = np.array([e4m3_value(c) for c in range(0x7f)], dtype=np.float64)
    pts = [vals, (vals[:-1] + vals[1:]) / 2]
    pts += [np.nextafter(p.astype(np.float32), np.float32(np.inf)).astype(np.float64) for p in list(pts)]
    pts += [np.nextafter(p.astype(np.float32), np.float32(-np.inf)).astype(np.float64) for p in pts[:2]]
    x = np.concatenate(pts + [np.array([449.0, 463.9, 464.0, 1e-12, 0.3, 0.7, 3.14159, 100.0, 447.9])])
    x = np.concatenate([x, -x]).astype(np.float32)
    x = x[np.abs(x) <= 464.0]
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([e4m3_encode(float(v)) for v in x], dtype=np.uint8)
    zero = (want & 0x7f) == 0                                  # +0 / -0: compare the magnitude only
    np.testing.assert_array_equal(got[~zero], want[~zero])
    assert ((got[zero] & 0x7f) == 0).all()
    for big in (464.1, 480.0, 1e6, 3e38):
        assert e4m3_encode(big) == 0x7e and e4m3_encode(-big) == 0xfe
    assert e4m3_encode(float("nan")) == 0x7f
    # decoding an encoded code gives the code back
    for c in list(range(0x7f)) + list(range(0x81, 0xff)):
        assert e4m3_encode(e4m3_value(c)) == c


def test_fp8_storage_equals_plain_attention_over_the_dequantised_rows():
    """With 8-bit storage the oracle must give exactly what the 16-bit oracle gives on rows that were
    quantised and dequantised beforehand with the library type (scales are powers of two, so that
    x_hat is a bf16 number) -- for a full head and for a compressed head's ring alike."""
    Hq, Hkv, D, B, S, W, n = 8, 2, 32, 2, 4, 12, 90
    K, V, q = rand_bf16((n, B, Hkv, D), 301), rand_bf16((n, B, Hkv, D), 302), rand_bf16((B, Hq, D), 303)
    ks, vs = np.array([0.5, 2.0], np.float32), np.array([0.25, 1.0], np.float32)
    a = Oracle(1, Hkv, Hq, D, B, n, [1, 0], S, W)
    a.set_fp8(ks, vs)
    fill(a, 0, K, V)

    def roundtrip(x, scale):      # e4m3 has 3 mantissa bits: value * 2^k is exact in bf16
        return ((x.float() / scale).to(torch.float8_e4m3fn).float() * scale).to(torch.bfloat16)

    K2, V2 = K.clone(), V.clone()
    for h in range(Hkv):
        K2[:, :, h], V2[:, :, h] = roundtrip(K[:, :, h], float(ks[h])), roundtrip(V[:, :, h], float(vs[h]))
    b = Oracle(1, Hkv, Hq, D, B, n, [1, 0], S, W)
    fill(b, 0, K2, V2)
    np.testing.assert_array_equal(a.decode(0, q), b.decode(0, q))
    # the stored entries are the codes: the full head's in token order, the ring's in slot order
    k_codes, v_codes, _ = a.export_head(0, 1, 0)
    want = (K[:, 1, 0].float() / 0.5).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    np.testing.assert_array_equal(k_codes[:n], want)
    ring_k, ring_v, tok = a.export_head(0, 1, 1)
    want = (V[tok, 1, 1].float() / 1.0).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    np.testing.assert_array_equal(ring_v, want)
    assert np.abs(a.decode(0, q) - Oracle_decode_plain(K, V, q, Hkv, Hq, D, B, n, S, W)).max() > 1e-4   # it does quantise
    with pytest.raises(RuntimeError, match="-7"):
        a.set_fp8(ks, vs)                                       # only while empty
    with pytest.raises(RuntimeError, match="-7"):
        Oracle(1, Hkv, Hq, D, B, n, [1, 0], S, W).set_fp8([0.0, 1.0], vs)


def Oracle_decode_plain(K, V, q, Hkv, Hq, D, B, n, S, W):
    o = Oracle(1, Hkv, Hq, D, B, n, [1, 0], S, W)
    fill(o, 0, K, V)
    return o.decode(0, q)
