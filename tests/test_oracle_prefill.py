"""Pins for the oracle's prefill attention (Eq. 2 with the mask of Eq. 5).

Each test checks the oracle against something fixed by the paper or by
mathematics, not against the oracle itself."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import ag_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_all_keep_is_textbook_causal_attention():
    # Eq. 5 with AG = 1 everywhere is the lower-triangular mask.
    B, h, n, D = 2, 3, 37, 16
    Q, K, V = (_rand((B, h, n, D), s) for s in (1, 2, 3))
    flags = np.ones((B, h, n), dtype=np.uint8)
    O = orc.prefill_attention(Q, K, V, flags)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q), torch.from_numpy(K), torch.from_numpy(V), is_causal=True).numpy()
    assert np.max(np.abs(O - ref)) < 1e-12


def test_all_keep_triple_loop():
    n, D = 9, 4
    Q, K, V = (_rand((n, D), s) for s in (4, 5, 6))
    O = orc.prefill_head(Q, K, V, np.ones(n, dtype=np.uint8))
    for j in range(n):
        w = [math.exp(sum(Q[j, c] * K[t, c] for c in range(D)) / math.sqrt(D)) for t in range(j + 1)]
        z = sum(w)
        for c in range(D):
            assert abs(O[j, c] - sum(w[t] * V[t, c] for t in range(j + 1)) / z) < 1e-12


def test_all_evict_leaves_only_the_diagonal():
    # Sec. 3.3: the diagonal is always preserved, so with every token evicted
    # each query sees only itself and O[j] = V[j] exactly.
    B, h, n, D = 1, 2, 33, 8
    Q, K, V = (_rand((B, h, n, D), s) for s in (7, 8, 9))
    O = orc.prefill_attention(Q, K, V, np.zeros((B, h, n), dtype=np.uint8))
    assert np.array_equal(O, V)


def _visible_set(flags, j):
    return [t for t in range(j + 1) if t == j or flags[t] == 1]


def _attend_set(q, K, V, keys, scale):
    logits = [scale * float(np.dot(q, K[t])) for t in keys]
    m = max(logits)
    w = [math.exp(x - m) for x in logits]
    z = sum(w)
    return sum(wi * V[t] for wi, t in zip(w, keys)) / z


@pytest.mark.parametrize("n", [1, 2, 5, 7])
def test_brute_force_every_flag_pattern(n):
    D = 3
    Q, K, V = (_rand((n, D), 10 + n + s) for s in (0, 1, 2))
    scale = 1.0 / math.sqrt(D)
    for pattern in itertools.product([0, 1], repeat=n):
        f = np.asarray(pattern, dtype=np.uint8)
        O = orc.prefill_head(Q, K, V, f)
        for j in range(n):
            want = _attend_set(Q[j], K, V, _visible_set(pattern, j), scale)
            assert np.max(np.abs(O[j] - want)) < 1e-12, (pattern, j)


def test_golden_uniform_attention_example():
    rows = {}
    with open(os.path.join(GOLDEN, "uniform_attention_n4.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            rows[key] = np.asarray([float(v) for v in vals])
    flags = rows["flags"].astype(np.uint8)
    V = rows["V"].reshape(4, 2)
    want = rows["O"].reshape(4, 2)
    K = _rand((4, 2), 21)
    O = orc.prefill_head(np.zeros((4, 2)), K, V, flags)
    assert np.max(np.abs(O - want)) < 1e-13


def test_two_key_row_is_a_logistic_mixture():
    # Row 1 with token 0 retained: softmax over two logits = logistic of their difference.
    D = 5
    Q, K, V = (_rand((2, D), s) for s in (31, 32, 33))
    O = orc.prefill_head(Q, K, V, np.asarray([1, 1], dtype=np.uint8), scale=0.7)
    a0 = 1.0 / (1.0 + math.exp(-0.7 * float(np.dot(Q[1], K[0] - K[1]))))
    assert np.max(np.abs(O[1] - (a0 * V[0] + (1 - a0) * V[1]))) < 1e-13
    assert np.array_equal(O[0], V[0])


def test_mask_matrix_entries():
    f = np.asarray([1, 0, 0, 1, 1], dtype=np.uint8)
    M = orc.eviction_mask(f)
    for j in range(5):
        for t in range(5):
            want = 0 if j < t else (1 if j == t else int(f[t]))
            assert M[j, t] == want
    assert np.array_equal(orc.eviction_mask(f, rows=[3, 1]), M[[3, 1]])


def test_column_structure_and_locality():
    n, D = 24, 6
    Q, K, V = (_rand((n, D), s) for s in (41, 42, 43))
    f = (np.random.default_rng(44).random(n) < 0.5).astype(np.uint8)
    f[5], f[11] = 0, 1
    O = orc.prefill_head(Q, K, V, f)
    # an evicted token's K/V matter only to its own row
    K2, V2 = K.copy(), V.copy()
    K2[5] += 3.0
    V2[5] -= 2.0
    O2 = orc.prefill_head(Q, K2, V2, f)
    changed = np.where(np.any(O != O2, axis=1))[0]
    assert list(changed) == [5]
    # flipping a flag changes only strictly later rows
    f3 = f.copy()
    f3[11] = 0
    O3 = orc.prefill_head(Q, K, V, f3)
    assert np.array_equal(O3[:12], O[:12])
    assert np.all(np.any(O3[12:] != O[12:], axis=1))
    # convex combination of visible value rows
    for j in range(n):
        vis = _visible_set(f, j)
        assert np.all(O[j] <= V[vis].max(axis=0) + 1e-12)
        assert np.all(O[j] >= V[vis].min(axis=0) - 1e-12)


def test_rows_subset_and_scale():
    n, D = 19, 4
    Q, K, V = (_rand((n, D), s) for s in (51, 52, 53))
    f = (np.random.default_rng(54).random(n) < 0.4).astype(np.uint8)
    full = orc.prefill_head(Q, K, V, f, scale=0.3)
    sub = orc.prefill_head(Q, K, V, f, scale=0.3, rows=[18, 0, 7])
    assert np.max(np.abs(sub - full[[18, 0, 7]])) < 1e-14
    # scale = 0 -> uniform over the visible set
    uni = orc.prefill_head(Q, K, V, f, scale=0.0)
    for j in (0, 7, 18):
        assert np.max(np.abs(uni[j] - V[_visible_set(f, j)].mean(axis=0))) < 1e-13


def test_pins_catch_a_planted_mistake(monkeypatch):
    # Plant "flag indexed by the query instead of the key" in the oracle and
    # check that the brute-force pin notices.
    def wrong_mask(flags_i, rows=None, window=1):
        f = np.asarray(flags_i).astype(np.int64)
        n = f.shape[0]
        j = (np.arange(n) if rows is None else np.asarray(rows))[:, None]
        t = np.arange(n)[None, :]
        return np.where(j < t, 0, np.where(j == t, 1, f[j]))
    monkeypatch.setattr(orc, "eviction_mask", wrong_mask)
    n, D = 5, 3
    Q, K, V = (_rand((n, D), 60 + s) for s in (0, 1, 2))
    f = np.asarray([1, 0, 1, 0, 1], dtype=np.uint8)
    O = orc.prefill_head(Q, K, V, f)
    bad = False
    for j in range(n):
        want = _attend_set(Q[j], K, V, _visible_set(f, j), 1.0 / math.sqrt(D))
        bad |= np.max(np.abs(O[j] - want)) > 1e-9
    assert bad


# ---- grouped-query attention: query heads in groups share a key/value head and its flags

def test_grouped_query_prefill_and_decode_equal_shared_heads_written_out():
    """h = 6 query heads over h_kv = 2 key/value heads give exactly what ordinary multi-head
    attention gives when each key/value head (and its flags, and its cache slab) is written out
    once per query head of its group."""
    rng = np.random.default_rng(70)
    B, h, h_kv, n, D = 2, 6, 2, 9, 4
    Q = rng.standard_normal((B, h, n, D))
    K = rng.standard_normal((B, h_kv, n, D))
    V = rng.standard_normal((B, h_kv, n, D))
    f = (rng.random((B, h_kv, n)) < 0.5).astype(np.uint8)
    rep = lambda a: np.repeat(a, h // h_kv, axis=1)
    assert [orc.kv_head_of(i, h, h_kv) for i in range(h)] == [0, 0, 0, 1, 1, 1]
    assert np.array_equal(orc.prefill_attention(Q, K, V, f), orc.prefill_attention(Q, rep(K), rep(V), rep(f)))
    q = rng.standard_normal((B, h, D))
    kn, vn = rng.standard_normal((B, h_kv, D)), rng.standard_normal((B, h_kv, D))
    o = orc.decode_attention(q, kn, vn, orc.compact_kv(K, V, f))
    o_rep = orc.decode_attention(q, rep(kn), rep(vn), orc.compact_kv(rep(K), rep(V), rep(f)))
    assert np.array_equal(o, o_rep)
    # and query heads of one group really differ only through q
    Q2 = Q.copy()
    Q2[:, 1] = Q2[:, 0]
    O2 = orc.prefill_attention(Q2, K, V, f)
    assert np.array_equal(O2[:, 0], O2[:, 1])


# ---- recent-token window (Appendix, Table 6: the w most recent tokens are always visible) ----
def _visible_set_window(flags, j, w):
    return [t for t in range(j + 1) if j - t < w or flags[t] == 1]


@pytest.mark.parametrize("n,w", [(6, 2), (7, 3), (7, 5), (5, 10)])
def test_window_brute_force_every_flag_pattern(n, w):
    D = 3
    Q, K, V = (_rand((n, D), 40 + n + s) for s in (0, 1, 2))
    scale = 1.0 / math.sqrt(D)
    for pattern in itertools.product([0, 1], repeat=n):
        f = np.asarray(pattern, dtype=np.uint8)
        O = orc.prefill_head(Q, K, V, f, window=w)
        for j in range(n):
            want = _attend_set(Q[j], K, V, _visible_set_window(pattern, j, w), scale)
            assert np.max(np.abs(O[j] - want)) < 1e-12, (pattern, j)


def test_window_of_one_is_the_published_method_and_a_full_window_is_causal_attention():
    n, D = 9, 4
    Q, K, V = (_rand((n, D), 70 + s) for s in (0, 1, 2))
    f = (np.random.default_rng(73).random(n) < 0.4).astype(np.uint8)
    assert np.array_equal(orc.eviction_mask(f, window=1), orc.eviction_mask(f))
    assert np.array_equal(orc.prefill_head(Q, K, V, f, window=1), orc.prefill_head(Q, K, V, f))
    # a window that covers the whole prompt leaves nothing to evict: the flags drop out
    causal = orc.prefill_head(Q, K, V, np.ones(n, dtype=np.uint8))
    np.testing.assert_allclose(orc.prefill_head(Q, K, V, f, window=n), causal, rtol=0, atol=1e-13)
    np.testing.assert_allclose(orc.prefill_head(Q, K, V, np.zeros(n, dtype=np.uint8), window=n + 3), causal, rtol=0, atol=1e-13)


def test_window_mask_entries_all_evicted_is_a_band():
    M = orc.eviction_mask(np.zeros(6, dtype=np.uint8), window=3)
    want = np.array([[1, 0, 0, 0, 0, 0],
                     [1, 1, 0, 0, 0, 0],
                     [1, 1, 1, 0, 0, 0],
                     [0, 1, 1, 1, 0, 0],
                     [0, 0, 1, 1, 1, 0],
                     [0, 0, 0, 1, 1, 1]])
    assert np.array_equal(M, want)
    # all evicted, window 2, value rows one-hot and equal scores: the mean of the last two values
    n = 5
    O = orc.prefill_head(np.zeros((n, 2)), np.ones((n, 2)), np.eye(n), np.zeros(n, dtype=np.uint8), window=2)
    want = np.zeros((n, n))
    want[0, 0] = 1.0
    for j in range(1, n):
        want[j, j] = want[j, j - 1] = 0.5
    np.testing.assert_allclose(O, want, rtol=0, atol=1e-15)
