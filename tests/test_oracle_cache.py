"""Pins for the oracle's selective caching, decode attention and append
(Sec. 3.1 decoding stage; Sec. 3.3 retention rule; Eq. 5 case j = t)."""
import math

import numpy as np
import pytest

from oracle import ag_oracle as orc


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_compaction_properties():
    B, h, n, D = 2, 3, 41, 4
    K = _rand((B, h, n, D), 1).astype(np.float32)
    V = _rand((B, h, n, D), 2).astype(np.float32)
    flags = (np.random.default_rng(3).random((B, h, n)) < 0.45).astype(np.uint8)
    flags[0, 0] = 0
    flags[1, 2] = 1
    cache = orc.compact_kv(K, V, flags)
    L = orc.cache_lengths(cache)
    assert L[0, 0] == 0 and L[1, 2] == n
    for b in range(B):
        for i in range(h):
            c = cache[b][i]
            idx = c["idx"]
            assert np.all(np.diff(idx) > 0)
            assert np.all(flags[b, i][idx] == 1)
            assert len(idx) + int((flags[b, i] == 0).sum()) == n
            assert c["k"].dtype == np.float32
            assert np.array_equal(c["k"], K[b, i][idx]) and np.array_equal(c["v"], V[b, i][idx])
            P = orc.exclusive_counts(flags[b, i])
            assert P[0] == 0 and P[n] == len(idx)
            assert np.array_equal(P[1:], np.cumsum(flags[b, i].astype(np.int64)))
            # rows r < P[j] of the cache are exactly the retained tokens before j
            for j in (0, 7, n - 1):
                assert list(idx[:P[j]]) == [t for t in range(j) if flags[b, i, t] == 1]


def test_decode_matches_longer_prefill():
    # Prefill over n + m tokens, rows n.., must equal m decode steps after a
    # prefill over n tokens when the decode tokens carry the same flags.
    B, h, n, m, D = 2, 2, 17, 6, 8
    Q, K, V = (_rand((B, h, n + m, D), s) for s in (11, 12, 13))
    flags = (np.random.default_rng(14).random((B, h, n + m)) < 0.5).astype(np.uint8)
    full = orc.prefill_attention(Q, K, V, flags)
    cache = orc.compact_kv(K[:, :, :n], V[:, :, :n], flags[:, :, :n])
    for s in range(m):
        t = n + s
        o = orc.decode_attention(Q[:, :, t], K[:, :, t], V[:, :, t], cache)
        assert np.max(np.abs(o - full[:, :, t])) < 1e-12
        orc.cache_append(cache, K[:, :, t], V[:, :, t], flags[:, :, t])
    want_len = flags.sum(axis=2)
    assert np.array_equal(orc.cache_lengths(cache), want_len)


def test_empty_cache_returns_own_value():
    D = 8
    q, k, v = (_rand((1, 1, D), s) for s in (21, 22, 23))
    cache = [[{"k": np.zeros((0, D)), "v": np.zeros((0, D)), "idx": np.zeros(0, dtype=np.int64)}]]
    o = orc.decode_attention(q, k, v, cache)
    assert np.array_equal(o, v)


def test_decode_two_keys_closed_form():
    D = 4
    q, kn, vn = (_rand((D,), s) for s in (31, 32, 33))
    kc, vc = _rand((1, D), 34), _rand((1, D), 35)
    o = orc.decode_head(q, kn, vn, kc, vc, scale=0.5)
    a = 1.0 / (1.0 + math.exp(-0.5 * float(np.dot(q, kc[0] - kn))))
    assert np.max(np.abs(o - (a * vc[0] + (1 - a) * vn))) < 1e-14


def test_append_is_conditional_and_bit_exact():
    B, h, D = 2, 2, 4
    cache = orc.compact_kv(np.zeros((B, h, 3, D), np.float32), np.zeros((B, h, 3, D), np.float32),
                           np.ones((B, h, 3), np.uint8))
    k = _rand((B, h, D), 41).astype(np.float32)
    v = _rand((B, h, D), 42).astype(np.float32)
    f = np.asarray([[1, 0], [0, 1]], dtype=np.uint8)
    orc.cache_append(cache, k, v, f)
    assert orc.cache_lengths(cache).tolist() == [[4, 3], [3, 4]]
    assert np.array_equal(cache[0][0]["k"][3], k[0, 0]) and np.array_equal(cache[1][1]["v"][3], v[1, 1])
    # a token whose flag evicts it still attended to itself in decode_attention
    # but never reaches the cache of later steps
    assert cache[0][1]["k"].shape[0] == 3


@pytest.mark.parametrize("w,n", [(2, 17), (5, 17), (10, 17), (5, 3), (4, 0)])
def test_window_decode_matches_longer_prefill(w, n):
    # the same statement two ways: the band mask on n + m tokens, and the cache with its
    # list of recent tokens carried through m decode steps (prompts shorter than the window too)
    B, h, m, D = 2, 2, 12, 8
    Q, K, V = (_rand((B, h, n + m, D), s) for s in (21, 22, 23))
    flags = (np.random.default_rng(24).random((B, h, n + m)) < 0.4).astype(np.uint8)
    full = orc.prefill_attention(Q, K, V, flags, window=w)
    assert not np.allclose(full, orc.prefill_attention(Q, K, V, flags))          # the window matters here
    cache = orc.compact_kv(K[:, :, :n], V[:, :, :n], flags[:, :, :n], window=w)
    for s in range(m):
        t = n + s
        o = orc.decode_attention(Q[:, :, t], K[:, :, t], V[:, :, t], cache)
        assert np.max(np.abs(o - full[:, :, t])) < 1e-12, s
        orc.cache_append(cache, K[:, :, t], V[:, :, t], flags[:, :, t], window=w)
        assert all(len(c["recent"]) == min(w - 1, t + 1) for row in cache for c in row)
    # the window never changes what is cached for good
    assert np.array_equal(orc.cache_lengths(cache), flags.sum(axis=2))
