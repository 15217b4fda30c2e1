"""Pins of the oracle's key/value projection (Eq. 2: K_i = X W^K_i, V_i = X W^V_i) and of the
projection followed by selective caching (Sec. 3.3).  CPU only."""
import numpy as np

from oracle import ag_oracle as orc


def _case(seed, B=2, n=7, d=5, h=3, D=4):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((B, n, d)), rng.standard_normal((d, h * D)), rng.standard_normal((d, h * D)),
            (rng.random((B, h, n)) < 0.5).astype(np.uint8))


def test_unit_rows_return_rows_of_the_weights():
    # token t = unit vector e_c  =>  K_i[t] = row c of W^K_i, exactly
    d, h, D = 6, 2, 3
    rng = np.random.default_rng(0)
    Wk, Wv = rng.standard_normal((d, h * D)), rng.standard_normal((d, h * D))
    X = np.eye(d)[None]                                   # n = d, token c = e_c
    K, V = orc.project_kv(X, Wk, Wv, h)
    for i in range(h):
        assert np.array_equal(K[0, i], Wk[:, i * D:(i + 1) * D])
        assert np.array_equal(V[0, i], Wv[:, i * D:(i + 1) * D])


def test_against_loops_written_out():
    X, Wk, Wv, _ = _case(1)
    B, n, d = X.shape
    h, D = 3, 4
    K, V = orc.project_kv(X, Wk, Wv, h)
    for b in range(B):
        for i in range(h):
            for t in range(n):
                for c in range(D):
                    k = sum(X[b, t, a] * Wk[a, i * D + c] for a in range(d))
                    v = sum(X[b, t, a] * Wv[a, i * D + c] for a in range(d))
                    assert abs(K[b, i, t, c] - k) < 1e-12 and abs(V[b, i, t, c] - v) < 1e-12


def test_against_library_contraction():
    X, Wk, Wv, _ = _case(2, B=3, n=9, d=8, h=2, D=5)
    K, V = orc.project_kv(X, Wk, Wv, 2)
    Kl = np.einsum("bnd,dhc->bhnc", X, Wk.reshape(8, 2, 5))
    Vl = np.einsum("bnd,dhc->bhnc", X, Wv.reshape(8, 2, 5))
    assert np.allclose(K, Kl, rtol=0, atol=1e-12) and np.allclose(V, Vl, rtol=0, atol=1e-12)


def test_keys_and_values_take_their_own_weights_and_heads_their_own_columns():
    X, Wk, Wv, _ = _case(3)
    K, V = orc.project_kv(X, Wk, Wv, 3)
    K0, V0 = orc.project_kv(X, Wk, np.zeros_like(Wv), 3)
    assert np.array_equal(K0, K) and not np.any(V0) and np.any(V)
    Wk2 = Wk.copy()
    Wk2[:, 4:8] += 1.0                                    # columns of head 1 only
    K2, _ = orc.project_kv(X, Wk2, Wv, 3)
    assert np.array_equal(K2[:, 0], K[:, 0]) and np.array_equal(K2[:, 2], K[:, 2])
    assert not np.allclose(K2[:, 1], K[:, 1])
    X2 = X.copy()
    X2[1, 3] += 1.0                                       # one token of one sequence
    K3, _ = orc.project_kv(X2, Wk, Wv, 3)
    changed = np.any(K3 != K, axis=(1, 3))
    assert changed[1, 3] and changed.sum() == 1


def test_cache_holds_the_projected_rows_of_the_retained_tokens():
    X, Wk, Wv, flags = _case(4)
    K, V, cache = orc.project_and_cache(X, Wk, Wv, flags)
    for b in range(2):
        for i in range(3):
            kept = [t for t in range(7) if flags[b, i, t]]
            assert np.array_equal(cache[b][i]["idx"], kept)
            assert len(cache[b][i]["k"]) == len(kept)
            for r, t in enumerate(kept):
                assert np.allclose(cache[b][i]["k"][r], X[b, t] @ Wk[:, i * 4:(i + 1) * 4], rtol=0, atol=1e-12)
                assert np.allclose(cache[b][i]["v"][r], X[b, t] @ Wv[:, i * 4:(i + 1) * 4], rtol=0, atol=1e-12)


def test_queries_unit_rows_loops_and_library():
    d, h, D = 6, 3, 2
    rng = np.random.default_rng(5)
    Wq = rng.standard_normal((d, h * D))
    Q = orc.project_q(np.eye(d)[None], Wq, h)             # token c = e_c  =>  Q_i[c] = row c of W^Q_i
    for i in range(h):
        assert np.array_equal(Q[0, i], Wq[:, i * D:(i + 1) * D])
    X = rng.standard_normal((2, 5, d))
    Q = orc.project_q(X, Wq, h)
    for b in range(2):
        for i in range(h):
            for t in range(5):
                for c in range(D):
                    assert abs(Q[b, i, t, c] - sum(X[b, t, a] * Wq[a, i * D + c] for a in range(d))) < 1e-12
    assert np.allclose(Q, np.einsum("bnd,dhc->bhnc", X, Wq.reshape(d, h, D)), rtol=0, atol=1e-12)
    # with the same weight, queries are what the key projection gives for as many heads
    K, _ = orc.project_kv(X, Wq, Wq, h)
    assert np.allclose(Q, K, rtol=0, atol=1e-12)
