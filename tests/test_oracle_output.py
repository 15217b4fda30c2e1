"""Pins of the oracle's output projection (Eq. 1: MHA(X) = [H_1 .. H_h] W^O, with the skip connection
a stack of layers adds).  CPU only."""
import numpy as np

from oracle import ag_oracle as orc


def _case(seed, B=2, h=3, n=5, D=4, d=6):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((B, h, n, D)), rng.standard_normal((h * D, d)), rng.standard_normal((B, n, d))


def test_identity_weight_is_pure_concatenation_of_the_heads():
    # W^O = I (d = h D): token t of the output is [H_1[t], ..., H_h[t]], exactly
    H, _, _ = _case(0)
    B, h, n, D = H.shape
    Y = orc.mha_output(H, np.eye(h * D))
    for b in range(B):
        for t in range(n):
            for i in range(h):
                assert np.array_equal(Y[b, t, i * D:(i + 1) * D], H[b, i, t])


def test_against_loops_written_out():
    H, Wo, X = _case(1)
    B, h, n, D = H.shape
    Y = orc.mha_output(H, Wo, X)
    for b in range(B):
        for t in range(n):
            for c in range(Wo.shape[1]):
                y = X[b, t, c] + sum(H[b, i, t, e] * Wo[i * D + e, c] for i in range(h) for e in range(D))
                assert abs(Y[b, t, c] - y) < 1e-12


def test_against_a_library_contraction():
    H, Wo, X = _case(2, B=3, h=4, n=9, D=5, d=7)
    Y = orc.mha_output(H, Wo)
    Yl = np.einsum("bhnc,hcd->bnd", H, Wo.reshape(4, 5, 7))
    assert np.allclose(Y, Yl, rtol=0, atol=1e-12)
    assert np.allclose(orc.mha_output(H, Wo, X), Yl + X, rtol=0, atol=1e-12)


def test_a_head_reaches_the_output_through_its_own_rows_of_the_weight_only():
    H, Wo, _ = _case(3)
    B, h, n, D = H.shape
    Y = orc.mha_output(H, Wo)
    Wo2 = Wo.copy()
    Wo2[D:2 * D] = 0.0                                    # rows of head 1
    H2 = H.copy()
    H2[:, 1] += 5.0                                       # head 1 changes, its rows of W^O are zero
    assert np.allclose(orc.mha_output(H2, Wo2), orc.mha_output(H, Wo2), rtol=0, atol=1e-12)
    assert not np.allclose(orc.mha_output(H2, Wo), Y)
    # a token's output depends on that token's head outputs only
    H3 = H.copy()
    H3[0, :, 2] += 1.0
    Y3 = orc.mha_output(H3, Wo)
    changed = np.abs(Y3 - Y).max(axis=-1) > 0
    want = np.zeros((B, n), dtype=bool)
    want[0, 2] = True
    assert np.array_equal(changed, want)


def test_zero_weight_leaves_the_skip_connection_and_no_skip_leaves_the_product():
    H, Wo, X = _case(4)
    assert np.array_equal(orc.mha_output(H, np.zeros_like(Wo), X), X)
    assert np.array_equal(orc.mha_output(H, Wo, np.zeros_like(X)), orc.mha_output(H, Wo))


def test_transposed_weight_or_head_major_concatenation_would_be_caught():
    # the order of the concatenation is head-major then feature (column i D + e), not feature-major
    H, _, _ = _case(5, B=1, h=2, n=1, D=2, d=4)
    Wo = np.arange(16, dtype=np.float64).reshape(4, 4)
    Y = orc.mha_output(H, Wo)[0, 0]
    concat = np.array([H[0, 0, 0, 0], H[0, 0, 0, 1], H[0, 1, 0, 0], H[0, 1, 0, 1]])
    assert np.allclose(Y, concat @ Wo, rtol=0, atol=1e-12)
    wrong_order = np.array([H[0, 0, 0, 0], H[0, 1, 0, 0], H[0, 0, 0, 1], H[0, 1, 0, 1]])
    assert not np.allclose(Y, wrong_order @ Wo)
    assert not np.allclose(Y, concat @ Wo.T)
