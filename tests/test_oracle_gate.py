"""Pins for the oracle's gate: MHA' (Sec. 3.3), Eq. 3, Eq. 4, gamma (Sec. 3.5)."""
import math

import numpy as np
import pytest
import torch

from oracle import ag_oracle as orc


def _w(shape, seed, std=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * std


def _gate_inputs(n=11, d=6, hg=2, Dg=4, h=3, seed=0):
    X = _w((n, d), seed)
    Wq, Wk, Wv = (_w((d, hg * Dg), seed + 1 + k, 0.5) for k in range(3))
    Wo = _w((hg * Dg, h), seed + 4, 0.5)
    return X, Wq, Wk, Wv, Wo


def test_zero_output_projection_gives_sigmoid_of_gamma():
    X, Wq, Wk, Wv, Wo = _gate_inputs()
    s, f = orc.attention_gate(X[None], Wq, Wk, Wv, 0 * Wo, 2, gamma=2.0, tau=0.5)
    assert np.all(s == 0)
    assert np.all(f == 1)          # Sigmoid(2) = 0.88 > 0.5: everything retained at init
    _, f0 = orc.attention_gate(X[None], Wq, Wk, Wv, 0 * Wo, 2, gamma=0.0, tau=0.5)
    assert np.all(f0 == 0)         # Sigmoid(0) = 0.5 is not > 0.5 (strict)
    _, f1 = orc.attention_gate(X[None], Wq, Wk, Wv, 0 * Wo, 2, gamma=None, tau=0.3)
    assert np.all(f1 == 1)         # 0.5 > 0.3


@pytest.mark.parametrize("causal", [True, False])
def test_identical_tokens_closed_form(causal):
    # If every row of X equals x then every value row equals x Wv, attention
    # averages identical rows, and s = x Wv Wo regardless of the mask.
    X, Wq, Wk, Wv, Wo = _gate_inputs(seed=3)
    X = np.tile(X[:1], (X.shape[0], 1))
    s = orc.mha_prime(X, Wq, Wk, Wv, Wo, 2, causal=causal)
    want = X[:1] @ Wv @ Wo
    assert np.max(np.abs(s - want)) < 1e-12


@pytest.mark.parametrize("causal", [True, False])
def test_single_token(causal):
    X, Wq, Wk, Wv, Wo = _gate_inputs(n=1, seed=5)
    s = orc.mha_prime(X, Wq, Wk, Wv, Wo, 2, causal=causal)
    assert np.max(np.abs(s - X @ Wv @ Wo)) < 1e-13


@pytest.mark.parametrize("causal", [True, False])
def test_against_library_attention(causal):
    n, d, hg, Dg, h = 23, 10, 3, 4, 5
    X, Wq, Wk, Wv, Wo = _gate_inputs(n, d, hg, Dg, h, seed=7)
    s = orc.mha_prime(X, Wq, Wk, Wv, Wo, hg, causal=causal)
    tX = torch.from_numpy(X)
    split = lambda W: (tX @ torch.from_numpy(W)).view(n, hg, Dg).transpose(0, 1)
    H = torch.nn.functional.scaled_dot_product_attention(split(Wq), split(Wk), split(Wv), is_causal=causal)
    want = (H.transpose(0, 1).reshape(n, hg * Dg) @ torch.from_numpy(Wo)).numpy()
    assert np.max(np.abs(s - want)) < 1e-12


def test_python_loops_tiny():
    n, d, hg, Dg, h = 5, 3, 2, 2, 3
    X, Wq, Wk, Wv, Wo = _gate_inputs(n, d, hg, Dg, h, seed=9)
    s = orc.mha_prime(X, Wq, Wk, Wv, Wo, hg, causal=True)
    proj = lambda W, t, c: sum(X[t, a] * W[a, c] for a in range(d))
    for j in range(n):
        Hrow = []
        for g in range(hg):
            cols = range(g * Dg, (g + 1) * Dg)
            w = [math.exp(sum(proj(Wq, j, c) * proj(Wk, t, c) for c in cols) / math.sqrt(Dg))
                 for t in range(j + 1)]
            z = sum(w)
            Hrow += [sum(w[t] * proj(Wv, t, c) for t in range(j + 1)) / z for c in cols]
        for i in range(h):
            assert abs(s[j, i] - sum(Hrow[c] * Wo[c, i] for c in range(hg * Dg))) < 1e-12


def test_causal_reading_ignores_the_future_and_global_does_not():
    X, Wq, Wk, Wv, Wo = _gate_inputs(n=12, seed=11)
    X2 = X.copy()
    X2[8:] += 1.0
    a = orc.mha_prime(X, Wq, Wk, Wv, Wo, 2, causal=True)
    b = orc.mha_prime(X2, Wq, Wk, Wv, Wo, 2, causal=True)
    assert np.array_equal(a[:8], b[:8]) and not np.allclose(a[8:], b[8:])
    a = orc.mha_prime(X, Wq, Wk, Wv, Wo, 2, causal=False)
    b = orc.mha_prime(X2, Wq, Wk, Wv, Wo, 2, causal=False)
    assert not np.allclose(a[:8], b[:8])


def test_threshold_rule_and_layout():
    s = np.asarray([[[-3.0, -0.1, 0.0, 0.1, 3.0], [0.0, 0.0, 0.0, 0.0, 0.0]]])   # [1, 2, 5]
    f = orc.gate_flags(s, gamma=None, tau=0.5)
    assert f.dtype == np.uint8 and f.shape == (1, 2, 5)
    assert f[0, 0].tolist() == [0, 0, 0, 1, 1]
    f = orc.gate_flags(s, gamma=np.asarray([0.0, 1e-9]), tau=0.5)
    assert f[0, 1].tolist() == [1, 1, 1, 1, 1]
    # tau = 0.3: keep iff s > logit(0.3) = -0.8473
    f = orc.gate_flags(s, gamma=None, tau=0.3)
    assert f[0, 0].tolist() == [0, 1, 1, 1, 1]
    # batch / head-major layout of gate_scores
    X, Wq, Wk, Wv, Wo = _gate_inputs(seed=13)
    Xb = np.stack([X, X[::-1]])
    sc = orc.gate_scores(Xb, Wq, Wk, Wv, Wo, 2)
    assert sc.shape == (2, 3, 11)
    assert np.array_equal(sc[1], orc.mha_prime(X[::-1], Wq, Wk, Wv, Wo, 2).T)


def test_keep_count_grows_with_gamma():
    X, Wq, Wk, Wv, Wo = _gate_inputs(n=64, seed=15)
    s = orc.gate_scores(X[None], Wq, Wk, Wv, Wo, 2)
    counts = [int(orc.gate_flags(s, g, 0.5).sum()) for g in (-5.0, -0.5, 0.0, 0.5, 5.0)]
    assert counts == sorted(counts) and counts[0] == 0 and counts[-1] == s.size


# ---- the local (linear) gate of Sec. 3.4, "Local or global?" / ablation setting (5)

def test_linear_gate_unit_rows_pick_rows_of_the_weight():
    """A token whose hidden state is the unit vector e_k scores W_lin[k, :] exactly."""
    d, h = 7, 3
    W = _w((d, h), 40)
    s = orc.linear_gate_scores(np.eye(d)[None], W)            # token t = e_t
    assert s.shape == (1, h, d)
    assert np.array_equal(s[0], W.T)


def test_linear_gate_python_loops_tiny():
    B, n, d, h = 2, 5, 4, 3
    X, W = _w((B, n, d), 41), _w((d, h), 42)
    ref = np.zeros((B, h, n))
    for b in range(B):
        for t in range(n):
            for i in range(h):
                acc = 0.0
                for k in range(d):
                    acc += X[b, t, k] * W[k, i]
                ref[b, i, t] = acc
    assert np.allclose(orc.linear_gate_scores(X, W), ref, rtol=0, atol=1e-14)


def test_linear_gate_is_local_and_linear():
    """A token's score ignores every other token (the opposite of MHA'), and scores add over inputs."""
    n, d, h = 9, 6, 4
    X, Y, W = _w((1, n, d), 43), _w((1, n, d), 44), _w((d, h), 45)
    s = orc.linear_gate_scores(X, W)
    X2 = X.copy()
    X2[0, 3] += 10.0
    s2 = orc.linear_gate_scores(X2, W)
    keep = np.arange(n) != 3
    assert np.array_equal(s[:, :, keep], s2[:, :, keep]) and not np.allclose(s[:, :, 3], s2[:, :, 3])
    assert np.allclose(orc.linear_gate_scores(X + 2 * Y, W), s + 2 * orc.linear_gate_scores(Y, W), atol=1e-12)


def test_linear_gate_flags_follow_eq4():
    X, W = _w((1, 6, 3), 46), _w((3, 2), 47)
    gamma, tau = np.array([0.3, -0.2]), 0.6
    s, f = orc.linear_gate(X, W, gamma, tau)
    want = 1.0 / (1.0 + np.exp(-(s + gamma[None, :, None]))) > tau
    assert np.array_equal(f, want.astype(np.uint8)) and f.dtype == np.uint8


# ---- batches of sequences of different lengths (padding is never retained)

def test_ragged_gate_padding_is_evicted_and_never_seen():
    """Whatever sits in the padding, the valid tokens score as their sequence alone does, in the
    causal and in the bidirectional reading of MHA', and every padding flag is 0."""
    n, d, hg, Dg, h = 9, 6, 2, 4, 3
    X = _w((2, n, d), 60)
    Wq, Wk, Wv = (_w((d, hg * Dg), 61 + k, 0.5) for k in range(3))
    Wo = _w((hg * Dg, h), 64, 0.5)
    lens = [n, 4]
    for causal in (True, False):
        fn = lambda x: orc.attention_gate(x, Wq, Wk, Wv, Wo, hg, gamma=0.1, tau=0.5, causal=causal)
        s, f = orc.ragged_gate(X, lens, fn)
        X2 = X.copy()
        X2[1, 4:] = 1e3                                        # garbage in the padding
        s2, f2 = orc.ragged_gate(X2, lens, fn)
        assert np.array_equal(s, s2) and np.array_equal(f, f2)
        assert np.all(f[1, :, 4:] == 0) and np.all(s[1, :, 4:] == 0)
        alone_s, alone_f = fn(X[1:2, :4])
        assert np.array_equal(s[1, :, :4], alone_s[0]) and np.array_equal(f[1, :, :4], alone_f[0])
        full_s, full_f = fn(X[0:1])
        assert np.array_equal(s[0], full_s[0]) and np.array_equal(f[0], full_f[0])
    # the bidirectional reading does depend on the length: a full-length run differs on the valid part
    s_full, _ = orc.attention_gate(X, Wq, Wk, Wv, Wo, hg, gamma=0.1, tau=0.5, causal=False)
    s_rag, _ = orc.ragged_gate(X, lens, lambda x: orc.attention_gate(x, Wq, Wk, Wv, Wo, hg, 0.1, 0.5, causal=False))
    assert not np.allclose(s_full[1, :, :4], s_rag[1, :, :4])


# ---- eviction guided by the previous layer (Sec. 4.4, settings (4-1) and (4-2)) ----
def _const_gate(keep, shape):
    """A gate whose answer is known without computing anything: W^{O'} = 0 gives score 0, so
    Sigmoid(gamma) > tau keeps every token (gamma large) or none (gamma very negative)."""
    B, h, n = shape
    rng = np.random.default_rng(5)
    X = rng.standard_normal((B, n, 8))
    Wq, Wk, Wv = (rng.standard_normal((8, 4)) for _ in range(3))
    gamma = np.full(h, 20.0 if keep else -20.0)
    return lambda: orc.attention_gate(X, Wq, Wk, Wv, np.zeros((4, h)), 2, gamma, 0.5)


@pytest.mark.parametrize("first_gated", [1, 2])
def test_previous_layer_flags_take_the_module_of_the_layer_before(first_gated):
    shape = (2, 3, 6)
    keeps = [False, True, False, False, True]          # what layer l's own module answers
    used = orc.previous_layer_flags([_const_gate(k, shape) for k in keeps], first_gated, shape)
    assert len(used) == len(keeps)
    for l, f in enumerate(used):
        assert f.shape == shape and f.dtype == np.uint8
        expect = 1 if l < first_gated else int(keeps[l - 1])
        assert (f == expect).all(), (l, first_gated)


def test_previous_layer_flags_take_the_hidden_states_of_the_layer_before():
    # one shared local gate with positive weights: a layer's flags are the sign of ITS hidden states
    shape = (1, 2, 5)
    W = np.ones((4, 2))
    signs = [+1.0, -1.0, -1.0, +1.0]
    Xs = [s * np.ones((1, 5, 4)) for s in signs]
    gates = [lambda X=X: orc.linear_gate(X, W, np.zeros(2), 0.5) for X in Xs]
    used = orc.previous_layer_flags(gates, 1, shape)
    assert [int(f.all()) for f in used] == [1, 1, 0, 0]
    assert [int(f.any()) for f in used] == [1, 1, 0, 0]


def test_previous_layer_flags_unevicted_layers_are_plain_causal_attention():
    shape = (1, 2, 7)
    used = orc.previous_layer_flags([_const_gate(False, shape)] * 2, 1, shape)
    rng = np.random.default_rng(11)
    Q, K, V = (rng.standard_normal((1, 2, 7, 4)) for _ in range(3))
    O = orc.prefill_attention(Q, K, V, used[0])
    ref = torch.nn.functional.scaled_dot_product_attention(*(torch.from_numpy(t) for t in (Q, K, V)), is_causal=True)
    np.testing.assert_allclose(O, ref.numpy(), rtol=1e-10, atol=1e-12)
    # and the layer after it, guided by a module that evicts everything, sees only the diagonal
    np.testing.assert_allclose(orc.prefill_attention(Q, K, V, used[1]), V, rtol=1e-12, atol=1e-12)


def test_previous_layer_flags_need_a_previous_layer():
    with pytest.raises(ValueError):
        orc.previous_layer_flags([_const_gate(True, (1, 1, 2))], 0, (1, 1, 2))
