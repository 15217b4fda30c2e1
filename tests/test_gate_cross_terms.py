"""Why MHA' of the gate (Sec. 3.3) carries every operand as a bf16 pair x = hi + lo and evaluates three
products per term: an emulation in numpy of what each dropped cross term does to the gate's scores.
The scores decide a hard threshold (Eq. 4) and are compared with the oracle to 1e-4; a scheme that
drops any one of `Phi Vlo`, `Plo Vhi` (or the cross terms of Q'K'^T) misses that by an order of
magnitude, the three-product scheme keeps it with room to spare."""
import numpy as np


def _bf16(x):
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16               # round to nearest even
    return r.astype(np.uint32).view(np.float32).astype(np.float64)


def _split(x):
    hi = _bf16(x)
    return hi, _bf16(np.asarray(x, dtype=np.float64) - hi)


def _scores(Q, K, V, Wo, gh, D, qk_terms, pv_terms):
    n = Q.shape[0]
    H = np.zeros((n, gh * D))
    for g in range(gh):
        q, k, v = (M[:, g * D:(g + 1) * D] for M in (Q, K, V))
        qh, ql = _split(q)
        kh, kl = _split(k)
        vh, vl = _split(v)
        S = {"exact": q @ k.T, "three": qh @ kh.T + qh @ kl.T + ql @ kh.T, "one": qh @ kh.T}[qk_terms] / np.sqrt(D)
        S = np.where(np.tril(np.ones((n, n), bool)), S, -np.inf)
        P = np.exp(S - S.max(1, keepdims=True))
        ph, pl = _split(P)
        num = {"exact": P @ v, "three": ph @ vh + ph @ vl + pl @ vh, "no_plo": ph @ vh + ph @ vl,
               "no_vlo": ph @ vh + pl @ vh}[pv_terms]
        H[:, g * D:(g + 1) * D] = num / P.sum(1, keepdims=True)
    return H @ Wo


def test_every_cross_term_is_needed_for_the_score_budget():
    rng = np.random.default_rng(0)
    n, d, gh, D, h = 384, 4096, 4, 128, 32                         # the 7B-shaped layer's gate, a short prompt
    X = _bf16(rng.standard_normal((n, d)))
    Wq, Wk, Wv = (_bf16(0.02 * rng.standard_normal((d, gh * D))) for _ in range(3))
    Wo = _bf16(0.02 * rng.standard_normal((gh * D, h)))
    Q, K, V = (np.float32(X @ W).astype(np.float64) for W in (Wq, Wk, Wv))   # the projection leaves float32
    ref = _scores(Q, K, V, Wo, gh, D, "exact", "exact")
    err = {(a, b): np.abs(_scores(Q, K, V, Wo, gh, D, a, b) - ref).max()
           for a, b in (("three", "three"), ("three", "no_plo"), ("three", "no_vlo"), ("one", "three"))}
    assert err[("three", "three")] < 2e-5                          # the scheme the kernels use
    assert err[("three", "no_plo")] > 3e-4                         # P V' without Plo Vhi
    assert err[("three", "no_vlo")] > 3e-4                         # P V' without Phi Vlo
    assert err[("one", "three")] > 3e-4                            # Q'K'^T in plain bf16
