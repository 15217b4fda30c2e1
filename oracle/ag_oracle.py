"""fp64 CPU oracle for the Attention-Gate (AG) gated attention layer.

TEST INFRASTRUCTURE ONLY.  This module is the slow, dense, obviously-correct
statement of what the layer computes.  It is imported by the tests, by the
smoke check and by the benchmark's CPU-baseline leg, and by nothing else: the
product path (the CUDA library and its Python binding) never calls it and
shares no code, table or helper with it.

Every function evaluates the paper's definition on the ORIGINAL, uncompacted
tensors in float64.  There is no compaction, no prefix-sum shortcut, no
tiling, no online softmax: those are the devices of the GPU path and are what
this oracle checks.

Layouts (same as the C boundary):
    X               [B, n, d]        hidden states
    Wq_g/Wk_g/Wv_g  [d, h' * D']     AG projections, row-major "in x out"
    Wo_g            [h' * D', h]     AG output projection (Sec. 3.3, W^{O'})
    Q, K, V, O      [B, h, n, D]
    Wo              [h * D, d]       output projection of Eq. 1 (W^O)
    scores          [B, h, n]        MHA'(X) transposed to head-major
    flags           [B, h, n] uint8  1 = retain, 0 = evict

Pins (see tests/test_oracle_*.py): all-keep == textbook causal attention,
all-evict == O[j] = V[j], brute force over explicit visible-key sets for all
2^n flag patterns at tiny n, uniform-attention closed forms, gate closed
forms (Wo'=0, identical rows, n=1), causality of MHA', prefill/decode
consistency; the output projection of Eq. 1 by W^O = identity (pure concatenation),
written-out loops, a library contraction and its locality in heads and tokens.  What remains unpinned: the paper prints no worked numeric
example and does not say whether MHA' is causal; "parity unpinned" applies to
that choice of reading only (both readings are implemented).
"""
import math

import numpy as np

F64 = np.float64


def _as_f64(a):
    return np.asarray(a, dtype=F64)


def softmax_rows(S):
    """Row softmax of a matrix whose masked entries are -inf (Eq. 2 with the
    additive term -INF(1-M) taken in the INF -> infinity limit).  Every row
    must have at least one finite entry; Eq. 5 guarantees it (the diagonal)."""
    m = np.max(S, axis=-1, keepdims=True)
    E = np.exp(S - m)
    return E / np.sum(E, axis=-1, keepdims=True)


# --------------------------------------------------------------------------
# Step 1: the gate.  Sec. 3.3 "Main architecture", Eq. 3, Eq. 4; gamma from
# Sec. 3.5 "Initialization".
# --------------------------------------------------------------------------
def mha_prime(X, Wq_g, Wk_g, Wv_g, Wo_g, gate_heads, causal=True):
    """MHA'(X) for one sequence: Eq. 1 / Eq. 2 with h' heads of width D' and
    the output projection W^{O'} in R^{h'D' x h}.  X [n, d] -> [n, h].

    `causal=True` applies the ordinary lower-triangular decoder mask inside
    MHA'; `causal=False` lets every token see the whole sequence.  The paper
    does not say which; causal is the default reading here."""
    X = _as_f64(X)
    Wq_g, Wk_g, Wv_g, Wo_g = map(_as_f64, (Wq_g, Wk_g, Wv_g, Wo_g))
    n = X.shape[0]
    width = Wq_g.shape[1]
    assert width % gate_heads == 0
    Dg = width // gate_heads
    Qg = X @ Wq_g
    Kg = X @ Wk_g
    Vg = X @ Wv_g
    heads = []
    for g in range(gate_heads):
        c = slice(g * Dg, (g + 1) * Dg)
        S = (Qg[:, c] @ Kg[:, c].T) / math.sqrt(Dg)
        if causal:
            j = np.arange(n)[:, None]
            t = np.arange(n)[None, :]
            S = np.where(t <= j, S, -np.inf)
        A = softmax_rows(S)
        heads.append(A @ Vg[:, c])
    H = np.concatenate(heads, axis=1)          # [n, h' D']
    return H @ Wo_g                            # [n, h]


def gate_scores(X, Wq_g, Wk_g, Wv_g, Wo_g, gate_heads, causal=True):
    """scores[b, i, t] = MHA'(X_b)[t, i] for every sequence of the batch."""
    X = _as_f64(X)
    out = [mha_prime(X[b], Wq_g, Wk_g, Wv_g, Wo_g, gate_heads, causal).T
           for b in range(X.shape[0])]
    return np.stack(out, axis=0)


def sigmoid(z):
    return 1.0 / (1.0 + np.exp(-_as_f64(z)))


def gate_flags(scores, gamma, tau):
    """Eq. 4 with the optional constant inside the Sigmoid:
    flag = 1 iff Sigmoid(s + gamma_i) > tau (strict).  gamma: scalar, [h] or
    None.  scores [B, h, n] -> uint8 [B, h, n]."""
    s = _as_f64(scores)
    if gamma is None:
        g = np.zeros(s.shape[1], dtype=F64)
    else:
        g = np.broadcast_to(_as_f64(gamma), (s.shape[1],))
    p = sigmoid(s + g[None, :, None])
    return (p > tau).astype(np.uint8)


def linear_gate_scores(X, W_lin):
    """The local gate of Sec. 3.4 ("Local or global?"; ablation setting (5)):
    MHA' is replaced by one linear layer, so a token's score depends on its own
    hidden state only: s[b, i, t] = X[b, t, :] . W_lin[:, i].
    X [B, n, d], W_lin [d, h] -> scores [B, h, n]."""
    X = _as_f64(X)
    W = _as_f64(W_lin)
    return np.stack([(X[b] @ W).T for b in range(X.shape[0])], axis=0)


def linear_gate(X, W_lin, gamma, tau):
    """Flags of the local gate: the threshold of Eq. 4 on linear_gate_scores."""
    s = linear_gate_scores(X, W_lin)
    return s, gate_flags(s, gamma, tau)


def attention_gate(X, Wq_g, Wk_g, Wv_g, Wo_g, gate_heads, gamma, tau, causal=True):
    """AG(X) = G(MHA'(X), tau), Eq. 3.  Returns (scores, flags)."""
    s = gate_scores(X, Wq_g, Wk_g, Wv_g, Wo_g, gate_heads, causal)
    return s, gate_flags(s, gamma, tau)


def ragged_gate(X, seq_lens, gate_fn):
    """A batch of sequences of different lengths, padded to a common n (the paper
    treats one sequence; sequences of a batch are independent).  Sequence b is
    its first seq_lens[b] tokens: the gate runs on exactly those (gate_fn maps
    [1, len, d] -> (scores, flags), e.g. a closure over attention_gate or
    linear_gate), the padding positions get score 0 and flag 0 (evicted), so
    nothing downstream ever retains them."""
    X = _as_f64(X)
    B, n = X.shape[0], X.shape[1]
    scores = flags = None
    for b in range(B):
        L = int(seq_lens[b])
        s, f = gate_fn(X[b:b + 1, :L])
        if scores is None:
            scores = np.zeros((B, s.shape[1], n), dtype=F64)
            flags = np.zeros((B, s.shape[1], n), dtype=np.uint8)
        scores[b, :, :L] = s[0]
        flags[b, :, :L] = f[0]
    return scores, flags


def previous_layer_flags(gate_fns, first_gated, shape):
    """Eviction guided by the previous layer (Sec. 4.4, ablation settings (4-1) and
    (4-2)): layer l evicts by the flags that layer l-1's AG module computes from
    layer l-1's hidden states, so a layer's gate no longer has to finish before
    that layer's attention starts.  Layers before `first_gated` (1 in setting
    (4-1), 2 in (4-2)) evict nothing: their flags are all 1.

    gate_fns[l]() returns (scores, flags) of layer l's AG module applied to layer
    l's own hidden states; shape = (B, h, n) of a flag tensor.  Returns the list
    of flag tensors the layers' attention uses, one per layer.  The last layer's
    own gate has no consumer and is not evaluated."""
    if first_gated < 1:
        raise ValueError("the first layer has no previous layer to take flags from")
    used = []
    for l in range(len(gate_fns)):
        if l < first_gated:
            used.append(np.ones(shape, dtype=np.uint8))
        else:
            used.append(gate_fns[l - 1]()[1])
    return used


# --------------------------------------------------------------------------
# Step 2: selective caching.  Sec. 3.3, sentence after Eq. 4: k_i^(t), v_i^(t)
# are retained iff AG(X)_i^(t) = 1.
# --------------------------------------------------------------------------
def retained_indices(flags_i):
    """Ascending list of token positions whose flag is 1, for one head."""
    return np.asarray([t for t in range(len(flags_i)) if flags_i[t] == 1],
                      dtype=np.int64)


def exclusive_counts(flags_i):
    """P[j] = #{t < j : flag[t] = 1} for j = 0..n (so P[n] is the retained
    length).  Written as the definition, one count per j."""
    n = len(flags_i)
    f = np.asarray(flags_i, dtype=np.int64)
    return np.asarray([int(f[:j].sum()) for j in range(n + 1)], dtype=np.int64)


def compact_kv(K, V, flags, window=1):
    """Ragged cache after prefill: cache[b][i] = dict(k=[L, D], v=[L, D],
    idx=[L]) holding exactly the retained tokens in ascending position.
    K, V [B, h, n, D] are copied bit-for-bit (dtype preserved).

    With a recent-token window (Appendix, Table 6: the `window` most recent
    tokens, the current one included, are visible whatever their flags) the
    slab also remembers the last window - 1 tokens as a list "recent" of
    (k, v, flag), oldest first: the next window - 1 queries still see them."""
    K = np.asarray(K)
    V = np.asarray(V)
    B, h, n = flags.shape
    cache = []
    for b in range(B):
        row = []
        for i in range(h):
            idx = retained_indices(flags[b, i])
            c = {"k": K[b, i][idx].copy(), "v": V[b, i][idx].copy(), "idx": idx}
            if window > 1:
                c["recent"] = [(K[b, i][t].copy(), V[b, i][t].copy(), int(flags[b, i][t]))
                               for t in range(max(0, n - (window - 1)), n)]
            row.append(c)
        cache.append(row)
    return cache


def project_kv(X, Wk, Wv, kv_heads):
    """Keys and values of the layer from its hidden states, Eq. 2: K_i = X W^K_i,
    V_i = X W^V_i, head i taking columns [i D, (i + 1) D) of the "in x out"
    weight.  X [B, n, d], Wk, Wv [d, kv_heads * D] -> K, V [B, kv_heads, n, D]
    in float64 (no rounding to a storage type)."""
    X, Wk, Wv = _as_f64(X), _as_f64(Wk), _as_f64(Wv)
    B, n, d = X.shape
    D = Wk.shape[1] // kv_heads
    K = np.empty((B, kv_heads, n, D), dtype=F64)
    V = np.empty((B, kv_heads, n, D), dtype=F64)
    for b in range(B):
        for i in range(kv_heads):
            K[b, i] = X[b] @ Wk[:, i * D:(i + 1) * D]
            V[b, i] = X[b] @ Wv[:, i * D:(i + 1) * D]
    return K, V


def project_q(X, Wq, heads):
    """Queries of the layer, Eq. 2: Q_i = X W^Q_i, head i taking columns
    [i D, (i + 1) D) of the "in x out" weight.  X [B, n, d], Wq [d, heads * D]
    -> Q [B, heads, n, D] in float64."""
    X, Wq = _as_f64(X), _as_f64(Wq)
    B, n, d = X.shape
    D = Wq.shape[1] // heads
    Q = np.empty((B, heads, n, D), dtype=F64)
    for b in range(B):
        for i in range(heads):
            for t in range(n):
                Q[b, i, t] = X[b, t] @ Wq[:, i * D:(i + 1) * D]
    return Q


def mha_output(H, Wo, X_res=None):
    """The layer's output, Eq. 1: MHA(X) = [H_1(X), ..., H_h(X)] W^O, the heads' outputs concatenated
    along the feature axis (head i in columns [i D, (i + 1) D)) and multiplied by W^O in R^{h D x d}.
    H [B, h, n, D] (the O of prefill attention), Wo [h D, d] -> [B, n, d] in float64.
    With X_res [B, n, d] the Transformer's skip connection is added: X_res + MHA(X) (the paper's Eq. 1
    stops at MHA(X); a stack of attention layers feeds this sum to the next layer)."""
    H, Wo = _as_f64(H), _as_f64(Wo)
    B, h, n, D = H.shape
    Y = np.zeros((B, n, Wo.shape[1]), dtype=F64)
    for b in range(B):
        for t in range(n):
            concat = np.concatenate([H[b, i, t] for i in range(h)])      # [h D]
            Y[b, t] = concat @ Wo
    if X_res is not None:
        Y = Y + _as_f64(X_res)
    return Y


def project_and_cache(X, Wk, Wv, flags):
    """Eq. 2's projection followed by selective caching (Sec. 3.3): the dense
    K, V [B, h, n, D] and the ragged cache of the retained rows, as
    (K, V, compact_kv(K, V, flags))."""
    K, V = project_kv(X, Wk, Wv, flags.shape[1])
    return K, V, compact_kv(K, V, flags)


# --------------------------------------------------------------------------
# Step 3: prefill attention under the eviction mask.  Eq. 2 and Eq. 5.
# --------------------------------------------------------------------------
def eviction_mask(flags_i, rows=None, window=1):
    """M_i[j, t] of Eq. 5 for one head: 0 above the diagonal (j < t), 1 on it,
    AG(X)_i^(t) below it.  j indexes queries (rows), t keys (columns).
    `rows` selects a subset of query positions; default all.

    window = number of recent tokens always retained, the current one included
    (Appendix, Table 6: 1 in the method as published, "only the current token
    is retained", 5 and 10 in settings (6-1), (6-2)): the diagonal widens to
    the band 0 <= j - t < window."""
    f = np.asarray(flags_i).astype(np.int64)
    n = f.shape[0]
    j = (np.arange(n) if rows is None else np.asarray(rows, dtype=np.int64))[:, None]
    t = np.arange(n)[None, :]
    below = np.broadcast_to(f[None, :], (j.shape[0], n))
    return np.where(j < t, 0, np.where(j - t < window, 1, below))


def prefill_head(Q_i, K_i, V_i, flags_i, scale=None, rows=None, window=1):
    """H_i = Softmax(Q K^T / sqrt(d_k) - INF (1 - M_i)) V for one head
    (Eq. 2) with M_i from Eq. 5.  Q_i, K_i, V_i [n, D] -> [len(rows), D]."""
    Q_i, K_i, V_i = map(_as_f64, (Q_i, K_i, V_i))
    D = Q_i.shape[1]
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    Qs = Q_i if rows is None else Q_i[np.asarray(rows, dtype=np.int64)]
    S = (Qs @ K_i.T) * scale
    M = eviction_mask(flags_i, rows, window)
    S = np.where(M == 1, S, -np.inf)
    A = softmax_rows(S)
    return A @ V_i


def kv_head_of(i, h, h_kv):
    """Grouped-query attention: h query heads share h_kv key/value heads, consecutive query heads
    in groups of h / h_kv (the paper's Mistral runs; h_kv = h is ordinary multi-head attention).
    The cache, and therefore the flag, belongs to the key/value head."""
    assert h % h_kv == 0
    return i // (h // h_kv)


def prefill_attention(Q, K, V, flags, scale=None, window=1):
    """All heads of all sequences: Q [B, h, n, D], K, V [B, h_kv, n, D], flags [B, h_kv, n]
    -> [B, h, n, D] float64.  Query head i reads key/value head kv_head_of(i) and its flags."""
    B, h, n, D = np.asarray(Q).shape
    h_kv = np.asarray(K).shape[1]
    O = np.empty((B, h, n, D), dtype=F64)
    for b in range(B):
        for i in range(h):
            g = kv_head_of(i, h, h_kv)
            O[b, i] = prefill_head(Q[b, i], K[b, g], V[b, g], flags[b, g], scale, window=window)
    return O


# --------------------------------------------------------------------------
# Step 4: decode over the retained cache + conditional append.  Sec. 3.1
# "decoding stage" (concatenate the new k, v with the cache, attend, update
# the cache), with the cache holding only retained tokens (Sec. 3.3) and the
# j = t case of Eq. 5 (a token always attends to itself).
# --------------------------------------------------------------------------
def decode_head(q, k_new, v_new, k_cache, v_cache, scale=None):
    """One query against the retained rows followed by its own (k, v)."""
    q, k_new, v_new = map(_as_f64, (q, k_new, v_new))
    D = q.shape[0]
    if scale is None:
        scale = 1.0 / math.sqrt(D)
    Kall = np.concatenate([_as_f64(k_cache).reshape(-1, D), k_new[None, :]], axis=0)
    Vall = np.concatenate([_as_f64(v_cache).reshape(-1, D), v_new[None, :]], axis=0)
    s = (Kall @ q) * scale
    a = softmax_rows(s[None, :])[0]
    return a @ Vall


def decode_attention(q, k_new, v_new, cache, scale=None):
    """q [B, h, D]; k_new, v_new [B, h_kv, D]; cache as returned by compact_kv (one slab per
    key/value head) -> [B, h, D].  Query head i reads slab kv_head_of(i).  A slab with a
    recent-token window also shows the query its evicted recent tokens (the retained ones are
    rows of the cache already)."""
    q = np.asarray(q)
    B, h, D = q.shape
    h_kv = np.asarray(k_new).shape[1]
    o = np.empty((B, h, D), dtype=F64)
    for b in range(B):
        for i in range(h):
            g = kv_head_of(i, h, h_kv)
            c = cache[b][g]
            kc, vc = c["k"], c["v"]
            evicted = [(k, v) for k, v, f in c.get("recent", []) if f == 0]
            if evicted:
                kc = np.concatenate([_as_f64(kc).reshape(-1, D)] + [_as_f64(k)[None, :] for k, _ in evicted], axis=0)
                vc = np.concatenate([_as_f64(vc).reshape(-1, D)] + [_as_f64(v)[None, :] for _, v in evicted], axis=0)
            o[b, i] = decode_head(q[b, i], k_new[b, g], v_new[b, g], kc, vc, scale)
    return o


def cache_append(cache, k_new, v_new, flag_new, window=1):
    """Append (k_new, v_new)[b, i] to slab (b, i) iff flag_new[b, i] = 1.
    Bit-for-bit copy; mutates and returns `cache`.  With a recent-token window
    the token also joins the slab's recent list, whose oldest entry leaves
    once the list holds window - 1 tokens."""
    k_new = np.asarray(k_new)
    v_new = np.asarray(v_new)
    B, h = flag_new.shape
    for b in range(B):
        for i in range(h):
            if flag_new[b, i] == 1:
                c = cache[b][i]
                c["k"] = np.concatenate([c["k"], k_new[b, i][None, :]], axis=0)
                c["v"] = np.concatenate([c["v"], v_new[b, i][None, :]], axis=0)
            if window > 1:
                c = cache[b][i]
                c["recent"] = (c.get("recent", []) + [(k_new[b, i].copy(), v_new[b, i].copy(), int(flag_new[b, i]))])[-(window - 1):]
    return cache


def cache_lengths(cache):
    return np.asarray([[c["k"].shape[0] for c in row] for row in cache], dtype=np.int64)
