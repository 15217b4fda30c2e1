"""Parity of ag_kv_project_cache with the oracle: the key/value projection of Eq. 2 whose
epilogue writes the retained rows straight into the ragged cache (Sec. 3.3).

The dense K, V are compared with the oracle's float64 projection element by element (one
rounding to bfloat16 plus float32 summation error); lengths and the positions of the cached
rows are bit-exact against the oracle's cache (a cached row must be the bit pattern of the
dense row at the oracle's r-th retained position); at the full layer size the dense outputs
are compared on sampled (head, token) rows the oracle computes one by one."""
import numpy as np
import pytest
import torch

import agtest as T
from oracle import ag_oracle as orc
from paper_2410_12876_b200 import binding as ag
from paper_2410_12876_b200 import inputs
from paper_2410_12876_b200.inputs import LayerShape

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    T.ensure_built()


def _close_to_rounded(got, ref, what):
    """|got - ref| <= half a bfloat16 ulp of ref (2^-8 |ref| bounds it) + float32 summation slack."""
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, what
    if got.size == 0:
        return
    assert np.all(np.isfinite(got)), what
    excess = np.abs(got - ref) - (2.0 ** -8 * np.abs(ref) + 1e-5)
    assert np.max(excess) <= 0, f"{what}: {np.max(excess):.3e} beyond one rounding"


def _flags(shape, seed):
    """Per-head Bernoulli flags with rates spread over [0, 1]; head 0 keeps nothing, head 1 everything."""
    rng = np.random.default_rng(seed)
    B, h, n = shape.batch, shape.kvh, shape.seq
    rate = rng.uniform(0.05, 0.95, size=(B, h, 1))
    f = (rng.random((B, h, n)) < rate).astype(np.uint8)
    f[:, 0] = 0
    if h > 1:
        f[:, 1] = 1
    return f


def gpu_project_cache(shape, X, W, flags, cap=None, with_q=False):
    """The fused projection on buffers that hold nothing of a previous call; with_q: the call that
    projects the queries too (Q is then the last item returned)."""
    desc = ag.make_desc(shape)
    B, h, n, D = shape.batch, shape.kvh, shape.seq, shape.head_dim
    if cap is None:
        cap = [n] * (B * h)
    cache = ag.RaggedCache.allocate(shape, cap, DEV)
    prefix = torch.full((B, h, n + 1), -1, dtype=torch.int32, device=DEV)
    idx = torch.full((B, h, n), -1, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    cache.len.fill_(-7)                                    # the call sets the lengths itself
    K = torch.full((B, h, n, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    V = torch.full_like(K, float("nan"))
    if with_q:
        Q = torch.full((B, shape.heads, n, D), float("nan"), dtype=torch.bfloat16, device=DEV)
        ag.ag_qkv_project_cache(desc, X, W["Wq"], W["Wk"], W["Wv"], flags, cache, prefix, idx, Q, K, V, status)
        torch.cuda.synchronize()
        return cache, prefix, idx, status, K, V, Q
    ag.ag_kv_project_cache(desc, X, W["Wk"], W["Wv"], flags, cache, prefix, idx, K, V, status)
    torch.cuda.synchronize()
    return cache, prefix, idx, status, K, V


def _check(shape, seed, cap=None, with_q=False):
    X = inputs.hidden_states(shape, seed, DEV)
    W = inputs.layer_weights(shape, seed + 10, DEV)
    fl = _flags(shape, seed + 20)
    flags = torch.from_numpy(fl).to(DEV)
    cache, prefix, idx, status, K, V, *rest = gpu_project_cache(shape, X, W, flags, cap, with_q)
    if with_q:
        _close_to_rounded(T.f64(rest[0]), orc.project_q(T.f64(X), T.f64(W["Wq"]), shape.heads), "dense Q")
    Kr, Vr, ocache = orc.project_and_cache(T.f64(X), T.f64(W["Wk"]), T.f64(W["Wv"]), fl)
    _close_to_rounded(T.f64(K), Kr, "dense K")
    _close_to_rounded(T.f64(V), Vr, "dense V")
    L = orc.cache_lengths(ocache).reshape(-1)
    capv = cache.cap.cpu().numpy()
    fits = L <= capv
    assert np.array_equal(cache.len.cpu().numpy(), np.where(fits, L, 0))
    assert int(status.item()) == (0 if fits.all() else ag.AG_DEV_OVERFLOW)
    kd, vd = T.bits(K), T.bits(V)
    kr, vr = T.bits(cache.k_rows), T.bits(cache.v_rows)
    off = cache.row_off.cpu().numpy()
    pre, ix = prefix.cpu().numpy(), idx.cpu().numpy()
    for b in range(shape.batch):
        for i in range(shape.kvh):
            s = b * shape.kvh + i
            pos = ocache[b][i]["idx"]                      # the oracle's retained positions
            assert np.array_equal(pre[b, i], orc.exclusive_counts(fl[b, i])), (b, i)
            assert np.array_equal(ix[b, i, :L[s]], pos) and np.all(ix[b, i, L[s]:] == -1), (b, i)
            if fits[s]:
                assert np.array_equal(kr[off[s]:off[s] + L[s]], kd[b, i][pos]), (b, i)
                assert np.array_equal(vr[off[s]:off[s] + L[s]], vd[b, i][pos]), (b, i)
                _close_to_rounded(T.f64(cache.k_rows[off[s]:off[s] + L[s]]), ocache[b][i]["k"], "cached keys")
                _close_to_rounded(T.f64(cache.v_rows[off[s]:off[s] + L[s]]), ocache[b][i]["v"], "cached values")
                # rows of the slab past its length were not written
                assert not kr[off[s] + L[s]:off[s] + capv[s]].any()
            else:
                assert not kr[off[s]:off[s] + capv[s]].any() and not vr[off[s]:off[s] + capv[s]].any()
    assert ag.ag_device_wait_timeouts() == 0
    return cache, prefix, K, V, fl


# (batch, seq, hidden, heads, head_dim, gate_heads, gate_head_dim, dtype)
CASES = {
    "two_heads_per_tile": LayerShape(2, 256, 512, 4, 128, 2, 128, "bf16"),
    "k_tail": LayerShape(1, 384, 520, 4, 128, 2, 128, "bf16"),                 # hidden not a multiple of 64
    "odd_heads": LayerShape(2, 128, 256, 3, 128, 1, 128, "bf16"),              # one head per tile
    "two_subtiles": LayerShape(1, 1280, 256, 16, 128, 2, 128, "bf16"),         # CTA pairs; the last pair tile has two of four sub-tiles
    "two_subtiles_odd_rows": LayerShape(1, 1152, 192, 18, 128, 2, 128, "bf16"),  # CTA pairs; nine sub-tiles: one CTA of the last pair has none
    "subtiles_of_two_sequences": LayerShape(3, 384, 128, 20, 128, 2, 128, "bf16"),
    "split_last_wave": LayerShape(1, 2560, 128, 16, 128, 2, 128, "bf16"),      # 80 pair tiles on 74 pairs: 6 are halved
    "split_last_wave_odd_rows": LayerShape(1, 2432, 128, 16, 128, 2, 128, "bf16"),
    "grouped_query": LayerShape(2, 256, 256, 8, 128, 2, 128, "bf16", kv_heads=2),
    "three_bands_of_row_tiles": LayerShape(1, 4864, 128, 2, 128, 1, 128, "bf16"),    # 38 row tiles: bands of 16, 16, 6
    "two_sequences_of_19_subtiles": LayerShape(2, 2432, 128, 8, 128, 2, 128, "bf16"),  # 38 sub-tiles: 10 pair tiles of rows, the last half empty
    "two_bands_of_pair_tiles": LayerShape(1, 8704, 128, 4, 128, 2, 128, "bf16"),     # 68 sub-tiles: bands of 16 pair tiles and 1
    "one_sequence_ragged_end": LayerShape(1, 333, 256, 4, 128, 2, 128, "bf16"),      # n not a multiple of 16
    "one_sequence_short": LayerShape(1, 48, 128, 6, 128, 2, 128, "bf16"),            # less than one tile
    "one_sequence_long_ragged": LayerShape(1, 2500, 128, 16, 128, 2, 128, "bf16"),   # split last wave, ragged end
    "batch_ragged_end": LayerShape(3, 200, 256, 4, 128, 2, 128, "bf16"),             # every sequence ends inside its last sub-tile
    "batch_ragged_two_subtiles": LayerShape(5, 333, 128, 20, 128, 2, 128, "bf16"),   # pair tiles whose sub-tiles belong to several sequences, ragged ends, halved last wave
}


@pytest.mark.parametrize("name", list(CASES))
def test_projection_and_cache(name):
    _check(CASES[name], 900)


@pytest.mark.parametrize("name", ["two_heads_per_tile", "k_tail", "odd_heads", "subtiles_of_two_sequences",
                                  "split_last_wave_odd_rows", "grouped_query", "one_sequence_ragged_end",
                                  "batch_ragged_end", "batch_ragged_two_subtiles"])
def test_projection_with_queries(name):
    """ag_qkv_project_cache: Q against the oracle's query projection, K, V and the cache as without it."""
    _check(CASES[name], 940, with_q=True)


def test_slab_too_small_is_skipped_and_reported():
    shape = CASES["two_heads_per_tile"]
    cap = [shape.seq] * (shape.batch * shape.kvh)
    cap[1] = 17                                            # head 1 keeps every token
    cap[5] = shape.seq - 1
    _check(shape, 910, cap)


def test_feeds_prefill_and_decode():
    """flags -> fused projection -> prefill attention and a decode step, against the
    oracle run on the projected K, V the library wrote."""
    shape = LayerShape(1, 512, 512, 4, 128, 2, 128, "bf16")
    cache, prefix, K, V, fl = _check(shape, 920)
    Q = inputs.randn((1, 4, 512, 128), 921, DEV, torch.bfloat16)
    flags = torch.from_numpy(fl).to(DEV)
    O = T.gpu_prefill(shape, Q, K, V, flags, cache, prefix)
    ref = orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), fl)
    T.check_close(T.f64(O), ref, "bf16", "prefill after the fused projection")
    q, kn, vn, fn = inputs.decode_inputs(shape, 922, 0, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=True)
    oc = orc.compact_kv(T.f64(K), T.f64(V), fl)
    ref = orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), oc)
    T.check_close(T.f64(o), ref, "bf16", "decode after the fused projection")


@pytest.mark.parametrize("w", [5, 10])
def test_recent_window_ring_filled_by_the_projection(w):
    """With a recent-token window the call leaves the ring as compaction leaves it: ring contents against
    the oracle's list, then prefill under the band mask and decode steps that read and move the ring."""
    shape = LayerShape(2, 256, 256, 4, 128, 2, 128, "bf16", recent_window=w)
    R = w - 1
    X = inputs.hidden_states(shape, 950 + w, DEV)
    W = inputs.layer_weights(shape, 960 + w, DEV)
    fl = _flags(shape, 970 + w)
    flags = torch.from_numpy(fl).to(DEV)
    steps = w + 2
    cache, prefix, idx, status, K, V, Q = gpu_project_cache(shape, X, W, flags, [shape.seq + steps] * 8, with_q=True)
    obits = orc.compact_kv(T.bits(K), T.bits(V), fl, window=w)          # the oracle's ring of the rows the call wrote
    live = cache.recent_live.cpu().numpy()
    rk = T.bits(cache.recent_k)
    got = [sorted(rk[s, r].tobytes() for r in range(R) if live[s, r]) for s in range(live.shape[0])]
    want = [sorted(np.ascontiguousarray(k).tobytes() for k, _, f in c["recent"] if f == 0) for row in obits for c in row]
    assert got == want
    assert np.array_equal(cache.pos.cpu().numpy(), np.full(8, shape.seq))
    O = T.gpu_prefill(shape, Q, K, V, flags, cache, prefix)
    T.check_close(T.f64(O), orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), fl, window=w), "bf16", "prefill")
    ocache = orc.compact_kv(T.f64(K), T.f64(V), fl, window=w)
    for s in range(steps):
        q, kn, vn, fn = inputs.decode_inputs(shape, 980 + w, s, DEV, keep_new=0.4)
        o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=True)
        T.check_close(T.f64(o), orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache), "bf16", f"decode {s}")
        orc.cache_append(ocache, T.f64(kn), T.f64(vn), fn.cpu().numpy(), window=w)
    assert int(status.item()) == 0


@pytest.mark.parametrize("with_q", [False, True])
def test_full_size_layer_sampled(with_q):
    """The 7B-shaped layer in the launch configurations bench.py times (keys and values; queries, keys and
    values): sampled dense rows against the oracle, lengths and every cached row against the flags."""
    shape = inputs.PREFILL7B
    X = inputs.hidden_states(shape, 2000, DEV)
    W = inputs.layer_weights(shape, 2010, DEV)
    fl = _flags(shape, 930)
    flags = torch.from_numpy(fl).to(DEV)
    cache, prefix, idx, status, K, V, Q = gpu_project_cache(shape, X, W, flags, with_q=with_q)[:7] if with_q else \
        (*gpu_project_cache(shape, X, W, flags), None)
    assert int(status.item()) == 0
    L = fl.sum(axis=2, dtype=np.int64).reshape(-1)
    assert np.array_equal(cache.len.cpu().numpy(), L)
    want = np.concatenate([np.zeros((1, shape.heads, 1), dtype=np.int64), np.cumsum(fl, axis=2, dtype=np.int64)], axis=2)
    assert np.array_equal(prefix.cpu().numpy(), want)
    Xf, Wk, Wv, Wq = T.f64(X)[0], T.f64(W["Wk"]), T.f64(W["Wv"]), T.f64(W["Wq"])
    rng = np.random.default_rng(931)
    D = shape.head_dim
    for i in range(shape.heads):
        rows = np.unique(np.concatenate([[0, 127, 128, shape.seq - 1], rng.integers(0, shape.seq, 12)]))
        _close_to_rounded(T.f64(K[0, i][torch.from_numpy(rows).to(DEV)]), Xf[rows] @ Wk[:, i * D:(i + 1) * D], "K")
        _close_to_rounded(T.f64(V[0, i][torch.from_numpy(rows).to(DEV)]), Xf[rows] @ Wv[:, i * D:(i + 1) * D], "V")
        if with_q:
            _close_to_rounded(T.f64(Q[0, i][torch.from_numpy(rows).to(DEV)]), Xf[rows] @ Wq[:, i * D:(i + 1) * D], "Q")
    off = cache.row_off.cpu().numpy()
    kd, vd, kr, vr = T.bits(K), T.bits(V), T.bits(cache.k_rows), T.bits(cache.v_rows)
    for i in range(shape.heads):
        pos = np.flatnonzero(fl[0, i])
        assert np.array_equal(kr[off[i]:off[i] + L[i]], kd[0, i][pos])
        assert np.array_equal(vr[off[i]:off[i] + L[i]], vd[0, i][pos])
    assert ag.ag_device_wait_timeouts() == 0


def test_rejects_what_it_has_no_kernel_for():
    shape = CASES["two_heads_per_tile"]
    X = inputs.hidden_states(shape, 1, DEV)
    W = inputs.layer_weights(shape, 2, DEV)
    flags = torch.ones(shape.batch, shape.kvh, shape.seq, dtype=torch.uint8, device=DEV)
    cache, prefix, idx, status, K, V = gpu_project_cache(shape, X, W, flags)
    for bad in (shape.with_(head_dim=64), shape.with_(dtype="f32"), shape.with_(hidden=516),
                shape.with_(recent_window=5)):              # the last one: a window, and a cache without a ring
        with pytest.raises(ag.AgError) as e:
            ag.ag_kv_project_cache(ag.make_desc(bad), X, W["Wk"], W["Wv"], flags, cache, prefix, idx, K, V, status)
        assert e.value.status in (ag.AG_ERR_UNSUPPORTED, ag.AG_ERR_INVALID_ARG)
    with pytest.raises(ag.AgError) as e:
        ag.ag_kv_project_cache(ag.make_desc(shape), X, W["Wk"], None, flags, cache, prefix, idx, K, V, status)
    assert e.value.status == ag.AG_ERR_INVALID_ARG
    with pytest.raises(ag.AgError) as e:
        ag.ag_qkv_project_cache(ag.make_desc(shape), X, None, W["Wk"], W["Wv"], flags, cache, prefix, idx, K, K, V, status)
    assert e.value.status == ag.AG_ERR_INVALID_ARG
