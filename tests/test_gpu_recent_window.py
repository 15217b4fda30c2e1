"""Recent-token window (Appendix, Table 6: the w most recent tokens stay visible whatever their
flags) on the GPU against the oracle: prefill under the band mask, the ring of recent tokens that
compaction leaves, decode steps that read it and appends that move it."""
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

SHAPES = {
    "tiny_f32": inputs.TINY,
    "bf16_tc": LayerShape(2, 333, 512, 8, 128, 2, 128, "bf16"),
    "bf16_d64": LayerShape(1, 200, 256, 4, 64, 2, 64, "bf16"),
    "f32_d128": LayerShape(1, 150, 128, 3, 128, 1, 128, "f32"),
    "bf16_gqa": LayerShape(2, 300, 512, 8, 128, 2, 128, "bf16", kv_heads=2),
    "bf16_many_slabs": LayerShape(9, 140, 256, 8, 128, 2, 128, "bf16"),      # decode through the workspace
}


@pytest.fixture(scope="module", autouse=True)
def _lib():
    T.ensure_built()


def _flags(shape, seed):
    """Bernoulli flags with one head that keeps everything and one that keeps nothing."""
    f = inputs.bernoulli_flags((shape.batch, shape.kvh, shape.seq), 0.4, seed)
    f[:, 0] = 1
    f[:, -1] = 0
    return f.to(DEV)


def _ring_as_lists(cache, shape, R):
    """Live ring entries of every slab as a sorted list of key rows (bit patterns), for comparison
    with the evicted entries of the oracle's recent list."""
    live = cache.recent_live.cpu().numpy()
    rk = T.bits(cache.recent_k)
    return [sorted(rk[s, r].tobytes() for r in range(R) if live[s, r]) for s in range(live.shape[0])]


def _oracle_ring(ocache):
    return [sorted(np.ascontiguousarray(k).tobytes() for k, _, f in c["recent"] if f == 0) for row in ocache for c in row]


@pytest.mark.parametrize("w", [2, 5, 10, 17])
@pytest.mark.parametrize("name", list(SHAPES))
def test_prefill_and_decode_under_a_window(name, w):
    shape = SHAPES[name].with_(recent_window=w)
    R = w - 1
    Q, K, V = inputs.qkv_gaussian(shape, 7000 + w, DEV)
    flags = _flags(shape, 7100 + w)
    steps = 2 * w + 3                                  # the ring turns over more than twice
    cap = [shape.seq + 2 * steps] * (shape.batch * shape.kvh)
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, cap=cap)
    T.check_compaction(shape, K, V, flags, cache, prefix, idx)           # what is cached for good is unchanged
    f_np = flags.cpu().numpy()
    ocache_bits = orc.compact_kv(T.bits(K), T.bits(V), f_np, window=w)
    assert _ring_as_lists(cache, shape, R) == _oracle_ring(ocache_bits)
    assert np.array_equal(cache.pos.cpu().numpy(), np.full(shape.batch * shape.kvh, shape.seq))

    O = T.gpu_prefill(shape, Q, K, V, flags, cache, prefix)
    O_ref = orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), f_np, window=w)
    T.check_close(T.f64(O), O_ref, shape.dtype, "prefill")
    # the window matters on these inputs: the published mask gives something else
    assert np.max(np.abs(O_ref - orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), f_np))) > 0.05

    ocache = orc.compact_kv(T.f64(K), T.f64(V), f_np, window=w)
    for fused in (False, True):
        for s in range(steps):
            q, kn, vn, fn = inputs.decode_inputs(shape, 7300 + 100 * fused, s, DEV, keep_new=0.4)
            o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=fused)
            o_ref = orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache)
            T.check_close(T.f64(o), o_ref, shape.dtype, f"decode step {s} ({'one call' if fused else 'two calls'})")
            orc.cache_append(ocache, T.f64(kn), T.f64(vn), fn.cpu().numpy(), window=w)
            orc.cache_append(ocache_bits, T.bits(kn), T.bits(vn), fn.cpu().numpy(), window=w)
        assert np.array_equal(cache.len.cpu().numpy(), orc.cache_lengths(ocache).reshape(-1))
        assert _ring_as_lists(cache, shape, R) == _oracle_ring(ocache_bits)
    assert int(status.item()) == 0
    assert np.array_equal(cache.pos.cpu().numpy(), np.full(shape.batch * shape.kvh, shape.seq + 2 * steps))


@pytest.mark.parametrize("n", [1, 3, 9])
def test_prompt_shorter_than_the_window(n):
    w = 10
    shape = LayerShape(2, n, 256, 4, 128, 2, 128, "bf16", recent_window=w)
    Q, K, V = inputs.qkv_gaussian(shape, 7500 + n, DEV)
    flags = inputs.bernoulli_flags((shape.batch, shape.heads, n), 0.3, 7510 + n).to(DEV)
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, cap=[n + 16] * (shape.batch * shape.heads))
    f_np = flags.cpu().numpy()
    O = T.gpu_prefill(shape, Q, K, V, flags, cache, prefix)
    # the window covers the whole prompt: ordinary causal attention, whatever the flags
    T.check_close(T.f64(O), orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), np.ones_like(f_np)), "bf16", "prefill")
    ocache = orc.compact_kv(T.f64(K), T.f64(V), f_np, window=w)
    for s in range(16):
        q, kn, vn, fn = inputs.decode_inputs(shape, 7600, s, DEV, keep_new=0.3)
        o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=bool(s % 2))
        T.check_close(T.f64(o), orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache), "bf16", f"decode step {s}")
        orc.cache_append(ocache, T.f64(kn), T.f64(vn), fn.cpu().numpy(), window=w)


def test_window_of_one_is_the_published_method_bit_for_bit():
    base = SHAPES["bf16_tc"]
    Q, K, V = inputs.qkv_gaussian(base, 7700, DEV)
    flags = _flags(base, 7710)
    outs = []
    for w in (0, 1):
        shape = base.with_(recent_window=w)
        cache, prefix, _, _ = T.gpu_compact(shape, K, V, flags)
        outs.append(T.gpu_prefill(shape, Q, K, V, flags, cache, prefix))
        assert cache.recent_k is None
    assert np.array_equal(T.bits(outs[0]), T.bits(outs[1]))


def test_window_argument_checks():
    base = SHAPES["bf16_tc"]
    Q, K, V = inputs.qkv_gaussian(base, 7800, DEV)
    flags = _flags(base, 7810)
    B, h, n = base.batch, base.heads, base.seq
    prefix = torch.empty(B, h, n + 1, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    with_ring = ag.RaggedCache.allocate(base.with_(recent_window=5), [n] * (B * h), DEV)
    no_ring = ag.RaggedCache.allocate(base, [n] * (B * h), DEV)

    def compact(desc, cache):
        ag.ag_compact_kv(desc, K, V, flags, cache, prefix, None, status, ag.workspace(desc, ag.AG_CALL_COMPACT))

    with pytest.raises(ag.AgError) as e:                       # longer than the library's ring
        compact(ag.make_desc(base.with_(recent_window=18)), with_ring)
    assert e.value.status == ag.AG_ERR_UNSUPPORTED
    with pytest.raises(ag.AgError) as e:
        compact(ag.make_desc(base.with_(recent_window=-1)), with_ring)
    assert e.value.status == ag.AG_ERR_INVALID_ARG
    with pytest.raises(ag.AgError) as e:                       # a window needs the cache's ring
        compact(ag.make_desc(base.with_(recent_window=5)), no_ring)
    assert e.value.status == ag.AG_ERR_INVALID_ARG
    q, kn, vn, _ = inputs.decode_inputs(base, 7820, 0, DEV)
    o = torch.empty_like(q)
    with pytest.raises(ag.AgError) as e:                       # the no-allocation entry does not read the ring
        ag.ag_decode_attn_noalloc(ag.make_desc(base.with_(recent_window=5)), q, kn, vn, with_ring, 0.0, o)
    assert e.value.status == ag.AG_ERR_UNSUPPORTED
    torch.cuda.synchronize()


@pytest.mark.parametrize("w", [5, 10])
def test_window_with_per_sequence_lengths(w):
    """A ragged batch under a recent-token window: the ring of a sequence takes the last tokens of
    its own prompt, and every valid row of prefill and of the decode steps equals what the sequence
    alone gives (the oracle runs each sequence on its own, without padding)."""
    shape = LayerShape(3, 300, 256, 4, 128, 2, 128, "bf16", recent_window=w)
    B, h, n = shape.batch, shape.heads, shape.seq
    lens = np.array([300, 7, 131], dtype=np.int32)              # full, shorter than the window, ragged
    lens_dev = torch.from_numpy(lens).to(DEV)
    Q, K, V = inputs.qkv_gaussian(shape, 7900 + w, DEV)
    f = inputs.bernoulli_flags((B, h, n), 0.5, 7910 + w).numpy()
    for b, L in enumerate(lens):
        f[b, :, L:] = 0                                        # what the gate calls guarantee for padding
    fl = torch.from_numpy(f).to(DEV)
    desc = ag.make_desc(shape, lens_dev)
    steps = w + 2
    cache = ag.RaggedCache.allocate(shape, [n + steps] * (B * h), DEV)
    prefix = torch.empty(B, h, n + 1, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ag.ag_compact_kv(desc, K, V, fl, cache, prefix, None, status, ag.workspace(desc, ag.AG_CALL_COMPACT))
    O = torch.full_like(Q, float("nan"))
    ag.ag_prefill_attn(desc, Q, K, V, fl, cache, prefix, 0.0, O, ag.workspace(desc, ag.AG_CALL_PREFILL))
    torch.cuda.synchronize()
    assert cache.pos.cpu().tolist() == np.repeat(lens, h).tolist()
    Qf, Kf, Vf = T.f64(Q), T.f64(K), T.f64(V)
    alone = []
    for b, L in enumerate(lens):
        ref = orc.prefill_attention(Qf[b:b + 1, :, :L], Kf[b:b + 1, :, :L], Vf[b:b + 1, :, :L], f[b:b + 1, :, :L], window=w)
        T.check_close(T.f64(O)[b, :, :L], ref[0], "bf16", f"prefill of sequence {b}")
        alone.append(orc.compact_kv(Kf[b:b + 1, :, :L], Vf[b:b + 1, :, :L], f[b:b + 1, :, :L], window=w))
    ws = ag.workspace(desc, ag.AG_CALL_DECODE)
    for step in range(steps):
        q, kn, vn, fn = inputs.decode_inputs(shape, 7920 + w, step, DEV, keep_new=0.5)
        o = torch.full_like(q, float("nan"))
        ag.ag_decode_step(desc, q, kn, vn, fn, cache, 0.0, o, status, ws)
        for b in range(B):
            ref = orc.decode_attention(T.f64(q[b:b + 1]), T.f64(kn[b:b + 1]), T.f64(vn[b:b + 1]), alone[b])
            T.check_close(T.f64(o[b:b + 1]), ref, "bf16", f"decode step {step}, sequence {b}")
            orc.cache_append(alone[b], T.f64(kn[b:b + 1]), T.f64(vn[b:b + 1]), fn[b:b + 1].cpu().numpy(), window=w)
    assert int(status.item()) == 0
