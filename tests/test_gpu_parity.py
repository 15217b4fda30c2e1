"""GPU-vs-oracle parity of every call of the C boundary, element by element, at
sizes the oracle finishes in seconds but that span several tiles and a ragged
tail.  The oracle never receives anything the GPU produced: flags for the
compaction / attention tests are synthetic, and in the end-to-end test each
side is driven by its own gate, whose flags must coincide."""
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

SMALL_BF16 = LayerShape(2, 333, 512, 8, 128, 2, 128, "bf16")
SMALL_BF16_D64 = LayerShape(1, 200, 256, 4, 64, 2, 64, "bf16")
SMALL_F32_D128 = LayerShape(1, 150, 128, 3, 128, 1, 128, "f32")
SHAPES = {"tiny": inputs.TINY, "bf16": SMALL_BF16, "bf16_d64": SMALL_BF16_D64, "f32_d128": SMALL_F32_D128}


@pytest.fixture(scope="module", autouse=True)
def _lib():
    T.ensure_built()


def _layer_inputs(shape, seed):
    X = inputs.hidden_states(shape, seed, DEV)
    W = inputs.layer_weights(shape, seed + 10, DEV)
    # larger gate output weights so that scores spread over a useful range at small n
    W["Wo_g"] = inputs.randn(tuple(W["Wo_g"].shape), seed + 17, DEV, shape.torch_dtype, 0.5)
    Q, K, V = inputs.project_qkv(shape, X, W)
    return X, W, Q, K, V


def _calibrated_gamma(shape, X, W, keep):
    s0, _ = T.oracle_gate(shape, X, W, None)
    return inputs.calibrate_gamma(torch.from_numpy(s0), keep, float(np.float32(shape.tau))).to(DEV)


@pytest.mark.parametrize("name", list(SHAPES))
@pytest.mark.parametrize("causal", [1, 0])
def test_gate_scores_and_flags(name, causal):
    shape = SHAPES[name].with_(gate_causal=causal)
    X, W, *_ = _layer_inputs(shape, 100)
    keep = inputs.keep_targets_uniform(shape.heads, 5)
    gamma = _calibrated_gamma(shape, X, W, keep)
    scores, flags = T.gpu_gate(shape, X, W, gamma)
    s_ref, f_ref = T.oracle_gate(shape, X, W, gamma)
    err = np.max(np.abs(T.f64(scores) - s_ref))
    assert err < 1e-4, err
    excluded = T.check_flags(shape, flags, s_ref, f_ref, gamma)
    assert excluded < 0.2
    got_keep = flags.float().mean(dim=(0, 2)).cpu().numpy()
    assert np.max(np.abs(got_keep - keep)) < 0.05
    # scores output is optional; gamma = NULL means 0
    _, flags2 = T.gpu_gate(shape, X, W, gamma, want_scores=False)
    assert torch.equal(flags, flags2)
    s0, f0 = T.gpu_gate(shape, X, W, None)
    s0_ref, f0_ref = T.oracle_gate(shape, X, W, None)
    T.check_flags(shape, f0, s0_ref, f0_ref, None)


def test_gate_tau_other_than_half():
    shape = inputs.TINY.with_(tau=0.3)
    X, W, *_ = _layer_inputs(shape, 110)
    scores, flags = T.gpu_gate(shape, X, W, None)
    s_ref, f_ref = T.oracle_gate(shape, X, W, None)
    T.check_flags(shape, flags, s_ref, f_ref, None)
    assert 0.0 < f_ref.mean() < 1.0


def _flag_patterns(shape, seed):
    B, h, n = shape.batch, shape.heads, shape.seq
    f = inputs.bernoulli_flags((B, h, n), 0.5, seed).numpy()
    f[0, 0] = 1                        # all keep
    f[0, 1 % h] = 0                    # all evict
    if h > 2:
        f[0, 2] = 0
        f[0, 2, n - 1] = 1             # only the last token
    if h > 3:
        f[0, 3] = 0
        f[0, 3, 0] = 1                 # only the first token
    return torch.from_numpy(f).to(DEV)


@pytest.mark.parametrize("name,n", [("tiny", 128), ("bf16", 333), ("bf16", 1), ("bf16", 1024),
                                     ("bf16", 1025), ("bf16_d64", 2049), ("f32_d128", 150)])
@pytest.mark.parametrize("want_idx", [True, False])
def test_compaction_bit_exact(name, n, want_idx):
    shape = SHAPES[name].with_(seq=n)
    Q, K, V = inputs.qkv_gaussian(shape, 200 + n, DEV)
    flags = _flag_patterns(shape, 210 + n)
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, want_idx=want_idx)
    T.check_compaction(shape, K, V, flags, cache, prefix, idx)
    assert int(status.item()) == 0


def test_compaction_count_pass_then_tight_slabs():
    shape = SMALL_BF16
    desc = ag.make_desc(shape)
    Q, K, V = inputs.qkv_gaussian(shape, 220, DEV)
    flags = _flag_patterns(shape, 221)
    B, h, n = shape.batch, shape.heads, shape.seq
    probe = ag.RaggedCache.allocate(shape, [0] * (B * h), DEV)
    prefix = torch.empty(B, h, n + 1, dtype=torch.int32, device=DEV)
    idx = torch.empty(B, h, n, dtype=torch.int32, device=DEV)
    ag.ag_compact_kv(desc, None, None, flags, probe, prefix, idx, None, None)
    L = probe.len.cpu().numpy()
    assert np.array_equal(L, flags.cpu().numpy().reshape(B * h, n).sum(axis=1))
    cache, prefix2, idx2, status = T.gpu_compact(shape, K, V, flags, cap=(L + 3).tolist())
    T.check_compaction(shape, K, V, flags, cache, prefix2, idx2)
    assert torch.equal(prefix, prefix2) and int(status.item()) == 0


def test_compaction_overflow_is_reported_not_written():
    shape = SMALL_BF16_D64
    Q, K, V = inputs.qkv_gaussian(shape, 230, DEV)
    flags = torch.ones(shape.batch, shape.heads, shape.seq, dtype=torch.uint8, device=DEV)
    cap = [shape.seq, 10, shape.seq, shape.seq]
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, cap=cap)
    assert int(status.item()) & ag.AG_DEV_OVERFLOW
    assert cache.len.cpu().tolist() == [shape.seq, 0, shape.seq, shape.seq]
    off = cache.row_off.cpu().numpy()
    assert torch.count_nonzero(cache.k_rows[off[1]:off[1] + 10]) == 0


@pytest.mark.parametrize("name", ["bf16", "bf16_d64", "f32_d128"])
def test_prefill_after_an_overflow_stays_inside_the_slab(name):
    """The LAST slab of the pool is too small for its retained tokens: compaction leaves it empty
    (len = 0, overflow bit) while its prefix counts stay full.  Prefill attention must then see the
    slab as empty - each of its queries attends to itself only, O = V exactly - read nothing past the
    end of the pool, and leave the other slabs as the oracle has them."""
    shape = SHAPES[name].with_(batch=1, seq=300)
    h, n = shape.heads, shape.seq
    Q, K, V = inputs.qkv_gaussian(shape, 240, DEV)
    f = inputs.bernoulli_flags((1, h, n), 0.5, 241).numpy()
    L = f.reshape(h, n).sum(axis=1)
    cap = L.copy()
    cap[-1] = L[-1] - 1                                          # one row short
    flags = torch.from_numpy(f).to(DEV)
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, cap=cap.tolist())
    assert int(status.item()) & ag.AG_DEV_OVERFLOW
    want_len = L.copy()
    want_len[-1] = 0
    assert cache.len.cpu().tolist() == want_len.tolist()
    O = T.gpu_prefill(shape, Q, K, V, flags, cache, prefix)
    assert torch.equal(O[0, h - 1], V[0, h - 1])                 # the emptied slab: the diagonal only
    # the oracle's view: that head evicts everything, the others are untouched
    f_seen = f.copy()
    f_seen[0, h - 1] = 0
    O_ref = orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), f_seen)
    T.check_close(T.f64(O), O_ref, shape.dtype, "prefill after an overflow")


@pytest.mark.parametrize("name", list(SHAPES))
def test_prefill_attention(name):
    shape = SHAPES[name]
    X, W, Q, K, V = _layer_inputs(shape, 300)
    flags = _flag_patterns(shape, 310)
    cache, prefix, idx, _ = T.gpu_compact(shape, K, V, flags)
    O = T.gpu_prefill(shape, Q, K, V, flags, cache, prefix)
    O_ref = orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), flags.cpu().numpy())
    T.check_close(T.f64(O), O_ref, shape.dtype, "prefill")
    # all-evict head: the diagonal only, O = V exactly (Sec. 3.3)
    assert torch.equal(O[0, 1 % shape.heads], V[0, 1 % shape.heads])
    # explicit softmax scale
    O2 = T.gpu_prefill(shape, Q, K, V, flags, cache, prefix, scale=0.05)
    O2_ref = orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), flags.cpu().numpy(), scale=float(np.float32(0.05)))
    T.check_close(T.f64(O2), O2_ref, shape.dtype, "prefill scale")


@pytest.mark.parametrize("n", [1, 63, 64, 65, 127, 128, 129, 257, 700])
def test_prefill_ragged_lengths(n):
    shape = SMALL_BF16.with_(seq=n, batch=1)
    Q, K, V = inputs.qkv_gaussian(shape, 320 + n, DEV)
    flags = inputs.bernoulli_flags((1, shape.heads, n), 0.6, 330 + n).to(DEV)
    cache, prefix, idx, _ = T.gpu_compact(shape, K, V, flags)
    O = T.gpu_prefill(shape, Q, K, V, flags, cache, prefix)
    O_ref = orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), flags.cpu().numpy())
    T.check_close(T.f64(O), O_ref, "bf16", f"n={n}")


def test_prefill_tight_slabs_and_uninitialised_tail():
    """Slabs laid out back to back with no slack, pool pre-filled with NaN
    bit patterns: nothing outside a slab's valid rows may leak into O."""
    shape = SMALL_BF16.with_(seq=300, batch=1)
    Q, K, V = inputs.qkv_gaussian(shape, 340, DEV)
    flags = inputs.bernoulli_flags((1, shape.heads, 300), 0.4, 341).to(DEV)
    L = flags.cpu().numpy().reshape(shape.heads, -1).sum(axis=1)
    cache = ag.RaggedCache.allocate(shape, (L + 1).tolist(), DEV)
    cache.k_rows.fill_(float("nan"))
    cache.v_rows.fill_(float("nan"))
    desc = ag.make_desc(shape)
    prefix = torch.empty(1, shape.heads, 301, dtype=torch.int32, device=DEV)
    ag.ag_compact_kv(desc, K, V, flags, cache, prefix, None, None, ag.workspace(desc, ag.AG_CALL_COMPACT))
    O = T.gpu_prefill(shape, Q, K, V, flags, cache, prefix)
    O_ref = orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), flags.cpu().numpy())
    T.check_close(T.f64(O), O_ref, "bf16", "tight slabs")


def test_tiny_layer_end_to_end():
    """Whole path on the fp32 correctness layer: the oracle runs on its own
    flags, the GPU on its own; the flags must coincide (calibration puts no
    score in the band) and every downstream output must agree."""
    shape = inputs.TINY
    X = inputs.hidden_states(shape, 1000, DEV)
    W = inputs.layer_weights(shape, 1010, DEV)
    Q, K, V = inputs.project_qkv(shape, X, W)
    gamma = _calibrated_gamma(shape, X, W, [0.5] * shape.heads)
    scores, flags = T.gpu_gate(shape, X, W, gamma)
    s_ref, f_ref = T.oracle_gate(shape, X, W, gamma)
    assert np.array_equal(flags.cpu().numpy(), f_ref)
    assert abs(f_ref.mean() - 0.5) < 0.02
    cap = [shape.seq + 16] * (shape.batch * shape.heads)
    for keep_new in (1.0, 0.5):
        cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, cap=cap)
        T.check_compaction(shape, K, V, flags, cache, prefix, idx)
        ocache = orc.compact_kv(T.f64(K), T.f64(V), f_ref)
        O = T.gpu_prefill(shape, Q, K, V, flags, cache, prefix)
        T.check_close(T.f64(O), orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), f_ref), "f32", "prefill")
        for step in range(16):
            x_new = inputs.randn((shape.batch, 1, shape.hidden), 1200 + step, DEV)
            q, kn, vn = [t[:, :, 0].contiguous() for t in inputs.project_qkv(shape.with_(seq=1), x_new, W)]
            fn = (torch.ones(shape.batch, shape.heads, dtype=torch.uint8) if keep_new == 1.0
                  else inputs.bernoulli_flags((shape.batch, shape.heads), 0.5, 1300 + step)).to(DEV)
            o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status)
            o_ref = orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache)
            T.check_close(T.f64(o), o_ref, "f32", f"decode step {step}")
            orc.cache_append(ocache, T.f64(kn), T.f64(vn), fn.cpu().numpy())
        assert np.array_equal(cache.len.cpu().numpy(), orc.cache_lengths(ocache).reshape(-1))
        assert int(status.item()) == 0


@pytest.mark.parametrize("fused", [False, True], ids=["two_calls", "one_call"])
@pytest.mark.parametrize("name", ["bf16", "bf16_d64", "f32_d128"])
def test_decode_and_append(name, fused):
    shape = SHAPES[name].with_(seq=700)
    Q, K, V = inputs.qkv_gaussian(shape, 400, DEV)
    flags = _flag_patterns(shape, 410)
    steps = 6
    B, h = shape.batch, shape.heads
    cap = (flags.cpu().numpy().reshape(B * h, -1).sum(axis=1) + steps).tolist()
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, cap=cap)
    ocache = orc.compact_kv(T.f64(K), T.f64(V), flags.cpu().numpy())
    for step in range(steps):
        q, kn, vn, fn = inputs.decode_inputs(shape, 420, step, DEV, keep_new=0.5)
        o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=fused)
        o_ref = orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache)
        T.check_close(T.f64(o), o_ref, shape.dtype, f"decode step {step}")
        orc.cache_append(ocache, T.f64(kn), T.f64(vn), fn.cpu().numpy())
    L = cache.len.cpu().numpy()
    assert np.array_equal(L, orc.cache_lengths(ocache).reshape(-1))
    assert int(status.item()) == 0
    # appended rows are bit copies, in order
    got = T.gpu_cache_as_lists(cache, shape)
    for b in range(B):
        for i in range(h):
            assert np.array_equal(got[b][i]["k"], ocache[b][i]["k"])
            assert np.array_equal(got[b][i]["v"], ocache[b][i]["v"])


def test_decode_long_slabs_many_chunks():
    """Slabs long enough for several split-K chunks of different fill."""
    shape = LayerShape(1, 3000, 512, 4, 128, 2, 128, "bf16")
    Q, K, V = inputs.qkv_gaussian(shape, 450, DEV)
    f = inputs.bernoulli_flags((1, 4, 3000), 0.5, 451).numpy()
    f[0, 0] = 1
    f[0, 1, 257:] = 0
    flags = torch.from_numpy(f).to(DEV)
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, cap=[3001] * 4)
    ocache = orc.compact_kv(T.f64(K), T.f64(V), f)
    q, kn, vn, fn = inputs.decode_inputs(shape, 460, 0, DEV, keep_new=1.0)
    o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status)
    T.check_close(T.f64(o), orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache), "bf16", "long slabs")


@pytest.mark.parametrize("shape", [LayerShape(9, 300, 256, 8, 128, 2, 128, "bf16"),
                                   LayerShape(17, 150, 128, 4, 64, 1, 64, "f32")],
                         ids=["bf16_72slabs", "f32_d64_68slabs"])
@pytest.mark.parametrize("fused", [False, True], ids=["two_calls", "one_call"])
def test_decode_many_slabs_takes_the_workspace_form(shape, fused):
    """More slabs than the one-cluster-per-slab form serves: chunk pass + merge through the
    workspace, at a size the oracle checks in full; ragged and empty slabs included."""
    Q, K, V = inputs.qkv_gaussian(shape, 470, DEV)
    f = inputs.bernoulli_flags((shape.batch, shape.heads, shape.seq), 0.6, 471).numpy()
    f[0, 0] = 1
    f[1, 1] = 0
    f[2, 2, 5:] = 0
    flags = torch.from_numpy(f).to(DEV)
    steps = 3
    cap = [shape.seq + steps] * (shape.batch * shape.heads)
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, cap=cap)
    ocache = orc.compact_kv(T.f64(K), T.f64(V), f)
    for step in range(steps):
        q, kn, vn, fn = inputs.decode_inputs(shape, 472, step, DEV, keep_new=0.5)
        o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=fused)
        o_ref = orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache)
        T.check_close(T.f64(o), o_ref, shape.dtype, f"decode step {step}")
        orc.cache_append(ocache, T.f64(kn), T.f64(vn), fn.cpu().numpy())
    assert np.array_equal(cache.len.cpu().numpy(), orc.cache_lengths(ocache).reshape(-1))
    assert int(status.item()) == 0


@pytest.mark.parametrize("fused", [False, True], ids=["two_calls", "one_call"])
def test_decode_empty_cache_returns_own_value_and_full_slab_reports_overflow(fused):
    shape = SMALL_BF16.with_(seq=64)
    Q, K, V = inputs.qkv_gaussian(shape, 500, DEV)
    flags = torch.zeros(shape.batch, shape.heads, shape.seq, dtype=torch.uint8, device=DEV)
    cap = [1] * (shape.batch * shape.heads)
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, cap=cap)
    q, kn, vn, fn = inputs.decode_inputs(shape, 510, 0, DEV, keep_new=1.0)
    o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=fused)
    assert torch.equal(o, vn)                                   # L = 0: only the self term
    assert int(status.item()) == 0 and cache.len.cpu().tolist() == cap
    q2, kn2, vn2, fn2 = inputs.decode_inputs(shape, 510, 1, DEV, keep_new=1.0)
    o2 = T.gpu_decode_step(shape, q2, kn2, vn2, fn2, cache, status, fused=fused)
    assert int(status.item()) & ag.AG_DEV_OVERFLOW                # slabs are full: write skipped
    assert cache.len.cpu().tolist() == cap
    assert torch.equal(cache.k_rows, kn.reshape(-1, shape.head_dim))
    one_row = [[{"k": T.f64(kn[b, i])[None], "v": T.f64(vn[b, i])[None]} for i in range(shape.heads)]
               for b in range(shape.batch)]
    o2_ref = orc.decode_attention(T.f64(q2), T.f64(kn2), T.f64(vn2), one_row)
    T.check_close(T.f64(o2), o2_ref, "bf16", "decode over one row")


@pytest.mark.parametrize("name", ["bf16", "f32_d128"])
def test_decode_from_a_cache_snapshot_repeats_bit_for_bit(name):
    """The cache after prefill is the whole state of a layer: copied aside, restored and decoded from
    again, it gives the same outputs and the same cache, bit for bit."""
    shape = SHAPES[name].with_(seq=500)
    Q, K, V = inputs.qkv_gaussian(shape, 620, DEV)
    flags = _flag_patterns(shape, 621)
    steps = 16
    cap = [shape.seq + steps] * (shape.batch * shape.heads)
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, cap=cap)
    snap = (cache.k_rows.clone(), cache.v_rows.clone(), cache.len.clone())
    runs = []
    for _ in range(2):
        cache.k_rows.copy_(snap[0]); cache.v_rows.copy_(snap[1]); cache.len.copy_(snap[2])
        outs = []
        for step in range(steps):
            q, kn, vn, fn = inputs.decode_inputs(shape, 630, step, DEV, keep_new=0.5)
            outs.append(T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=True))
        runs.append(outs + [cache.k_rows.clone(), cache.v_rows.clone(), cache.len.clone()])
    for a, b in zip(*runs):
        assert torch.equal(a, b)
    assert int(status.item()) == 0


def test_results_are_bitwise_repeatable():
    shape = SMALL_BF16
    X, W, Q, K, V = _layer_inputs(shape, 600)
    runs = []
    for _ in range(2):
        scores, flags = T.gpu_gate(shape, X, W, None)
        cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags)
        O = T.gpu_prefill(shape, Q, K, V, flags, cache, prefix)
        q, kn, vn, fn = inputs.decode_inputs(shape, 610, 0, DEV)
        o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status)
        L = cache.len.cpu()
        runs.append([scores, flags, prefix, O, o, cache.len.clone(), cache.k_rows.clone()])
    for a, b in zip(*runs):
        assert torch.equal(a, b)


def test_no_device_wait_expired():
    """Runs after the other tests of this file: no bounded wait inside a kernel gave up."""
    assert ag.ag_device_wait_timeouts() == 0
