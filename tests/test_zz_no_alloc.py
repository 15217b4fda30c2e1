"""The decode call for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option: inside a
process whose own pool already owns all of the GPU's memory, or on a step that
cannot afford the stall an allocation may bring.  They cannot hand
ag_decode_attn its split-K workspace, so ag_decode_attn_noalloc keeps that
scratch in a fixed array inside the library.  These tests check, through the C
boundary, that it gives what ag_decode_attn gives, twice in a row (the array
is shared and keeps the previous call's contents), and that it refuses
problems larger than the array.

This file is named to be collected last, so a run that stops at the first
failure has already been through every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import agtest as T
from paper_2410_12876_b200 import binding as ag
from paper_2410_12876_b200 import inputs
from paper_2410_12876_b200.inputs import LayerShape


@pytest.fixture(scope="module", autouse=True)
def _lib():
    T.ensure_built()


def test_too_large_a_problem_is_refused_on_the_host():
    lib = ag.lib()
    p = 4096
    cache = ag.ag_cache(p, p, 1 << 20, p, p, p, 16)
    ok_size = ag.make_desc(LayerShape(32, 8192, 4096, 32, 128, 4, 128, "bf16"))     # 1024 slabs: fits
    too_big = ag.make_desc(LayerShape(33, 8192, 4096, 32, 128, 4, 128, "bf16"))    # 1056 slabs: does not
    assert ag.ag_workspace_bytes(ok_size, ag.AG_CALL_DECODE) == 17039360
    st = lib.ag_decode_attn_noalloc(ctypes.byref(too_big), p, p, p, ctypes.byref(cache), 0.0, p, None)
    assert st == ag.AG_ERR_CAPACITY
    assert "capacity" in ag.ag_status_string(st)
    # argument checks come first, as in the other calls
    assert lib.ag_decode_attn_noalloc(ctypes.byref(ok_size), None, p, p, ctypes.byref(cache), 0.0, p, None) \
        == ag.AG_ERR_INVALID_ARG
    assert lib.ag_decode_attn_noalloc(ctypes.byref(ok_size), p + 2, p, p, ctypes.byref(cache), 0.0, p, None) \
        == ag.AG_ERR_INVALID_ARG


def test_a_bad_head_grouping_is_refused_on_the_host():
    """The descriptor checks are those of every other call: a key/value head count that does not divide
    the heads (or exceeds them) would make the kernel index slabs that do not exist."""
    lib = ag.lib()
    p = 4096
    cache = ag.ag_cache(p, p, 1 << 20, p, p, p, 16)
    for kv_heads, want in ((3, ag.AG_ERR_INVALID_ARG), (16, ag.AG_ERR_INVALID_ARG), (-1, ag.AG_ERR_INVALID_ARG)):
        desc = ag.make_desc(LayerShape(2, 64, 256, 8, 128, 2, 128, "bf16", kv_heads=kv_heads))
        assert lib.ag_decode_attn_noalloc(ctypes.byref(desc), p, p, p, ctypes.byref(cache), 0.0, p, None) == want
    windowed = ag.make_desc(LayerShape(2, 64, 256, 8, 128, 2, 128, "bf16", recent_window=5))
    assert lib.ag_decode_attn_noalloc(ctypes.byref(windowed), p, p, p, ctypes.byref(cache), 0.0, p, None) \
        == ag.AG_ERR_UNSUPPORTED


def _oracle_cache(shape, K, V, f):
    from oracle import ag_oracle as orc
    return orc, orc.compact_kv(T.f64(K), T.f64(V), f)


# Up to 64 slabs the decode call keeps its partial results on chip and touches no scratch at all; above,
# it goes through the scratch (the caller's workspace, or here the array inside the library).  Both
# sizes are run: the first shows the entry point itself, the other two make the kernels write and
# read the shared array.
CASES = {
    "16_slabs_no_scratch": LayerShape(2, 900, 512, 8, 128, 2, 128, "bf16"),
    "72_slabs_bf16": LayerShape(9, 900, 256, 8, 128, 2, 128, "bf16"),
    "68_slabs_f32_d64": LayerShape(17, 300, 128, 4, 64, 1, 64, "f32"),
}


@pytest.mark.gpu
@pytest.mark.parametrize("case", list(CASES))
def test_matches_the_workspace_call_twice_in_a_row(case):
    dev = "cuda"
    shape = CASES[case]
    desc = ag.make_desc(shape)
    Q, K, V = inputs.qkv_gaussian(shape, 700, dev)
    f = inputs.bernoulli_flags((shape.batch, shape.heads, shape.seq), 0.6, 701).numpy()
    f[0, 1] = 0                                     # an empty slab: only the self term
    f[1, 2] = 1                                     # a full one: several split-K chunks
    f[1, 3, 7:] = 0                                 # a short one: one partly filled chunk
    flags = torch.from_numpy(f).to(dev)
    cap = (f.reshape(shape.batch * shape.heads, -1).sum(axis=1) + 2).tolist()
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, flags, cap=cap)
    orc, ocache = _oracle_cache(shape, K, V, f)
    ws = ag.workspace(desc, ag.AG_CALL_DECODE)
    # The array keeps whatever the previous call (of this or an earlier test) left in it, and the
    # caller's workspace starts as NaN: neither may show in the result.
    ws.view(torch.float32).fill_(float("nan"))
    for step in range(2):
        q, kn, vn, fn = inputs.decode_inputs(shape, 710, step, dev, keep_new=0.5)
        want = torch.full_like(q, float("nan"))
        got = torch.full_like(q, float("nan"))
        ag.ag_decode_attn(desc, q, kn, vn, cache, 0.0, want, ws)
        ag.ag_decode_attn_noalloc(desc, q, kn, vn, cache, 0.0, got)
        torch.cuda.synchronize()
        T.check_close(T.f64(got), T.f64(want), shape.dtype, f"no-alloc decode, call {step}")
        assert torch.equal(got, want)               # same kernels, same order: same bits
        T.check_close(T.f64(got), orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache), shape.dtype,
                      f"no-alloc decode against the oracle, call {step}")
        # the second call sees other lengths (about half of the slabs grow by a row)
        ag.ag_cache_append(desc, kn, vn, fn, cache, status)
        orc.cache_append(ocache, T.f64(kn), T.f64(vn), fn.cpu().numpy())
    assert int(status.item()) == 0
