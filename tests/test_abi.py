"""Host-side checks of the C boundary: the library builds, loads, exports every
function include/ag.h declares, sizes workspaces, and rejects bad arguments
before touching the GPU.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

from paper_2410_12876_b200 import build as ag_build
from paper_2410_12876_b200 import binding as ag
from paper_2410_12876_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ag_build.build()
    return ag.lib()


def test_every_declared_function_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "ag.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ag_[a-z_]+)\s*\(", header))
    assert declared == set(ag.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_struct_layout_matches_header():
    assert ctypes.sizeof(ag.ag_layer_desc) == 56            # ten 4-byte fields, the seq_lens pointer, kv_heads, recent_window
    assert ag.ag_layer_desc.seq_lens.offset == 40
    assert ag.ag_layer_desc.kv_heads.offset == 48
    assert ag.ag_layer_desc.recent_window.offset == 52
    assert ctypes.sizeof(ag.ag_cache) == 88
    assert ag.ag_cache.max_cap.offset == 48
    assert ag.ag_cache.recent_k.offset == 56 and ag.ag_cache.pos.offset == 80


def test_workspace_sizes(lib):
    d = ag.make_desc(inputs.PREFILL7B)
    rows, GD = 4096, 512
    assert ag.ag_workspace_bytes(d, ag.AG_CALL_GATE) >= rows * 4 * GD * 4
    assert ag.ag_workspace_bytes(d, ag.AG_CALL_COMPACT) == 32 * 4096 * 4
    assert ag.ag_workspace_bytes(d, ag.AG_CALL_DECODE) > 0
    assert ag.ag_workspace_bytes(d, ag.AG_CALL_APPEND) == 0
    bad = ag.make_desc(inputs.PREFILL7B.with_(head_dim=96))
    assert ag.ag_workspace_bytes(bad, ag.AG_CALL_DECODE) == 0


def test_status_strings(lib):
    assert ag.ag_status_string(0) == "ok"
    for s in (-1, -2, -3, -4, -5, -99):
        assert ag.ag_status_string(s)


def _cache_struct(pool_rows=64, max_cap=16, ptr=4096):
    return ag.ag_cache(ptr, ptr, pool_rows, ptr, ptr, ptr, max_cap)


def test_bad_arguments_are_rejected_on_the_host(lib):
    d = ag.make_desc(inputs.TINY)
    p = 4096  # an aligned, never dereferenced address
    byref = ctypes.byref
    # null pointer
    assert lib.ag_gate_forward(byref(d), None, p, p, p, p, None, None, p, p, 1 << 30, None) == ag.AG_ERR_INVALID_ARG
    # misaligned pointer
    assert lib.ag_gate_forward(byref(d), p + 4, p, p, p, p, None, None, p, p, 1 << 30, None) == ag.AG_ERR_INVALID_ARG
    # workspace too small / missing
    assert lib.ag_gate_forward(byref(d), p, p, p, p, p, None, None, p, p, 16, None) == ag.AG_ERR_WORKSPACE
    assert lib.ag_gate_forward(byref(d), p, p, p, p, p, None, None, p, None, 0, None) == ag.AG_ERR_WORKSPACE
    # h' >= h is outside the method (Sec. 3.3 requires h' < h)
    d2 = ag.make_desc(inputs.TINY.with_(gate_heads=4))
    assert lib.ag_gate_forward(byref(d2), p, p, p, p, p, None, None, p, p, 1 << 30, None) == ag.AG_ERR_INVALID_ARG
    # tau outside (0, 1)
    d3 = ag.make_desc(inputs.TINY.with_(tau=1.0))
    assert lib.ag_gate_forward(byref(d3), p, p, p, p, p, None, None, p, p, 1 << 30, None) == ag.AG_ERR_INVALID_ARG
    # unsupported head_dim, empty sequence
    d4 = ag.make_desc(inputs.TINY.with_(head_dim=80))
    c = _cache_struct()
    assert lib.ag_decode_attn(byref(d4), p, p, p, byref(c), 0.0, p, p, 1 << 30, None) == ag.AG_ERR_UNSUPPORTED
    d5 = ag.make_desc(inputs.TINY.with_(seq=0))
    assert lib.ag_decode_attn(byref(d5), p, p, p, byref(c), 0.0, p, p, 1 << 30, None) == ag.AG_ERR_INVALID_ARG
    # cache checks: K without V, max_cap beyond the pool, missing arrays
    assert lib.ag_compact_kv(byref(d), p, None, p, byref(c), p, p, None, None, 0, None) == ag.AG_ERR_INVALID_ARG
    big = _cache_struct(pool_rows=8, max_cap=16)
    assert lib.ag_prefill_attn(byref(d), p, p, p, p, byref(big), p, 0.0, p, None, 0, None) == ag.AG_ERR_CAPACITY
    nolen = ag.ag_cache(p, p, 64, p, p, None, 16)
    assert lib.ag_cache_append(byref(d), p, p, p, byref(nolen), None, None) == ag.AG_ERR_INVALID_ARG
    # negative / non-finite softmax scale
    assert lib.ag_prefill_attn(byref(d), p, p, p, p, byref(c), p, -1.0, p, None, 0, None) == ag.AG_ERR_INVALID_ARG
    assert lib.ag_decode_attn(byref(d), p, p, p, byref(c), float("inf"), p, p, 1 << 30, None) == ag.AG_ERR_INVALID_ARG


def test_projection_calls_reject_on_the_host(lib):
    """ag_kv_project_cache / ag_qkv_project_cache: argument checks and kernel coverage, nothing launched."""
    p = 4096
    byref = ctypes.byref
    c = _cache_struct()
    ok = ag.make_desc(inputs.LayerShape(2, 256, 512, 4, 128, 2, 128, "bf16"))
    kv = lambda d, X=p, Wk=p, Wv=p, fl=p, pre=p, K=p, V=p: lib.ag_kv_project_cache(
        byref(d), X, Wk, Wv, fl, byref(c), pre, None, K, V, None, None)
    assert kv(ok, X=None) == ag.AG_ERR_INVALID_ARG
    assert kv(ok, V=None) == ag.AG_ERR_INVALID_ARG
    assert kv(ok, pre=None) == ag.AG_ERR_INVALID_ARG
    assert kv(ok, Wk=p + 2) == ag.AG_ERR_INVALID_ARG
    assert kv(ag.make_desc(inputs.TINY)) == ag.AG_ERR_UNSUPPORTED                                      # float32, head_dim 64
    assert kv(ag.make_desc(inputs.LayerShape(2, 256, 516, 4, 128, 2, 128, "bf16"))) == ag.AG_ERR_UNSUPPORTED   # hidden not a multiple of 8
    assert kv(ag.make_desc(inputs.LayerShape(2, 256, 516, 4, 128, 2, 128, "bf16"))) == ag.AG_ERR_UNSUPPORTED   # rows of X not 16-byte multiples
    assert kv(ag.make_desc(inputs.LayerShape(2, 256, 512, 4, 128, 2, 128, "bf16", recent_window=5))) == ag.AG_ERR_INVALID_ARG  # no ring
    assert lib.ag_qkv_project_cache(byref(ok), p, None, p, p, p, byref(c), p, None, p, p, p, None, None) == ag.AG_ERR_INVALID_ARG
    assert lib.ag_qkv_project_cache(byref(ok), p, p, p, p, p, byref(c), p, None, None, p, p, None, None) == ag.AG_ERR_INVALID_ARG


def test_binding_raises_with_status(lib):
    d = ag.make_desc(inputs.TINY.with_(gate_heads=7))
    with pytest.raises(ag.AgError) as e:
        ag.ag_gate_forward(d, 4096, 4096, 4096, 4096, 4096, None, None, 4096, None, stream=0)
    assert e.value.status == ag.AG_ERR_INVALID_ARG
