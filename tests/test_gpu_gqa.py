"""Grouped-query attention (desc.kv_heads): query heads in groups share a key/value head, its
flags and its cache slab.  Whole path against the oracle."""
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


SHAPES = {
    "bf16_tc_8over2": LayerShape(2, 333, 512, 8, 128, 2, 128, "bf16", kv_heads=2),
    "bf16_d64_4over1": LayerShape(1, 200, 256, 4, 64, 2, 64, "bf16", kv_heads=1),
    "f32_6over3": LayerShape(1, 150, 128, 6, 128, 1, 128, "f32", kv_heads=3),
    "bf16_many_slabs": LayerShape(5, 140, 256, 16, 128, 2, 128, "bf16", kv_heads=4),   # 80 query slabs: workspace form
}


@pytest.mark.parametrize("fused", [False, True], ids=["two_calls", "one_call"])
@pytest.mark.parametrize("name", list(SHAPES))
def test_gqa_layer(name, fused):
    shape = SHAPES[name]
    B, h, hk, n = shape.batch, shape.heads, shape.kvh, shape.seq
    X = inputs.hidden_states(shape, 900, DEV)
    W = inputs.layer_weights(shape, 910, DEV)
    W["Wo_g"] = inputs.randn(tuple(W["Wo_g"].shape), 917, DEV, shape.torch_dtype, 0.5)
    Q, K, V = inputs.project_qkv(shape, X, W)
    assert Q.shape[1] == h and K.shape[1] == hk and W["Wo_g"].shape[1] == hk

    # gate: one flag column per key/value head
    gamma = torch.from_numpy(np.random.default_rng(3).uniform(-0.2, 0.2, hk).astype(np.float32)).to(DEV)
    scores, flags = T.gpu_gate(shape, X, W, gamma)
    assert tuple(flags.shape) == (B, hk, n)
    s_ref, f_ref = T.oracle_gate(shape, X, W, gamma)
    assert np.max(np.abs(T.f64(scores) - s_ref)) < 1e-4
    T.check_flags(shape, flags, s_ref, f_ref, gamma)

    # downstream on the oracle's flags
    f = np.ascontiguousarray(f_ref)
    fl = torch.from_numpy(f).to(DEV)
    steps = 3
    cap = (f.reshape(B * hk, -1).sum(axis=1) + steps).tolist()
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, fl, cap=cap)
    T.check_compaction(shape, K, V, fl, cache, prefix, idx)
    O = T.gpu_prefill(shape, Q, K, V, fl, cache, prefix)
    T.check_close(T.f64(O), orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), f), shape.dtype, "prefill")
    ocache = orc.compact_kv(T.f64(K), T.f64(V), f)
    for step in range(steps):
        q, kn, vn, fn = inputs.decode_inputs(shape, 920, step, DEV, keep_new=0.6)
        assert q.shape[1] == h and kn.shape[1] == hk and fn.shape[1] == hk
        o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=fused)
        T.check_close(T.f64(o), orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache), shape.dtype, f"decode {step}")
        orc.cache_append(ocache, T.f64(kn), T.f64(vn), fn.cpu().numpy())
    assert np.array_equal(cache.len.cpu().numpy(), orc.cache_lengths(ocache).reshape(-1))
    assert int(status.item()) == 0 and ag.ag_device_wait_timeouts() == 0


def test_gqa_rejects_heads_that_do_not_divide():
    shape = LayerShape(1, 64, 256, 6, 128, 2, 128, "bf16", kv_heads=4)
    Q, K, V = inputs.qkv_gaussian(shape.with_(kv_heads=3), 1, DEV)
    with pytest.raises(ag.AgError):
        ag.ag_workspace_bytes(ag.make_desc(shape), ag.AG_CALL_DECODE) or ag.ag_decode_attn(
            ag.make_desc(shape), Q[:, :, 0].contiguous(), K[:, :, 0].contiguous(), V[:, :, 0].contiguous(),
            ag.RaggedCache.allocate(shape, [4] * 4, DEV), 0.0, torch.empty_like(Q[:, :, 0]), None)


@pytest.mark.parametrize("heads,kv_heads", [(16, 8), (24, 8), (16, 4), (16, 2), (16, 1)],
                         ids=["group2", "group3", "group4", "group8", "group16"])
@pytest.mark.parametrize("n", [700, 65, 1])
def test_gqa_decode_chunk_pass_on_tensor_cores(heads, kv_heads, n):
    """bf16, head_dim 128, more than 64 query slabs: the group's heads are the rows of one MMA tile.
    Slabs of every length from empty to full, several tiles and a ragged tail, caches that grow."""
    shape = LayerShape(5, n, 256, heads, 128, 2, 128, "bf16", kv_heads=kv_heads)
    B, hk = shape.batch, shape.kvh
    Q, K, V = inputs.qkv_gaussian(shape, 950 + heads + kv_heads, DEV)
    keep = np.linspace(0.0, 1.0, B * hk).reshape(B, hk, 1)        # slab 0 keeps nothing, the last one everything
    f = (np.random.default_rng(951).random((B, hk, n)) < keep).astype(np.uint8)
    f[-1, -1] = 1
    fl = torch.from_numpy(f).to(DEV)
    steps = 4
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, fl, cap=[n + steps] * (B * hk))
    ocache = orc.compact_kv(T.f64(K), T.f64(V), f)
    for fused in (False, True):
        for step in range(steps // 2):
            q, kn, vn, fn = inputs.decode_inputs(shape, 960 + 10 * fused, step, DEV, keep_new=0.6)
            o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=fused)
            T.check_close(T.f64(o), orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache), "bf16", f"decode {step}")
            orc.cache_append(ocache, T.f64(kn), T.f64(vn), fn.cpu().numpy())
    assert np.array_equal(cache.len.cpu().numpy(), orc.cache_lengths(ocache).reshape(-1))
    assert int(status.item()) == 0
