"""Seeded sweep of random layer shapes through the whole path (gate -> compaction -> prefill ->
decode steps), every call against the oracle.  The fixed cases elsewhere pin known edges; this
one walks sizes that straddle tile, segment, chunk and cluster boundaries in combinations nobody
picked by hand."""
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


def _random_shape(rng, dtype):
    heads = int(rng.integers(2, 10))
    if dtype == "bf16":
        head_dim, gate_head_dim = 128, 128                      # the tensor-core kernels
        hidden = int(rng.integers(8, 80)) * 8
    else:
        head_dim, gate_head_dim = int(rng.choice([64, 128])), int(rng.choice([64, 128]))
        hidden = int(rng.integers(4, 24)) * 8
    return LayerShape(int(rng.integers(1, 4)), int(rng.integers(1, 600)), hidden, heads, head_dim,
                      int(rng.integers(1, heads)), gate_head_dim, dtype,
                      gate_causal=int(rng.integers(0, 2)))


@pytest.mark.parametrize("case", range(24))
def test_random_layer(case):
    rng = np.random.default_rng(9000 + case)
    shape = _random_shape(rng, "bf16" if case % 3 else "f32")
    seed = 9100 + 10 * case
    X = inputs.hidden_states(shape, seed, DEV)
    W = inputs.layer_weights(shape, seed + 1, DEV)
    W["Wo_g"] = inputs.randn(tuple(W["Wo_g"].shape), seed + 2, DEV, shape.torch_dtype, 0.5)
    Q, K, V = inputs.project_qkv(shape, X, W)
    B, h, n = shape.batch, shape.heads, shape.seq

    # gate: scores, and flags outside the band
    s0, _ = T.oracle_gate(shape, X, W, None)
    keep = rng.uniform(0.2, 0.9, h)
    gamma = inputs.calibrate_gamma(torch.from_numpy(s0), keep, float(np.float32(shape.tau))).to(DEV)
    scores, flags = T.gpu_gate(shape, X, W, gamma)
    s_ref, f_ref = T.oracle_gate(shape, X, W, gamma)
    assert np.max(np.abs(T.f64(scores) - s_ref)) < 1e-4, shape
    T.check_flags(shape, flags, s_ref, f_ref, gamma)

    # downstream on the oracle's flags, with one head emptied and one kept whole
    f = np.ascontiguousarray(f_ref).copy()
    f[0, 0] = 0
    f[-1, -1] = 1
    fl = torch.from_numpy(f).to(DEV)
    steps = 3
    cap = (f.reshape(B * h, -1).sum(axis=1) + steps).tolist()               # tight slabs
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, fl, cap=cap)
    T.check_compaction(shape, K, V, fl, cache, prefix, idx)
    O = T.gpu_prefill(shape, Q, K, V, fl, cache, prefix)
    T.check_close(T.f64(O), orc.prefill_attention(T.f64(Q), T.f64(K), T.f64(V), f), shape.dtype, f"prefill {shape}")
    assert torch.equal(O[0, 0], V[0, 0])                                     # emptied head: the diagonal only

    ocache = orc.compact_kv(T.f64(K), T.f64(V), f)
    for step in range(steps):
        q, kn, vn, fn = inputs.decode_inputs(shape, seed + 5, step, DEV, keep_new=0.7)
        o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=bool((case + step) % 2))
        o_ref = orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache)
        T.check_close(T.f64(o), o_ref, shape.dtype, f"decode {step} {shape}")
        orc.cache_append(ocache, T.f64(kn), T.f64(vn), fn.cpu().numpy())
    assert np.array_equal(cache.len.cpu().numpy(), orc.cache_lengths(ocache).reshape(-1))
    assert int(status.item()) == 0 and ag.ag_device_wait_timeouts() == 0
