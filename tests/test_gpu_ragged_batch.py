"""Batches of sequences of different lengths (desc.seq_lens): the gate calls treat positions
past seq_lens[b] as padding; everything downstream then never sees them."""
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
    "bf16_tc": LayerShape(3, 333, 512, 8, 128, 2, 128, "bf16"),
    "bf16_d64": LayerShape(3, 200, 256, 4, 64, 2, 64, "bf16"),
    "f32": LayerShape(3, 150, 128, 3, 128, 1, 128, "f32"),
}


def _lens(shape):
    n = shape.seq
    return np.array([n, 1, n // 2 + 3], dtype=np.int32)


def _check_valid_region(shape, lens, scores, flags, s_ref, f_ref, gamma):
    g = np.zeros(shape.heads) if gamma is None else T.f64(gamma)
    tau = float(np.float32(shape.tau))
    fg = flags.cpu().numpy()
    sg = T.f64(scores)
    for b, L in enumerate(lens):
        assert np.max(np.abs(sg[b, :, :L] - s_ref[b, :, :L])) < 1e-4
        dist = np.abs(s_ref[b, :, :L] + g[:, None] - np.log(tau / (1 - tau)))
        outside = dist >= T.FLAG_BAND
        assert np.array_equal(fg[b, :, :L][outside], f_ref[b, :, :L][outside])
        assert np.all(fg[b, :, L:] == 0)                       # padding is evicted


@pytest.mark.parametrize("causal", [1, 0])
@pytest.mark.parametrize("name", list(SHAPES))
def test_ragged_gate(name, causal):
    shape = SHAPES[name].with_(gate_causal=causal)
    lens = _lens(shape)
    lens_dev = torch.from_numpy(lens).to(DEV)
    X = inputs.hidden_states(shape, 800, DEV)
    W = inputs.layer_weights(shape, 810, DEV)
    W["Wo_g"] = inputs.randn(tuple(W["Wo_g"].shape), 817, DEV, shape.torch_dtype, 0.5)
    gamma = torch.from_numpy(np.random.default_rng(5).uniform(-0.3, 0.3, shape.heads).astype(np.float32)).to(DEV)
    tau = float(np.float32(shape.tau))
    fn = lambda x: orc.attention_gate(x, T.f64(W["Wq_g"]), T.f64(W["Wk_g"]), T.f64(W["Wv_g"]), T.f64(W["Wo_g"]),
                                      shape.gate_heads, T.f64(gamma), tau, causal=bool(causal))
    s_ref, f_ref = orc.ragged_gate(T.f64(X), lens, fn)
    B, h, n = shape.batch, shape.heads, shape.seq
    scores = torch.empty(B, h, n, dtype=torch.float32, device=DEV)
    flags = torch.full((B, h, n), 7, dtype=torch.uint8, device=DEV)
    desc = ag.make_desc(shape, lens_dev)
    ag.ag_gate_forward(desc, X, W["Wq_g"], W["Wk_g"], W["Wv_g"], W["Wo_g"], gamma, scores, flags,
                       ag.workspace(desc, ag.AG_CALL_GATE))
    _check_valid_region(shape, lens, scores, flags, s_ref, f_ref, gamma)


@pytest.mark.parametrize("name", list(SHAPES))
def test_ragged_linear_gate(name):
    shape = SHAPES[name]
    lens = _lens(shape)
    lens_dev = torch.from_numpy(lens).to(DEV)
    X = inputs.hidden_states(shape, 820, DEV)
    W = inputs.linear_gate_weight(shape, 821, DEV)
    tau = float(np.float32(shape.tau))
    s_ref, f_ref = orc.ragged_gate(T.f64(X), lens, lambda x: orc.linear_gate(x, T.f64(W), None, tau))
    B, h, n = shape.batch, shape.heads, shape.seq
    scores = torch.empty(B, h, n, dtype=torch.float32, device=DEV)
    flags = torch.full((B, h, n), 7, dtype=torch.uint8, device=DEV)
    ag.ag_gate_linear_forward(ag.make_desc(shape, lens_dev), X, W, None, scores, flags)
    _check_valid_region(shape, lens, scores, flags, s_ref, f_ref, None)


def test_ragged_batch_through_the_layer():
    """Flags of a ragged batch drive compaction, prefill and a decode step: every valid row equals
    what the sequence alone gives; the cache holds no padding."""
    shape = SHAPES["bf16_tc"]
    lens = _lens(shape)
    B, h, n = shape.batch, shape.heads, shape.seq
    Q, K, V = inputs.qkv_gaussian(shape, 830, DEV)
    f = inputs.bernoulli_flags((B, h, n), 0.6, 831).numpy()
    for b, L in enumerate(lens):
        f[b, :, L:] = 0                                        # what the gate calls guarantee
    fl = torch.from_numpy(f).to(DEV)
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, fl, cap=[n + 1] * (B * h))
    T.check_compaction(shape, K, V, fl, cache, prefix, idx)
    O = T.gpu_prefill(shape, Q, K, V, fl, cache, prefix)
    # the same call told the lengths (it then skips the query tiles that hold padding only): the valid rows are the same bits
    desc_l = ag.make_desc(shape, torch.from_numpy(lens).to(DEV))
    O_l = torch.full_like(Q, float("nan"))
    ag.ag_prefill_attn(desc_l, Q, K, V, fl, cache, prefix, 0.0, O_l, ag.workspace(desc_l, ag.AG_CALL_PREFILL))
    for b, L in enumerate(lens):
        assert torch.equal(O_l[b, :, :L], O[b, :, :L])
    Qf, Kf, Vf = T.f64(Q), T.f64(K), T.f64(V)
    for b, L in enumerate(lens):
        alone = orc.prefill_attention(Qf[b:b + 1, :, :L], Kf[b:b + 1, :, :L], Vf[b:b + 1, :, :L], f[b:b + 1, :, :L])
        T.check_close(T.f64(O)[b, :, :L], alone[0], "bf16", f"prefill of sequence {b}")
    ocache = orc.compact_kv(Kf, Vf, f)
    q, kn, vn, fn = inputs.decode_inputs(shape, 832, 0, DEV, keep_new=0.5)
    o = T.gpu_decode_step(shape, q, kn, vn, fn, cache, status, fused=True)
    T.check_close(T.f64(o), orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache), "bf16", "decode")
    assert int(status.item()) == 0
