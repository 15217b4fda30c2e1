"""Eviction guided by the previous layer (Sec. 4.4, ablation settings (4-1) and (4-2)) on the GPU:
a small stack whose gate passes run on a second stream beside the attention of the same layer,
against the oracle's statement of which flags each layer uses.  Each side runs its own gates."""
import numpy as np
import pytest
import torch

import agtest as T
from oracle import ag_oracle as orc
from paper_2410_12876_b200 import binding as ag
from paper_2410_12876_b200 import inputs
from paper_2410_12876_b200.inputs import LayerShape
from paper_2410_12876_b200.schedule import PreviousLayerGate

pytestmark = pytest.mark.gpu
DEV = "cuda"
DECODE_STEPS = 3


@pytest.fixture(scope="module", autouse=True)
def _lib():
    T.ensure_built()


class _Layer:
    """Inputs and output buffers of one layer of the stack (its own hidden states and weights)."""

    def __init__(self, shape, seed, keep):
        self.shape, self.desc = shape, ag.make_desc(shape)
        B, h, n = shape.batch, shape.heads, shape.seq
        self.X = inputs.hidden_states(shape, seed, DEV)
        self.W = inputs.layer_weights(shape, seed + 10, DEV)
        self.W["Wo_g"] = inputs.randn(tuple(self.W["Wo_g"].shape), seed + 17, DEV, shape.torch_dtype, 0.5)
        self.Q, self.K, self.V = inputs.project_qkv(shape, self.X, self.W)
        s0, _ = T.oracle_gate(shape, self.X, self.W, None)
        self.gamma = inputs.calibrate_gamma(torch.from_numpy(s0), keep, float(np.float32(shape.tau))).to(DEV)
        self.cache = ag.RaggedCache.allocate(shape, [n + DECODE_STEPS] * (B * h), DEV)
        self.prefix = torch.full((B, h, n + 1), -1, dtype=torch.int32, device=DEV)
        self.O = torch.full_like(self.Q, float("nan"))
        self.status = torch.zeros(1, dtype=torch.int32, device=DEV)
        self.dq = [inputs.decode_inputs(shape, seed + 500, s, DEV) for s in range(DECODE_STEPS)]
        self.o = [torch.full_like(self.dq[0][0], float("nan")) for _ in range(DECODE_STEPS)]
        self.flags_used = torch.full((B, h, n), 9, dtype=torch.uint8, device=DEV)
        self.ws = {c: ag.workspace(self.desc, c) for c in (ag.AG_CALL_GATE, ag.AG_CALL_COMPACT, ag.AG_CALL_PREFILL,
                                                            ag.AG_CALL_DECODE)}

    def gate(self, flags_out):
        W = self.W
        ag.ag_gate_forward(self.desc, self.X, W["Wq_g"], W["Wk_g"], W["Wv_g"], W["Wo_g"], self.gamma, None, flags_out,
                           self.ws[ag.AG_CALL_GATE])

    def attend(self, flags):
        self.flags_used.copy_(flags)                 # what this layer ran under, for the comparison below
        ag.ag_compact_kv(self.desc, self.K, self.V, flags, self.cache, self.prefix, None, self.status,
                         self.ws[ag.AG_CALL_COMPACT])
        ag.ag_prefill_attn(self.desc, self.Q, self.K, self.V, flags, self.cache, self.prefix, 0.0, self.O,
                           self.ws[ag.AG_CALL_PREFILL])
        for s, (q, kn, vn, fn) in enumerate(self.dq):
            ag.ag_decode_step(self.desc, q, kn, vn, fn, self.cache, 0.0, self.o[s], self.status, self.ws[ag.AG_CALL_DECODE])


@pytest.mark.parametrize("first_gated", [1, 2])
@pytest.mark.parametrize("shape", [inputs.TINY, LayerShape(2, 333, 512, 8, 128, 2, 128, "bf16")], ids=["tiny_f32", "bf16"])
def test_stack_guided_by_the_previous_layer(shape, first_gated):
    n_layers = 5
    keeps = [0.3, 0.7, 0.5, 0.2, 0.6]                # a different keep rate per layer's AG module
    layers = [_Layer(shape, 4000 + 50 * l, [keeps[l]] * shape.heads) for l in range(n_layers)]
    B, h, n = shape.batch, shape.heads, shape.seq
    bufs = [torch.full((B, h, n), 7, dtype=torch.uint8, device=DEV) for _ in range(2)]
    ones = torch.ones(B, h, n, dtype=torch.uint8, device=DEV)
    sched = PreviousLayerGate(first_gated, bufs, ones, DEV)
    for _ in range(2):                               # the second pass re-uses buffers and events
        sched.run(n_layers, lambda l, out: layers[l].gate(out), lambda l, f: layers[l].attend(f))
    torch.cuda.synchronize()

    gates = [lambda L=L: T.oracle_gate(shape, L.X, L.W, L.gamma) for L in layers]
    used = orc.previous_layer_flags(gates, first_gated, (B, h, n))
    for l, L in enumerate(layers):
        f_ref = used[l]
        assert np.array_equal(L.flags_used.cpu().numpy(), f_ref), f"layer {l}"
        if l >= first_gated:
            assert abs(f_ref.mean() - keeps[l - 1]) < 0.05      # the PREVIOUS module's keep rate
        assert int(L.status.item()) == 0
        Q, K, V = T.f64(L.Q), T.f64(L.K), T.f64(L.V)
        T.check_close(T.f64(L.O), orc.prefill_attention(Q, K, V, f_ref), shape.dtype, f"prefill, layer {l}")
        ocache = orc.compact_kv(K, V, f_ref)
        for s, (q, kn, vn, fn) in enumerate(L.dq):
            o_ref = orc.decode_attention(T.f64(q), T.f64(kn), T.f64(vn), ocache)
            T.check_close(T.f64(L.o[s]), o_ref, shape.dtype, f"decode step {s}, layer {l}")
            orc.cache_append(ocache, T.f64(kn), T.f64(vn), fn.cpu().numpy())
        assert np.array_equal(L.cache.len.cpu().numpy(), orc.cache_lengths(ocache).reshape(-1))


def test_needs_a_previous_layer():
    with pytest.raises(ValueError):
        PreviousLayerGate(0, [None, None], None, DEV)
