"""A chained stack of attention layers on the GPU: layer l + 1 runs on the hidden states layer l
produced, X_{l+1} = X_l + [H_1 .. H_h] W^O (Eq. 1 with the skip connection; nothing normalises in
between).  Each layer's calls are checked against the oracle fed with the hidden states the GPU
itself handed to that layer: a flag that flips inside the threshold band at layer l would otherwise
change every later layer, and bf16 rounding drifts from layer to layer."""
import numpy as np
import pytest
import torch

import agtest as T
from oracle import ag_oracle as orc
from paper_2410_12876_b200 import binding as ag
from paper_2410_12876_b200 import inputs
from paper_2410_12876_b200.inputs import LayerShape
from paper_2410_12876_b200.schedule import ChainedLayerBuffers, chained_layer

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    T.ensure_built()


def _close_to_rounded(got, ref, what, slack=2e-5):
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    assert np.all(np.isfinite(got)), what
    excess = np.abs(got - ref) - (2.0 ** -8 * np.abs(ref) + slack)
    assert np.max(excess) <= 0, f"{what}: {np.max(excess):.3e} beyond one rounding"


@pytest.mark.parametrize("shape", [LayerShape(2, 256, 512, 8, 128, 2, 128, "bf16"),
                                   LayerShape(1, 333, 256, 4, 128, 2, 128, "bf16")], ids=["batch2", "ragged_end"])
def test_chained_stack_layer_by_layer(shape):
    n_layers = 4
    seed = 9000
    keeps = [0.8, 0.6, 0.4, 0.25]
    buf = ChainedLayerBuffers(ag, shape, extra_rows=2, device=DEV)
    X = [inputs.hidden_states(shape, seed, DEV)] + [torch.full((shape.batch, shape.seq, shape.hidden), float("nan"),
                                                               dtype=shape.torch_dtype, device=DEV) for _ in range(n_layers)]
    tau = float(np.float32(shape.tau))
    for l in range(n_layers):
        W = inputs.layer_weights(shape, inputs.stack_layer_seed(seed, l) + 10, DEV)
        W["Wo_g"] = inputs.randn(tuple(W["Wo_g"].shape), seed + 17 + l, DEV, shape.torch_dtype, 0.5)
        W["Wo"] = inputs.output_weight(shape, inputs.stack_layer_seed(seed, l) + 30, DEV, n_layers)
        # gamma from the oracle's scores of THIS layer's input (an input of both sides)
        s0, _ = T.oracle_gate(shape, X[l], W, None)
        gamma = inputs.calibrate_gamma(torch.from_numpy(s0), [keeps[l]] * shape.heads, tau).to(DEV)
        chained_layer(ag, buf, X[l], W, gamma, X[l + 1])
        torch.cuda.synchronize()
        assert int(buf.status.item()) == 0
        # gate: scores and flags against the oracle on the same hidden states
        s_ref, f_ref = T.oracle_gate(shape, X[l], W, gamma)
        assert np.max(np.abs(T.f64(buf.scores) - s_ref)) < 1e-4
        T.check_flags(shape, buf.flags, s_ref, np.ascontiguousarray(f_ref), gamma)
        fl = buf.flags.cpu().numpy()                      # what the GPU's later calls ran under
        assert abs(fl.mean() - keeps[l]) < 0.05
        # projection (Eq. 2) of the same hidden states, caching under the GPU's flags
        Xd = T.f64(X[l])
        K_ref, V_ref, pc = orc.project_and_cache(Xd, T.f64(W["Wk"]), T.f64(W["Wv"]), fl)
        Q_ref = orc.project_q(Xd, T.f64(W["Wq"]), shape.heads)
        _close_to_rounded(T.f64(buf.Q), Q_ref, f"Q, layer {l}")
        _close_to_rounded(T.f64(buf.K), K_ref, f"K, layer {l}")
        _close_to_rounded(T.f64(buf.V), V_ref, f"V, layer {l}")
        assert np.array_equal(buf.cache.len.cpu().numpy(), orc.cache_lengths(pc).reshape(-1))
        # prefill attention on the Q, K, V the GPU projected (their bf16 values), Eq. 5 from the flags
        O_ref = orc.prefill_attention(T.f64(buf.Q), T.f64(buf.K), T.f64(buf.V), fl)
        T.check_close(T.f64(buf.O), O_ref, "bf16", f"prefill, layer {l}")
        # output projection + skip connection (Eq. 1) of the O the GPU produced
        Y_ref = orc.mha_output(T.f64(buf.O), T.f64(W["Wo"]), Xd)
        _close_to_rounded(T.f64(X[l + 1]), Y_ref, f"hidden states after layer {l}")
    # the hidden states stay of order one through the stack (the weights are scaled for that)
    assert 0.5 < float(X[n_layers].float().std()) < 2.0
    assert ag.ag_device_wait_timeouts() == 0
