"""Parity of the local (linear) gate, ag_gate_linear_forward, with the oracle
(Sec. 3.4 "Local or global?", ablation setting (5); threshold of Eq. 4)."""
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


def _run(shape, seed, want_scores=True, gamma="random"):
    X = inputs.hidden_states(shape, seed, DEV)
    W = inputs.linear_gate_weight(shape, seed + 1, DEV)
    B, h, n = shape.batch, shape.heads, shape.seq
    if gamma == "random":
        gamma = torch.from_numpy(np.random.default_rng(seed + 2).uniform(-0.5, 0.5, h).astype(np.float32)).to(DEV)
    scores = torch.full((B, h, n), float("nan"), dtype=torch.float32, device=DEV) if want_scores else None
    flags = torch.full((B, h, n), 7, dtype=torch.uint8, device=DEV)
    ag.ag_gate_linear_forward(ag.make_desc(shape), X, W, gamma, scores, flags)
    torch.cuda.synchronize()
    g = None if gamma is None else T.f64(gamma)
    s_ref, f_ref = orc.linear_gate(T.f64(X), T.f64(W), g, float(np.float32(shape.tau)))
    if want_scores:
        err = np.max(np.abs(T.f64(scores) - s_ref))
        assert err < 1e-4, err
    excluded = T.check_flags(shape, flags, s_ref, np.ascontiguousarray(f_ref), gamma)
    assert excluded < 0.01, excluded
    return flags, f_ref


# (batch, seq, hidden, heads, head_dim, gate_heads, gate_head_dim, dtype); the gate_* fields are unused here
CASES = {
    "bf16_small": LayerShape(2, 333, 512, 8, 128, 2, 128, "bf16"),          # tensor cores, one CTA per 128 tokens
    "bf16_one_token": LayerShape(1, 1, 512, 8, 128, 2, 128, "bf16"),
    "bf16_k_tail": LayerShape(1, 200, 520, 16, 128, 2, 128, "bf16"),        # hidden not a multiple of 64
    "bf16_split_k": LayerShape(1, 700, 4096, 32, 128, 4, 128, "bf16"),      # a cluster splits the hidden dimension
    "bf16_40_heads": LayerShape(1, 300, 1024, 40, 128, 4, 128, "bf16"),     # the 64-column form
    "bf16_12_heads": LayerShape(1, 150, 256, 12, 64, 2, 64, "bf16"),        # W rows not 16-byte multiples: CUDA cores
    "bf16_72_heads": LayerShape(1, 90, 256, 72, 64, 2, 64, "bf16"),         # more heads than the tensor-core form serves
    "f32": LayerShape(1, 150, 128, 3, 128, 1, 128, "f32"),
    "tiny": inputs.TINY,
}


@pytest.mark.parametrize("name", list(CASES))
def test_linear_gate_scores_and_flags(name):
    _run(CASES[name], 700)


def test_linear_gate_without_scores_or_gamma():
    shape = CASES["bf16_small"]
    f1, _ = _run(shape, 710, want_scores=False, gamma=None)
    f2, _ = _run(shape, 710, want_scores=True, gamma=None)
    assert torch.equal(f1, f2)


def test_linear_gate_full_size_layer_feeds_the_cache():
    """The 7B-shaped layer: every score against the oracle, then the flags drive compaction as the
    global gate's do."""
    shape = inputs.PREFILL7B
    flags, f_ref = _run(shape, 720)
    Q, K, V = inputs.qkv_gaussian(shape, 721, DEV)
    fl = torch.from_numpy(np.ascontiguousarray(f_ref)).to(DEV)      # downstream runs on the oracle's flags
    cache, prefix, idx, status = T.gpu_compact(shape, K, V, fl)
    T.check_compaction(shape, K, V, fl, cache, prefix, idx)
    assert ag.ag_device_wait_timeouts() == 0


def test_linear_gate_rejects_bad_arguments():
    shape = CASES["bf16_small"]
    X = inputs.hidden_states(shape, 1, DEV)
    W = inputs.linear_gate_weight(shape, 2, DEV)
    flags = torch.empty(shape.batch, shape.heads, shape.seq, dtype=torch.uint8, device=DEV)
    with pytest.raises(ag.AgError):
        ag.ag_gate_linear_forward(ag.make_desc(shape), X, None, None, None, flags)
    with pytest.raises(ag.AgError):
        ag.ag_gate_linear_forward(ag.make_desc(shape.with_(tau=1.5)), X, W, None, None, flags)
