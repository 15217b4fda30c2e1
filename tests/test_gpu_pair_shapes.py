"""Seeded random shapes that reach the CTA-pair forms of the projection GEMMs (more than one wave of
tiles): ragged sequence ends, pair tiles whose sub-tiles belong to several sequences, halved last
waves, few and many k-blocks - against the same oracle checks as the fixed cases."""
import numpy as np
import pytest
import torch

import agtest as T
import test_gpu_kv_project as kvp
import test_gpu_out_project as outp
from oracle import ag_oracle as orc
from paper_2410_12876_b200 import binding as ag
from paper_2410_12876_b200 import inputs
from paper_2410_12876_b200.inputs import LayerShape

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    T.ensure_built()


def _shapes(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        heads = int(rng.choice([2, 4, 6, 8, 16]))
        hidden = int(rng.choice([256, 512, 768, 1024, 2048]))
        batch, seq = int(rng.integers(1, 13)), int(rng.integers(100, 2000))
        tiles = batch * ((seq + 127) // 128)
        # both GEMMs beyond two waves of 128-row tiles on 148 SMs (with room: SM counts differ little), and
        # small enough for the oracle
        if (hidden // 128) * tiles > 320 and 3 * heads * tiles > 320 and batch * seq * hidden * heads <= 60_000_000:
            out.append(LayerShape(batch, seq, hidden, heads, 128, max(1, heads // 4), 128, "bf16"))
    return out


SHAPES = _shapes(6, 20241201)


@pytest.mark.parametrize("k", range(len(SHAPES)))
def test_projection_and_cache_on_random_pair_shapes(k):
    kvp._check(SHAPES[k], 9100 + k, with_q=bool(k & 1))


@pytest.mark.parametrize("k", range(len(SHAPES)))
def test_output_projection_on_random_pair_shapes(k):
    shape = SHAPES[k]
    B, h, n, D, d = shape.batch, shape.heads, shape.seq, shape.head_dim, shape.hidden
    O = inputs.randn((B, h, n, D), 9200 + k, DEV, shape.torch_dtype)
    Wo = inputs.randn((h * D, d), 9300 + k, DEV, shape.torch_dtype, 0.05)
    X = inputs.hidden_states(shape, 9400 + k, DEV)
    Y = torch.full((B, n, d), float("nan"), dtype=shape.torch_dtype, device=DEV)
    ag.ag_out_project(ag.make_desc(shape), O, Wo, X, Y)
    torch.cuda.synchronize()
    outp._close_to_rounded(T.f64(Y), orc.mha_output(T.f64(O), T.f64(Wo), T.f64(X)), shape.dtype, f"shape {k}")
    assert ag.ag_device_wait_timeouts() == 0
