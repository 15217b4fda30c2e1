"""Parity of ag_out_project with the oracle: the output projection of Eq. 1,
MHA(X) = [H_1 .. H_h] W^O, with the skip connection of a stack of layers added in the same pass.

Every output element is compared with the oracle's float64 value: it may differ by one rounding
to the layer dtype plus float32 summation error.  The shapes take every tile form of the
tensor-core kernel (one or two 128-token sub-tiles per CTA, 256- and 128-column tiles, a split last
wave, sequences that end inside their last sub-tile, sub-tiles of two sequences in one tile)
and the CUDA-core form (float32, head_dim 64, a width the tiles do not divide)."""
import ctypes

import numpy as np
import pytest
import torch

import agtest as T
from oracle import ag_oracle as orc
from paper_2410_12876_b200 import binding as ag
from paper_2410_12876_b200 import inputs
from paper_2410_12876_b200.inputs import LayerShape

DEV = "cuda"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    T.ensure_built()


def _close_to_rounded(got, ref, dtype, what):
    """|got - ref| <= half an ulp of the layer dtype at ref + float32 summation slack."""
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, what
    assert np.all(np.isfinite(got)), what
    rel = 2.0 ** -8 if dtype == "bf16" else 2.0 ** -22
    excess = np.abs(got - ref) - (rel * np.abs(ref) + 2e-5)
    assert np.max(excess) <= 0, f"{what}: {np.max(excess):.3e} beyond one rounding"


SHAPES = {
    # name: (shape, what it reaches)
    "one_sub_tile_per_cta": LayerShape(2, 256, 512, 8, 128, 2, 128, "bf16"),          # 256-column tiles, MT = 1
    "two_sequences_in_a_tile": LayerShape(21, 128, 2048, 8, 128, 2, 128, "bf16"),     # CTA pairs: four sub-tiles per pair tile, each of another sequence; the last pair tile has one
    "split_last_wave": LayerShape(2, 2560, 2048, 4, 128, 2, 128, "bf16"),             # CTA pairs: 10 pair tiles of rows x 8 of columns
    "pairs_one_head": LayerShape(3, 640, 2048, 1, 128, 1, 128, "bf16"),                # CTA pairs with two k-blocks only: fewer than the stages
    "pairs_two_heads": LayerShape(3, 640, 2048, 2, 128, 1, 128, "bf16"),               # four k-blocks: every slice of the skip connection released at the last
    "single_sequence_ragged_end": LayerShape(1, 333, 512, 4, 128, 2, 128, "bf16"),    # the last sub-tile reaches past the sequence
    "columns_128": LayerShape(1, 300, 384, 3, 128, 1, 128, "bf16"),                   # 128-column tiles, odd head count
    "cuda_cores_f32": inputs.TINY,
    "cuda_cores_bf16_d64": LayerShape(2, 150, 256, 4, 64, 2, 64, "bf16"),
    "cuda_cores_odd_width": LayerShape(2, 100, 200, 2, 128, 1, 128, "bf16"),
    "batch_ragged_end": LayerShape(3, 100, 256, 2, 128, 1, 128, "bf16"),              # every sequence ends inside its only sub-tile
    "batch_ragged_two_subtiles": LayerShape(21, 200, 2048, 8, 128, 2, 128, "bf16"),   # CTA pairs, ragged ends
}


@pytest.mark.gpu
@pytest.mark.parametrize("name", list(SHAPES))
@pytest.mark.parametrize("skip", [True, False], ids=["with_skip", "no_skip"])
def test_output_projection(name, skip):
    shape = SHAPES[name]
    B, h, n, D, d = shape.batch, shape.heads, shape.seq, shape.head_dim, shape.hidden
    seed = 8000
    O = inputs.randn((B, h, n, D), seed + 1, DEV, shape.torch_dtype)
    Wo = inputs.randn((h * D, d), seed + 2, DEV, shape.torch_dtype, 0.05)
    X = inputs.hidden_states(shape, seed + 3, DEV) if skip else None
    Y = torch.full((B, n, d), float("nan"), dtype=shape.torch_dtype, device=DEV)
    ag.ag_out_project(ag.make_desc(shape), O, Wo, X, Y)
    torch.cuda.synchronize()
    ref = orc.mha_output(T.f64(O), T.f64(Wo), None if X is None else T.f64(X))
    _close_to_rounded(T.f64(Y), ref, shape.dtype, f"{name}, skip={skip}")
    assert ag.ag_device_wait_timeouts() == 0


@pytest.mark.gpu
def test_layer_output_at_the_7b_shape_on_sampled_tokens():
    """The Llama-2-7B-shaped layer (4096 tokens, 32 heads x 128 -> 4096): two-sub-tile CTAs over
    several waves; the oracle evaluates sampled tokens one by one."""
    shape = inputs.PREFILL7B
    B, h, n, D, d = shape.batch, shape.heads, shape.seq, shape.head_dim, shape.hidden
    O = inputs.randn((B, h, n, D), 8101, DEV, shape.torch_dtype)
    Wo = inputs.output_weight(shape, 8102, DEV)
    X = inputs.hidden_states(shape, 8103, DEV)
    Y = torch.full((B, n, d), float("nan"), dtype=shape.torch_dtype, device=DEV)
    ag.ag_out_project(ag.make_desc(shape), O, Wo, X, Y)
    torch.cuda.synchronize()
    assert torch.isfinite(Y.float()).all()
    toks = np.unique(np.concatenate([[0, 1, 127, 128, 255, 256, n - 129, n - 1],
                                     np.random.default_rng(3).integers(0, n, size=120)]))
    ti = torch.from_numpy(toks).to(DEV)
    ref = orc.mha_output(T.f64(O[:, :, ti]), T.f64(Wo), T.f64(X[:, ti]))
    _close_to_rounded(T.f64(Y[:, ti]), ref, "bf16", "7B-shaped layer")
    assert ag.ag_device_wait_timeouts() == 0


@pytest.mark.gpu
def test_layer_output_at_batch_8_on_cta_pairs():
    """Batch 8 x 4096 tokens (the stack's layer): many waves of tiles, which run on CTA pairs (two CTAs
    share each MMA, each loading half of every W^O stage); the oracle evaluates sampled tokens of
    every sequence."""
    shape = inputs.STACK7B
    B, h, n, D, d = shape.batch, shape.heads, shape.seq, shape.head_dim, shape.hidden
    O = inputs.randn((B, h, n, D), 8201, DEV, shape.torch_dtype)
    Wo = inputs.output_weight(shape, 8202, DEV)
    X = inputs.hidden_states(shape, 8203, DEV)
    Y = torch.full((B, n, d), float("nan"), dtype=shape.torch_dtype, device=DEV)
    ag.ag_out_project(ag.make_desc(shape), O, Wo, X, Y)
    torch.cuda.synchronize()
    assert torch.isfinite(Y.float()).all()
    toks = np.unique(np.concatenate([[0, 127, 128, 255, 256, 383, 384, 511, 512, n - 1],
                                     np.random.default_rng(4).integers(0, n, size=30)]))
    ti = torch.from_numpy(toks).to(DEV)
    ref = orc.mha_output(T.f64(O[:, :, ti]), T.f64(Wo), T.f64(X[:, ti]))
    _close_to_rounded(T.f64(Y[:, ti]), ref, "bf16", "batch-8 layer on CTA pairs")
    # a ragged variant of the same size class: sequences that end inside a sub-tile, on the same path
    shape2 = LayerShape(80, 200, 2048, 8, 128, 2, 128, "bf16")
    O2 = inputs.randn((80, 8, 200, 128), 8211, DEV, torch.bfloat16)
    Wo2 = inputs.randn((1024, 2048), 8212, DEV, torch.bfloat16, 0.05)
    X2 = inputs.hidden_states(shape2, 8213, DEV)
    Y2 = torch.full((80, 200, 2048), float("nan"), dtype=torch.bfloat16, device=DEV)
    ag.ag_out_project(ag.make_desc(shape2), O2, Wo2, X2, Y2)
    torch.cuda.synchronize()
    bsel = torch.tensor([0, 1, 2, 3, 40, 79], device=DEV)
    ref2 = orc.mha_output(T.f64(O2[bsel]), T.f64(Wo2), T.f64(X2[bsel]))
    _close_to_rounded(T.f64(Y2[bsel]), ref2, "bf16", "ragged batch on CTA pairs")
    assert torch.isfinite(Y2.float()).all()
    assert ag.ag_device_wait_timeouts() == 0


def test_argument_checks_on_the_host():
    lib = ag.lib()
    p = 4096
    desc = ag.make_desc(LayerShape(2, 256, 512, 8, 128, 2, 128, "bf16"))
    call = lambda *a: lib.ag_out_project(ctypes.byref(desc), *a, None)
    assert call(None, p, p, 2 * p) == ag.AG_ERR_INVALID_ARG
    assert call(p, None, p, 2 * p) == ag.AG_ERR_INVALID_ARG
    assert call(p, p, p, None) == ag.AG_ERR_INVALID_ARG
    assert call(p, p, p + 4, 2 * p) == ag.AG_ERR_INVALID_ARG          # misaligned skip connection
    assert call(p, p, p, p) == ag.AG_ERR_INVALID_ARG                  # Y must not be X_res
    bad = ag.make_desc(LayerShape(2, 256, 0, 8, 128, 2, 128, "bf16"))
    assert lib.ag_out_project(ctypes.byref(bad), p, p, p, 2 * p, None) == ag.AG_ERR_INVALID_ARG
