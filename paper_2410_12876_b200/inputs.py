"""Seeded synthetic inputs for the AG-gated attention layer.

This module only draws random tensors and lays out buffers.  It contains none
of the layer's arithmetic (no gate, no mask, no softmax): both the CUDA path
and the CPU checker are fed from here, so nothing in it may be something
either of them is meant to verify.  The only linear algebra is the upstream
Q/K/V projection X W (Eq. 2's inputs), which lies outside the layer.

Shapes follow Llama-2-7B (d = 4096, 32 heads x 128) with the AG size the
paper's ablation table uses (4 gate heads x 128), and keep rates span the
eviction range its result tables report (roughly 35-70 % evicted).
"""
from dataclasses import dataclass, replace
import math

import numpy as np
import torch


@dataclass(frozen=True)
class LayerShape:
    batch: int
    seq: int
    hidden: int
    heads: int
    head_dim: int
    gate_heads: int
    gate_head_dim: int
    dtype: str = "bf16"        # "f32" | "bf16"
    tau: float = 0.5
    gate_causal: int = 1
    kv_heads: int = 0          # key/value heads (grouped-query attention); 0 = one per query head
    recent_window: int = 0     # recent tokens always visible, the current one included; 0 or 1 = itself only

    @property
    def kvh(self):
        return self.kv_heads if self.kv_heads > 0 else self.heads

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def with_(self, **kw):
        return replace(self, **kw)


# The five workloads.  "tiny" is the fp32 correctness layer; "prefill7b" is
# the Llama-2-7B-shaped layer the headline number is quoted on.
TINY = LayerShape(1, 128, 256, 4, 64, 2, 64, "f32")
PREFILL7B = LayerShape(1, 4096, 4096, 32, 128, 4, 128, "bf16")
DECODE_RAGGED = LayerShape(32, 8192, 4096, 32, 128, 4, 128, "bf16")
DEEP_LAYER = LayerShape(1, 16384, 4096, 32, 128, 4, 128, "bf16")
STACK7B = LayerShape(8, 4096, 4096, 32, 128, 4, 128, "bf16")
# grouped-query variant of the ragged decode shape (Mistral-7B-like: 32 query heads over 8 key/value heads)
DECODE_RAGGED_GQA = LayerShape(32, 8192, 4096, 32, 128, 4, 128, "bf16", kv_heads=8)


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def randn(shape, seed, device="cpu", dtype=torch.float32, std=1.0):
    """N(0, std^2) drawn in float32 with a seeded generator, rounded once."""
    t = torch.randn(*shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    if std != 1.0:
        t = t * std
    return t.to(dtype)


def hidden_states(shape, seed, device="cpu"):
    """X [B, n, d] ~ N(0, 1)."""
    return randn((shape.batch, shape.seq, shape.hidden), seed, device, shape.torch_dtype)


def layer_weights(shape, seed, device="cpu"):
    """All projection weights ~ N(0, 0.02), stored "in x out"."""
    d, hD, gD = shape.hidden, shape.heads * shape.head_dim, shape.gate_heads * shape.gate_head_dim
    kD = shape.kvh * shape.head_dim
    dt = shape.torch_dtype
    return {
        "Wq": randn((d, hD), seed + 1, device, dt, 0.02),
        "Wk": randn((d, kD), seed + 2, device, dt, 0.02),
        "Wv": randn((d, kD), seed + 3, device, dt, 0.02),
        "Wq_g": randn((d, gD), seed + 4, device, dt, 0.02),
        "Wk_g": randn((d, gD), seed + 5, device, dt, 0.02),
        "Wv_g": randn((d, gD), seed + 6, device, dt, 0.02),
        "Wo_g": randn((gD, shape.kvh), seed + 7, device, dt, 0.02),      # one flag column per key/value head
    }


def output_weight(shape, seed, device="cpu", n_layers=1):
    """W^O [h D, d] of Eq. 1 ~ N(0, 0.02 / sqrt(2 n_layers)): with the skip connection of a stack of
    n_layers layers and nothing that normalises between them, the hidden states keep their scale."""
    return randn((shape.heads * shape.head_dim, shape.hidden), seed, device, shape.torch_dtype,
                 0.02 / math.sqrt(2.0 * n_layers))


def linear_gate_weight(shape, seed, device="cpu"):
    """W_lin [d, h] ~ N(0, 1/d) for the local gate (scores of O(1) for unit-variance hidden states)."""
    return randn((shape.hidden, shape.heads), seed, device, shape.torch_dtype, 1.0 / math.sqrt(shape.hidden))


def project_qkv(shape, X, W):
    """Upstream projection Q_i = X W^Q_i etc. -> Q [B, h, n, D], K, V [B, h_kv, n, D] in
    the layer dtype.  float64 accumulate for the fp32 layer, float32 otherwise."""
    acc = torch.float64 if shape.dtype == "f32" else torch.float32
    out = []
    for name in ("Wq", "Wk", "Wv"):
        y = (X.to(acc) @ W[name].to(acc)).to(shape.torch_dtype)
        heads = shape.heads if name == "Wq" else shape.kvh
        y = y.view(shape.batch, shape.seq, heads, shape.head_dim).permute(0, 2, 1, 3)
        out.append(y.contiguous())
    return out


def qkv_gaussian(shape, seed, device="cpu", std=1.0):
    """Q, K, V ~ N(0, std^2) directly (workloads that give no hidden size)."""
    sq = (shape.batch, shape.heads, shape.seq, shape.head_dim)
    skv = (shape.batch, shape.kvh, shape.seq, shape.head_dim)
    return [randn(sq if k == 0 else skv, seed + k, device, shape.torch_dtype, std) for k in range(3)]


def stack_layer_seed(seed, layer):
    """Seed base of layer `layer` of a stack: every layer has its own hidden states and weights."""
    return int(seed) + 1000 * (int(layer) + 1)


def stack_layer_inputs(shape, seed, layer, device="cpu"):
    """Hidden states X_l ~ N(0, 1), weights ~ N(0, 0.02) and the upstream projections Q, K, V of one
    layer of a stack, all seeded by the layer's number."""
    base = stack_layer_seed(seed, layer)
    X = hidden_states(shape, base, device)
    W = layer_weights(shape, base + 10, device)
    Q, K, V = project_qkv(shape, X, W)
    return X, W, Q, K, V


def keep_targets_uniform(heads, seed, lo=0.3, hi=0.8):
    """Per-head target keep rate ~ U[lo, hi]."""
    return np.random.default_rng(seed).uniform(lo, hi, size=heads)


def keep_targets_layer(heads, seed, layer, n_layers=32):
    """Per-head keep rate for layer `layer` of a stack whose mean eviction
    rises linearly from 10 % (first layer) to 90 % (last)."""
    mean_keep = 1.0 - (0.10 + 0.80 * layer / max(1, n_layers - 1))
    jitter = np.random.default_rng(seed + layer).uniform(-0.05, 0.05, size=heads)
    return np.clip(mean_keep + jitter, 0.02, 0.98)


def calibrate_gamma(scores_gamma0, keep, tau):
    """Per-head additive constant that makes a fraction keep[i] of the tokens
    of head i land above the threshold, given the scores the gate produced
    with gamma = 0.  The cut is placed midway between two adjacent order
    statistics so that no score sits on the threshold.  scores [B, h, n]."""
    s = scores_gamma0.detach().to("cpu", torch.float64).numpy()
    B, h, n = s.shape
    cut_logit = math.log(tau / (1.0 - tau))
    gamma = np.zeros(h, dtype=np.float64)
    for i in range(h):
        v = np.sort(s[:, i, :].reshape(-1))
        m = v.size
        n_keep = int(round(float(keep[i]) * m))
        n_keep = min(max(n_keep, 0), m)
        if n_keep == 0:
            cut = v[-1] + 1.0
        elif n_keep == m:
            cut = v[0] - 1.0
        else:
            cut = 0.5 * (v[m - n_keep - 1] + v[m - n_keep])
        gamma[i] = cut_logit - cut
    return torch.from_numpy(gamma.astype(np.float32))


def bernoulli_flags(shape_tuple, p, seed):
    """uint8 array of i.i.d. Bernoulli(p) keep flags."""
    r = np.random.default_rng(seed).random(size=shape_tuple)
    return torch.from_numpy((r < p).astype(np.uint8))


def deep_layer_flags(shape, seed, n_empty=8, keep=0.1):
    """Deep-layer pattern: `n_empty` heads (seeded choice) evict everything,
    the others keep i.i.d. Bernoulli(keep).  Returns (flags [B, h, n], empty_heads)."""
    rng = np.random.default_rng(seed)
    empty = np.sort(rng.permutation(shape.heads)[:n_empty])
    f = (rng.random(size=(shape.batch, shape.heads, shape.seq)) < keep).astype(np.uint8)
    f[:, empty, :] = 0
    return torch.from_numpy(f), empty


def ragged_lengths(n_slabs, L, seed, lo=0.2, hi=0.9):
    """Retained length per slab ~ U{ceil(lo L) .. floor(hi L)}."""
    a, b = math.ceil(lo * L), math.floor(hi * L)
    return np.random.default_rng(seed).integers(a, b + 1, size=n_slabs).astype(np.int32)


def slab_layout(cap):
    """Tight back-to-back slabs: row_off[s] = sum of cap[:s]; returns
    (row_off int64, pool_rows)."""
    cap = np.asarray(cap, dtype=np.int64)
    off = np.zeros(cap.size, dtype=np.int64)
    if cap.size > 1:
        off[1:] = np.cumsum(cap[:-1])
    return off, int(cap.sum())


def decode_inputs(shape, seed, step, device="cpu", keep_new=0.5):
    """q [B, h, D], k_new, v_new [B, h_kv, D] ~ N(0, 1) and flag_new [B, h_kv] for one step."""
    s = (shape.batch, shape.heads, shape.head_dim)
    skv = (shape.batch, shape.kvh, shape.head_dim)
    base = seed + 10 * step
    q = randn(s, base + 1, device, shape.torch_dtype)
    k = randn(skv, base + 2, device, shape.torch_dtype)
    v = randn(skv, base + 3, device, shape.torch_dtype)
    if keep_new >= 1.0:
        f = torch.ones(shape.batch, shape.kvh, dtype=torch.uint8)
    else:
        f = bernoulli_flags((shape.batch, shape.kvh), keep_new, base + 4)
    return q, k, v, f.to(device)


def to_f64(t):
    """Exact widening of a float32 / bfloat16 tensor to a float64 numpy array."""
    return t.detach().to("cpu", torch.float32).to(torch.float64).numpy()
