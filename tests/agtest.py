"""Shared helpers of the GPU parity tests: run the CUDA calls through the C
boundary and compare with the CPU oracle on the same seeded inputs."""
import math

import numpy as np
import torch

from oracle import ag_oracle as orc
from paper_2410_12876_b200 import binding as ag
from paper_2410_12876_b200 import build as ag_build
from paper_2410_12876_b200 import inputs

f64 = inputs.to_f64

# Tolerances on attention outputs against the fp64 oracle.
#  bf16: the stated bar (max-abs 2e-2, relative L2 1e-2).
#  f32 : float32 accumulation over <= a few thousand terms of O(1) magnitude.
TOL = {"bf16": (2e-2, 1e-2), "f32": (1e-4, 1e-5)}
# Gate scores closer than this to the threshold (in score units, measured on
# the oracle's fp64 scores) are excluded from the bit-exact flag comparison.
FLAG_BAND = 1e-3


def ensure_built():
    ag_build.build()
    return ag.lib()


def bits(t):
    """Raw bit pattern of a float32 / bfloat16 tensor as a numpy integer array."""
    return t.detach().cpu().contiguous().view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32).numpy()


def check_close(got, want, dtype, what=""):
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    max_abs, rel_l2 = TOL[dtype]
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    err = np.max(np.abs(got - want)) if got.size else 0.0
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300) if got.size else 0.0
    assert err <= max_abs, f"{what}: max-abs {err:.3e} > {max_abs}"
    assert rel <= rel_l2, f"{what}: rel-L2 {rel:.3e} > {rel_l2}"
    return err, rel


def gpu_gate(shape, X, W, gamma, want_scores=True):
    desc = ag.make_desc(shape)
    dev = X.device
    B, h, n = shape.batch, shape.kvh, shape.seq              # one flag column per key/value head
    scores = torch.empty(B, h, n, dtype=torch.float32, device=dev) if want_scores else None
    flags = torch.full((B, h, n), 7, dtype=torch.uint8, device=dev)
    ws = ag.workspace(desc, ag.AG_CALL_GATE)
    ag.ag_gate_forward(desc, X, W["Wq_g"], W["Wk_g"], W["Wv_g"], W["Wo_g"], gamma, scores, flags, ws)
    return scores, flags


def oracle_gate(shape, X, W, gamma):
    g = None if gamma is None else f64(gamma)
    tau = float(np.float32(shape.tau))
    return orc.attention_gate(f64(X), f64(W["Wq_g"]), f64(W["Wk_g"]), f64(W["Wv_g"]), f64(W["Wo_g"]),
                              shape.gate_heads, g, tau, causal=bool(shape.gate_causal))


def check_flags(shape, flags_gpu, scores_ref, flags_ref, gamma):
    """Bit-exact outside the band |s + gamma - logit(tau)| < FLAG_BAND;
    returns the fraction of (head, token) pairs inside the band."""
    tau = float(np.float32(shape.tau))
    g = np.zeros(shape.kvh) if gamma is None else f64(gamma)
    dist = np.abs(scores_ref + g[None, :, None] - math.log(tau / (1 - tau)))
    outside = dist >= FLAG_BAND
    fg = flags_gpu.cpu().numpy()
    assert set(np.unique(fg)) <= {0, 1}
    assert np.array_equal(fg[outside], flags_ref[outside])
    return float(1.0 - outside.mean())


def gpu_compact(shape, K, V, flags, cap=None, want_idx=True):
    desc = ag.make_desc(shape)
    dev = flags.device
    B, h, n = shape.batch, shape.kvh, shape.seq              # one cache slab per key/value head
    if cap is None:
        cap = [n] * (B * h)
    cache = ag.RaggedCache.allocate(shape, cap, dev)
    prefix = torch.full((B, h, n + 1), -1, dtype=torch.int32, device=dev)
    idx = torch.full((B, h, n), -1, dtype=torch.int32, device=dev) if want_idx else None
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = None if want_idx else ag.workspace(desc, ag.AG_CALL_COMPACT)
    ag.ag_compact_kv(desc, K, V, flags, cache, prefix, idx, status, ws)
    return cache, prefix, idx, status


def check_compaction(shape, K, V, flags, cache, prefix, idx):
    """prefix, idx, len and the copied rows, all bit-exact against the oracle."""
    fl = flags.cpu().numpy()
    ocache = orc.compact_kv(bits(K), bits(V), fl)
    L = orc.cache_lengths(ocache).reshape(-1)
    assert np.array_equal(cache.len.cpu().numpy(), L)
    pre = prefix.cpu().numpy()
    ix = idx.cpu().numpy() if idx is not None else None
    kr, vr = bits(cache.k_rows), bits(cache.v_rows)
    off = cache.row_off.cpu().numpy()
    for b in range(shape.batch):
        for i in range(shape.kvh):
            s = b * shape.kvh + i
            c = ocache[b][i]
            assert np.array_equal(pre[b, i], orc.exclusive_counts(fl[b, i]))
            if ix is not None:
                assert np.array_equal(ix[b, i, :L[s]], c["idx"])
            assert np.array_equal(kr[off[s]:off[s] + L[s]], c["k"])
            assert np.array_equal(vr[off[s]:off[s] + L[s]], c["v"])


def gpu_prefill(shape, Q, K, V, flags, cache, prefix, scale=0.0):
    desc = ag.make_desc(shape)
    O = torch.full_like(Q, float("nan"))
    ag.ag_prefill_attn(desc, Q, K, V, flags, cache, prefix, scale, O, ag.workspace(desc, ag.AG_CALL_PREFILL))
    return O


def gpu_decode_step(shape, q, kn, vn, fn, cache, status, ws=None, scale=0.0, fused=False):
    """One decode step: ag_decode_attn + ag_cache_append, or ag_decode_step (both in one call)."""
    desc = ag.make_desc(shape)
    if ws is None:
        ws = ag.workspace(desc, ag.AG_CALL_DECODE)
    o = torch.full_like(q, float("nan"))
    if fused:
        ag.ag_decode_step(desc, q, kn, vn, fn, cache, scale, o, status, ws)
    else:
        ag.ag_decode_attn(desc, q, kn, vn, cache, scale, o, ws)
        ag.ag_cache_append(desc, kn, vn, fn, cache, status)
    return o


def gpu_cache_as_lists(cache, shape):
    """The valid rows of a device cache as per-slab fp64 arrays (exact widening),
    for comparison with the oracle's cache; never used as an oracle input."""
    L = cache.len.cpu().numpy()
    off = cache.row_off.cpu().numpy()
    kr, vr = f64(cache.k_rows), f64(cache.v_rows)
    out = []
    for b in range(shape.batch):
        row = []
        for i in range(shape.kvh):
            s = b * shape.kvh + i
            row.append({"k": kr[off[s]:off[s] + L[s]].copy(), "v": vr[off[s]:off[s] + L[s]].copy()})
        out.append(row)
    return out
