"""Benchmark of the AG-gated attention layer on B200.

One step = one pass of the whole hot path over one batch of seeded synthetic
input: gate -> per-head compaction -> masked prefill attention -> D decode
steps (decode attention + conditional append) on the cache just built.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload prefill7b]
    python bench.py --impl reference ...      # the fp64 CPU oracle, timed as it stands

Prints ONE JSON line (rank 0).  `value` is tokens/s with inputs resident in
HBM; `e2e` is the same metric through the C boundary with pinned host buffers
copied in and results copied out inside the timed region.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2410_12876_b200 import inputs  # noqa: E402

METRIC = "prefill & decode tokens/s per AG-gated layer"
UNIT = "tokens/s"
WORKLOADS = {
    # name: (shape, decode steps per step, description)
    "prefill7b": (inputs.PREFILL7B, 16, "Llama-2-7B-shaped AG-gated layer, batch 1 x seq 4096, keep rates U[0.3,0.8] per head"),
    "tiny": (inputs.TINY, 16, "fp32 correctness layer, batch 1 x seq 128, ~50% keep"),
}
# kernels launched per call of the library
LAUNCHES = {"gate": 3, "compact": 2, "prefill": 1, "decode": 2, "append": 1}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu, self.proc, self.path = gpu_index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [r.split(",") for r in open(self.path).read().strip().splitlines() if r.count(",") >= 8]
        os.unlink(self.path)
        if not rows:
            return out
        try:
            sm = np.asarray([float(r[1]) for r in rows])
            power = np.asarray([float(r[3]) for r in rows])
            busy = sm[power >= 0.5 * power.max()] if power.max() > 0 else sm
            out["sm_mhz"] = float(np.median(busy))
            out["sm_max_mhz"] = float(rows[0][2])
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            out["reasons"] = [n for k, n in enumerate(names) if any("Active" in r[5 + k] and "Not" not in r[5 + k] for r in rows)]
            out["samples"] = len(rows)
        except Exception:
            pass
        return out


# ----------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------
class LayerRun:
    """Device buffers of one workload and the five calls of one step."""

    def __init__(self, name, seed, dev):
        from paper_2410_12876_b200 import binding as ag
        self.ag = ag
        self.shape, self.decode_steps, self.desc_text = WORKLOADS[name]
        sh = self.shape
        self.dev = dev
        self.desc = ag.make_desc(sh)
        B, h, n, D = sh.batch, sh.heads, sh.seq, sh.head_dim
        self.X = inputs.hidden_states(sh, seed, dev)
        self.W = inputs.layer_weights(sh, seed + 10, dev)
        self.Q, self.K, self.V = inputs.project_qkv(sh, self.X, self.W)
        self.scores = torch.empty(B, h, n, dtype=torch.float32, device=dev)
        self.flags = torch.empty(B, h, n, dtype=torch.uint8, device=dev)
        self.prefix = torch.empty(B, h, n + 1, dtype=torch.int32, device=dev)
        self.O = torch.empty_like(self.Q)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.ws = {c: ag.workspace(self.desc, c, dev) for c in
                   (ag.AG_CALL_GATE, ag.AG_CALL_COMPACT, ag.AG_CALL_PREFILL, ag.AG_CALL_DECODE)}
        # dense-capacity slabs: n rows + the decode steps of one pass
        self.cache = ag.RaggedCache.allocate(sh, [n + self.decode_steps] * (B * h), dev)
        self.dq = [inputs.decode_inputs(sh, seed + 500, s, dev, keep_new=0.5) for s in range(self.decode_steps)]
        self.o = torch.empty(B, h, D, dtype=sh.torch_dtype, device=dev)
        # gamma: per-head keep rate ~ U[0.3, 0.8], calibrated on the scores at gamma = 0
        self.gamma = None
        self.gate()
        keep = inputs.keep_targets_uniform(h, seed + 20) if name != "tiny" else [0.5] * h
        self.gamma = inputs.calibrate_gamma(self.scores, keep, sh.tau).to(dev)
        self.keep_target = np.asarray(keep)

    def gate(self):
        W, ag = self.W, self.ag
        ag.ag_gate_forward(self.desc, self.X, W["Wq_g"], W["Wk_g"], W["Wv_g"], W["Wo_g"], self.gamma,
                           self.scores, self.flags, self.ws[ag.AG_CALL_GATE])

    def compact(self):
        ag = self.ag
        ag.ag_compact_kv(self.desc, self.K, self.V, self.flags, self.cache, self.prefix, None, self.status,
                         self.ws[ag.AG_CALL_COMPACT])

    def prefill(self):
        ag = self.ag
        ag.ag_prefill_attn(self.desc, self.Q, self.K, self.V, self.flags, self.cache, self.prefix, 0.0, self.O,
                           self.ws[ag.AG_CALL_PREFILL])

    def decode(self, s):
        ag = self.ag
        q, kn, vn, fn = self.dq[s]
        ag.ag_decode_attn(self.desc, q, kn, vn, self.cache, 0.0, self.o, self.ws[ag.AG_CALL_DECODE])
        ag.ag_cache_append(self.desc, kn, vn, fn, self.cache, self.status)

    def step(self, ev=None):
        """One pass; ev (optional) = dict of lists of (start, end) CUDA events per call."""
        def timed(key, fn, *a):
            if ev is None:
                return fn(*a)
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record()
            fn(*a)
            e.record()
            ev[key].append((s, e))
        timed("gate", self.gate)
        timed("compact", self.compact)
        timed("prefill", self.prefill)
        timed("decode", lambda: [self.decode(s) for s in range(self.decode_steps)])

    def tokens_per_step(self):
        return self.shape.batch * (self.shape.seq + self.decode_steps)

    def launches_per_step(self):
        return (LAUNCHES["gate"] + LAUNCHES["compact"] + LAUNCHES["prefill"] +
                self.decode_steps * (LAUNCHES["decode"] + LAUNCHES["append"]))

    def effective_prefill_flops(self):
        """4 D sum_j (1 + P[j]): QK^T and PV over the visible (query, key) pairs only."""
        P = self.prefix[:, :, :-1].to(torch.float64)
        return float(4.0 * self.shape.head_dim * (P.sum() + P.numel()))

    def gate_flops(self):
        sh = self.shape
        GD = sh.gate_heads * sh.gate_head_dim
        rows = sh.batch * sh.seq
        return (2.0 * rows * sh.hidden * 3 * GD + 4.0 * sh.gate_head_dim * sh.gate_heads * sh.batch * sh.seq * (sh.seq + 1) / 2
                + 2.0 * rows * GD * sh.heads)


def flush_l2(buf):
    buf.zero_()


def run_ours(args, rank, world, dev):
    torch.cuda.set_device(dev)
    run = LayerRun(args.workload, 2000 + 100 * rank, dev)
    l2buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist = dist_

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        run.step()
    barrier()
    sampler = ClockSampler(torch.cuda.current_device())
    if rank == 0:
        sampler.start()
    ev = {k: [] for k in ("gate", "compact", "prefill", "decode")}
    step_ev = []
    barrier()
    for _ in range(args.steps):
        flush_l2(l2buf)
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        run.step(ev)
        e.record()
        step_ev.append((s, e))
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = sum(s.elapsed_time(e) for s, e in step_ev)
    per_call_ms = {k: float(np.mean([s.elapsed_time(e) for s, e in v])) for k, v in ev.items()}
    assert int(run.status.item()) == 0, "device reported a cache overflow"

    # end to end: pinned host inputs in, results out, through the same calls
    sh = run.shape
    host_in = [t.detach().cpu().pin_memory() for t in (run.X, run.Q, run.K, run.V)]
    dev_in = [run.X, run.Q, run.K, run.V]
    host_O = torch.empty(run.O.shape, dtype=run.O.dtype).pin_memory()
    host_flags = torch.empty(run.flags.shape, dtype=torch.uint8).pin_memory()
    host_o = torch.empty(run.o.shape, dtype=run.o.dtype).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = sum(t.numel() * t.element_size() for t in (host_O, host_flags, host_o))
    e2e_steps = max(1, min(args.steps, 10))
    barrier()
    t_e2e = 0.0
    for _ in range(e2e_steps):
        flush_l2(l2buf)
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for d, hsrc in zip(dev_in, host_in):
            d.copy_(hsrc, non_blocking=True)
        run.step()
        host_O.copy_(run.O, non_blocking=True)
        host_flags.copy_(run.flags, non_blocking=True)
        host_o.copy_(run.o, non_blocking=True)
        e.record()
        e.synchronize()
        t_e2e += s.elapsed_time(e)
    barrier()

    times = torch.tensor([total_ms, t_e2e], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    total_ms, t_e2e = times.tolist()
    if rank != 0:
        return None
    tokens = run.tokens_per_step() * world
    peaks = _peaks()
    f_eff = run.effective_prefill_flops()
    dom = max(per_call_ms, key=per_call_ms.get)
    prefill_tflops = f_eff / (per_call_ms["prefill"] * 1e-3) / 1e12
    gate_tflops = run.gate_flops() / (per_call_ms["gate"] * 1e-3) / 1e12
    roof = {"bound": "tensor", "kernel": "ag_prefill_attn", "achieved": prefill_tflops, "peak": peaks["bf16_tflops"],
            "unit": "TFLOP/s", "frac": prefill_tflops / peaks["bf16_tflops"], "traffic": None,
            "peak_source": peaks["source"], "algorithmic_flops": f_eff, "ms": per_call_ms["prefill"]}
    ms_step = total_ms / args.steps
    out = {
        "metric": METRIC, "value": tokens * args.steps / (total_ms * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if sh.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": args.workload, "description": run.desc_text, "batch": sh.batch, "seq": sh.seq,
                   "hidden": sh.hidden, "heads": sh.heads, "head_dim": sh.head_dim, "gate_heads": sh.gate_heads,
                   "gate_head_dim": sh.gate_head_dim, "decode_steps_per_step": run.decode_steps,
                   "mean_keep": float(run.flags.float().mean().item()), "l2": "flushed between steps (256 MiB write)",
                   "replicas": world},
        "clocks": clocks,
        "e2e": {"value": tokens * e2e_steps / (t_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": run.launches_per_step() * args.steps,
        "roofline": roof,
        "per_call_ms": per_call_ms,
        "dominant_call": dom,
        "prefill_tokens_per_s": sh.batch * sh.seq / ((per_call_ms["gate"] + per_call_ms["compact"] + per_call_ms["prefill"]) * 1e-3),
        "decode_tokens_per_s": sh.batch * run.decode_steps / (per_call_ms["decode"] * 1e-3),
        "gate_tflops": gate_tflops,
    }
    return out, run


# ----------------------------------------------------------------------------
# the oracle, timed as it stands (cpu_baseline and --impl reference)
# ----------------------------------------------------------------------------
def oracle_sample(name, seed, n_heads_sample=2, decode_steps=2):
    """Time the fp64 oracle on a bounded sample of the workload and scale to a
    whole step.  Sample: the full gate, then compaction + prefill attention +
    `decode_steps` decode steps for `n_heads_sample` of the heads."""
    from oracle import ag_oracle as orc
    shape, dsteps, _ = WORKLOADS[name]
    f64 = inputs.to_f64
    X = inputs.hidden_states(shape, seed, "cpu")
    W = inputs.layer_weights(shape, seed + 10, "cpu")
    hs = min(n_heads_sample, shape.heads)
    D = shape.head_dim
    Wsub = {k: (v[:, :hs * D] if k in ("Wq", "Wk", "Wv") else v) for k, v in W.items()}
    sub = shape.with_(heads=hs)
    Q, K, V = inputs.project_qkv(sub, X, Wsub)
    Xd, Qd, Kd, Vd = f64(X), f64(Q), f64(K), f64(V)
    Wg = [f64(W[k]) for k in ("Wq_g", "Wk_g", "Wv_g", "Wo_g")]
    t0 = time.perf_counter()
    s = orc.gate_scores(Xd, *Wg, shape.gate_heads, causal=bool(shape.gate_causal))
    t_gate = time.perf_counter() - t0
    keep = inputs.keep_targets_uniform(shape.heads, seed + 20) if name != "tiny" else [0.5] * shape.heads
    gamma = inputs.calibrate_gamma(torch.from_numpy(s), keep, shape.tau).numpy().astype(np.float64)
    t0 = time.perf_counter()
    flags = orc.gate_flags(s, gamma, shape.tau)
    t_gate += time.perf_counter() - t0
    fl = flags[:, :hs]
    t0 = time.perf_counter()
    cache = orc.compact_kv(Kd, Vd, fl)
    O = orc.prefill_attention(Qd, Kd, Vd, fl)
    t_heads = time.perf_counter() - t0
    ds = min(decode_steps, dsteps)
    t0 = time.perf_counter()
    for step in range(ds):
        q, kn, vn, fn = inputs.decode_inputs(sub, seed + 500, step, "cpu", keep_new=0.5)
        orc.decode_attention(f64(q), f64(kn), f64(vn), cache)
        orc.cache_append(cache, f64(kn), f64(vn), fn.numpy())
    t_dec = time.perf_counter() - t0
    scale_h = shape.heads / hs
    est = t_gate + scale_h * t_heads + scale_h * t_dec * (dsteps / max(ds, 1))
    tokens = shape.batch * (shape.seq + dsteps)
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = len(os.sched_getaffinity(0))
    return {"value": tokens / est, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": f"full gate + {hs} of {shape.heads} heads of compaction/prefill + {ds} of {dsteps} decode steps, "
                      f"scaled to the whole step (gate {t_gate:.2f}s, heads {t_heads:.2f}s, decode {t_dec:.3f}s)",
            "est_step_s": est}


def run_reference(args, rank, world):
    if rank != 0:
        return None
    shape, dsteps, text = WORKLOADS[args.workload]
    vals = []
    for k in range(args.warmup + args.steps):
        r = oracle_sample(args.workload, 2000, n_heads_sample=1, decode_steps=1)
        if k >= args.warmup:
            vals.append(r)
    est = float(np.mean([r["est_step_s"] for r in vals]))
    tokens = shape.batch * (shape.seq + dsteps)
    v = tokens / est
    base = dict(vals[-1])
    base["value"] = v
    base.pop("est_step_s", None)
    return {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": est * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "description": text},
            "cpu_baseline": base,
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="prefill7b", choices=list(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        out = run_reference(args, rank, world)
        if out is not None:
            print(json.dumps(out))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU path")
    from paper_2410_12876_b200 import build as ag_build
    if rank == 0:
        ag_build.build()
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    res = run_ours(args, rank, world, torch.device("cuda", local))
    if rank == 0:
        out, run = res
        if not args.no_cpu_baseline and world == 1:
            cb = oracle_sample(args.workload, 2000)
            cb.pop("est_step_s", None)
            out["cpu_baseline"] = cb
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
