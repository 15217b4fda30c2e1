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
    "prefill7b_proj": (inputs.PREFILL7B, 16, "the prefill7b layer owning its projection: Q, K, V = X [Wq | Wk | Wv] are computed in the "
                                             "step and the retained rows go straight into the cache (ag_qkv_project_cache in place of ag_compact_kv)"),
    "tiny": (inputs.TINY, 16, "fp32 correctness layer, batch 1 x seq 128, ~50% keep"),
    "deep_layer": (inputs.DEEP_LAYER, 128, "deep-layer pattern, batch 1 x seq 16384: 24 heads keep ~10%, 8 heads keep nothing"),
    "stack7b": (inputs.STACK7B, 256, "32 AG-gated layers back to back, batch 8 x seq 4096; per-layer mean eviction rising from 10% to 90%"),
    "stack7b_prev": (inputs.STACK7B, 256, "the stack7b layers with eviction guided by the previous layer (ablation setting 4-1): "
                                         "layer l runs under the flags of layer l-1's gate, the first layer evicts nothing, "
                                         "each gate pass runs on a second stream beside its layer's attention"),
    "prefill7b_out": (inputs.PREFILL7B, 16, "the prefill7b layer from hidden states to hidden states: gate, Q, K, V projection into the cache, "
                                           "prefill attention, output projection with the skip connection (Eq. 1), 16 decode steps"),
    "stack7b_chain": (inputs.STACK7B, 256, "32 chained AG-gated layers, batch 8 x seq 4096: every layer projects its Q, K, V from the "
                                          "hidden states the previous layer produced, X_{l+1} = X_l + [H_1 .. H_h] W^O (no normalisation, "
                                          "no feed-forward block in between); per-layer mean eviction rising from 10% to 90%"),
    "decode_ragged": (inputs.DECODE_RAGGED, 256, "ragged decode, batch 32 x 32 heads, retained lengths U[0.2,0.9] x 8192, keep-new Bernoulli(0.5)"),
    "decode_ragged_gqa": (inputs.DECODE_RAGGED_GQA, 256, "ragged decode with grouped-query attention, batch 32 x 32 query heads over 8 key/value heads, retained lengths U[0.2,0.9] x 8192"),
}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (None for workloads that were not captured).  To be reset to
# None whenever the kernel changes after the capture.
TRAFFIC = {
    ("prefill7b", "prefill"): 155.20e6 + 17.45e6,        # prefill_tc_kernel
    ("prefill7b", "decode"): 41.22e6 + 0.003e6,          # decode_cluster_mma_kernel
    ("prefill7b", "compact"): 41.26e6 + 2.46e6,          # compact_kernel<256> (written rows still in L2 at kernel end)
    ("prefill7b", "kv_project_cache"): 182.23e6 + 82.20e6,   # kv_proj_cache_pair_kernel
    ("prefill7b_proj", "prefill"): 155.20e6 + 17.45e6,
    ("prefill7b_proj", "decode"): 41.22e6 + 0.003e6,
    ("prefill7b_proj", "project"): 251.70e6 + 121.58e6,  # kv_proj_cache_pair_kernel with the query projection
    ("prefill7b_out", "prefill"): 155.20e6 + 17.45e6,
    ("prefill7b_out", "project"): 251.70e6 + 121.58e6,
    ("prefill7b_out", "out_project"): 132.63e6 + 16.75e6,    # out_proj_pair_kernel
    ("deep_layer", "prefill"): 364.64e6 + 106.70e6,      # prefill_tc_kernel
    ("deep_layer", "compact"): 20.48e6 + 0.34e6,         # compact_kernel<256>
    ("decode_ragged", "decode"): 2.3530e9 + 7.1e6,       # decode_partial_kernel<bf16,128>
}
# kernels launched per call of the library
# (decode step, attention + append: one cluster kernel up to DECODE_CLUSTER_MAX_SLABS slabs, else chunk pass + merge)
LAUNCHES = {"gate": 3, "compact": 1, "prefill": 1, "decode": 2}
DECODE_CLUSTER_MAX_SLABS = 64
L2_BYTES = 126e6
MIN_TIMED_S = 0.6     # a run's timed region lasts at least about this long


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler:
    """SM clock and throttle reasons sampled through NVML (read-only) every few milliseconds
    while the timed region runs; falls back to polling nvidia-smi when NVML is not importable."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, gpu_index):
        import threading
        self.gpu, self.samples, self.stop_flag = gpu_index, [], threading.Event()
        self.thread, self.max_mhz, self.proc, self.path = None, None, None, None

    def _nvml_index(self):
        vis = os.environ.get("CUDA_VISIBLE_DEVICES")
        if vis:
            ids = [v.strip() for v in vis.split(",") if v.strip()]
            if self.gpu < len(ids) and ids[self.gpu].isdigit():
                return int(ids[self.gpu])
        return self.gpu

    def start(self):
        import threading
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(self._nvml_index())
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))

            def loop():
                while not self.stop_flag.is_set():
                    try:
                        self.samples.append((float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)),
                                             int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)),
                                             pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0))
                    except Exception:
                        pass
                    time.sleep(0.004)
            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
        except Exception:
            self.thread = None
            try:
                fd, self.path = tempfile.mkstemp(suffix=".csv")
                os.close(fd)
                q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active"
                self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                              "-lms", "20", "-i", str(self._nvml_index())],
                                             stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
            except Exception:
                self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        if self.thread is not None:
            self.stop_flag.set()
            self.thread.join(timeout=2)
            if self.samples:
                sm = np.asarray([x[0] for x in self.samples])
                pw = np.asarray([x[2] for x in self.samples])
                busy = sm[pw >= 0.5 * pw.max()] if pw.max() > 0 else sm
                bits = 0
                for x in self.samples:
                    bits |= x[1]
                out.update(sm_mhz=float(np.median(busy)), samples=len(self.samples), power_w_max=float(pw.max()),
                           reasons=[n for b, n in self.REASONS.items() if bits & b])
            return out
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            rows = [r.split(",") for r in open(self.path).read().strip().splitlines() if r.count(",") >= 3]
            os.unlink(self.path)
            try:
                sm = np.asarray([float(r[0]) for r in rows])
                bits = 0
                for r in rows:
                    bits |= int(r[3].strip(), 16)
                out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(rows[0][1]), samples=len(rows),
                           reasons=[n for b, n in self.REASONS.items() if bits & b])
            except Exception:
                pass
        return out


# ----------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------
class LayerRun:
    """Device buffers of one workload and the five calls of one step."""

    def __init__(self, name, seed, dev, recent_window=0):
        from paper_2410_12876_b200 import binding as ag
        self.ag = ag
        self.shape, self.decode_steps, self.desc_text = WORKLOADS[name]
        if recent_window > 1:
            assert name not in ("decode_ragged", "decode_ragged_gqa"), "the window needs a prompt to fill its ring from"
            self.shape = self.shape.with_(recent_window=recent_window)
        sh = self.shape
        self.dev = dev
        self.desc = ag.make_desc(sh)
        B, h, n, D = sh.batch, sh.heads, sh.seq, sh.head_dim
        self.name = name
        self.use_graph = True
        self._groups = {}
        self.has_gate = name in ("prefill7b", "prefill7b_proj", "prefill7b_out", "tiny", "stack7b", "stack7b_prev", "stack7b_chain")
        self.chain = name in ("stack7b_chain", "prefill7b_out")     # layer l + 1 runs on layer l's output
        self.project = name == "prefill7b_proj" or self.chain       # Q, K, V are computed in the step
        self.layers = 32 if name.startswith("stack7b") else 1
        self.first_gated = 1 if name == "stack7b_prev" else 0      # 0: every layer evicts by its own gate
        self.has_prefill = name not in ("decode_ragged", "decode_ragged_gqa")
        if self.chain:
            # one X_0; every layer has its own weights (Wq, Wk, Wv, Wo and the gate's); the hidden states
            # of the later layers are produced by the stack itself, in two buffers used in turn
            self.X0 = inputs.hidden_states(sh, seed, dev)
            self.Xbuf = [torch.empty_like(self.X0), torch.empty_like(self.X0)]
            self.Ws = []
            for l in range(self.layers):
                W = inputs.layer_weights(sh, inputs.stack_layer_seed(seed, l) + 10, dev)
                W["Wo"] = inputs.output_weight(sh, inputs.stack_layer_seed(seed, l) + 30, dev, self.layers)
                self.Ws.append(W)
            self.X, self.W = self.X0, self.Ws[0]
            self.Q = torch.empty(B, h, n, D, dtype=sh.torch_dtype, device=dev)
            self.K = torch.empty(B, sh.kvh, n, D, dtype=sh.torch_dtype, device=dev)
            self.V = torch.empty_like(self.K)
            self.K2, self.V2 = self.K, self.V
        elif self.has_gate and self.layers > 1:
            # every layer of a stack has its own hidden states X_l, weights and upstream Q, K, V
            self.layer_in = [inputs.stack_layer_inputs(sh, seed, l, dev) for l in range(self.layers)]
            self.X, self.W, self.Q, self.K, self.V = self.layer_in[0]
        elif self.has_gate:
            self.X = inputs.hidden_states(sh, seed, dev)
            self.W = inputs.layer_weights(sh, seed + 10, dev)
            self.Q, self.K, self.V = inputs.project_qkv(sh, self.X, self.W)
            if self.project:
                self.K2, self.V2 = self.K, self.V                  # the step writes them itself
        elif self.has_prefill:
            self.Q, self.K, self.V = inputs.qkv_gaussian(sh, seed, dev)
        else:
            self.Q = torch.empty(0, dtype=sh.torch_dtype, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        calls = [ag.AG_CALL_DECODE] + ([ag.AG_CALL_COMPACT, ag.AG_CALL_PREFILL] if self.has_prefill else []) \
            + ([ag.AG_CALL_GATE] if self.has_gate else [])
        self.ws = {c: ag.workspace(self.desc, c, dev) for c in calls}
        if self.has_prefill:
            self.scores = torch.empty(B, h, n, dtype=torch.float32, device=dev)
            self.flags = torch.empty(B, h, n, dtype=torch.uint8, device=dev)
            self.cur_flags = self.flags                             # what compaction and prefill run under
            self.prefix = torch.empty(B, h, n + 1, dtype=torch.int32, device=dev)
            self.O = torch.empty_like(self.Q)
            # dense-capacity slabs: n rows + the decode steps of one pass
            self.cache = ag.RaggedCache.allocate(sh, [n + self.decode_steps] * (B * h), dev)
        else:
            # the cache is the input: tight slabs of seeded random length, filled with N(0, 1)
            self.L0 = inputs.ragged_lengths(B * sh.kvh, n, seed + 30)       # one slab per key/value head
            self.cache = ag.RaggedCache.allocate(sh, (self.L0.astype(np.int64) + 256).tolist(), dev)
            for t, sd in ((self.cache.k_rows, seed + 31), (self.cache.v_rows, seed + 32)):
                step_rows = 1 << 20
                for r0 in range(0, t.shape[0], step_rows):
                    r1 = min(t.shape[0], r0 + step_rows)
                    t[r0:r1] = inputs.randn((r1 - r0, D), sd + r0, dev, sh.torch_dtype)
            self.len0 = torch.from_numpy(self.L0).to(dev)
            self.cache.len.copy_(self.len0)
        # new-token flags: Bernoulli(0.1) on the deep layer, every token kept in the stack (the paper's
        # decode stage runs no gate), Bernoulli(0.5) elsewhere
        keep_new = 0.1 if name == "deep_layer" else 1.0 if self.layers > 1 else 0.5
        # decode tokens: one list of steps per layer (a stack's layers each decode their own)
        self.dqs = [[inputs.decode_inputs(sh, inputs.stack_layer_seed(seed, l) + 500 if self.layers > 1 else seed + 500,
                                          s, dev, keep_new=keep_new) for s in range(self.decode_steps)]
                    for l in range(self.layers)]
        # the decode tokens of a layer live in ONE device buffer (the tensors above become views of it), so that
        # the end-to-end pass sends them with one copy instead of four small ones per step
        self.dq_flat = []
        for l, dq in enumerate(self.dqs):
            sizes = [t.numel() * t.element_size() for q in dq for t in q]
            offs = np.concatenate([[0], np.cumsum([(x + 255) // 256 * 256 for x in sizes])])
            flat = torch.empty(int(offs[-1]), dtype=torch.uint8, device=dev)
            views, k = [], 0
            for q in dq:
                step = []
                for t in q:
                    v = flat[int(offs[k]):int(offs[k]) + sizes[k]].view(t.dtype).view(t.shape)
                    v.copy_(t)
                    step.append(v)
                    k += 1
                views.append(tuple(step))
            self.dqs[l] = views
            self.dq_flat.append(flat)
        self.dq = self.dqs[0]
        self.layer = 0
        self.graphs = {}
        self.o = torch.empty(B, h, D, dtype=sh.torch_dtype, device=dev)
        # gamma: per-head keep rate ~ U[0.3, 0.8], calibrated on the scores at gamma = 0
        self.gamma = None
        if self.chain:
            # gamma of layer l is calibrated on the hidden states the stack itself hands to layer l
            self.gammas = []
            for l in range(self.layers):
                self.set_layer(l)
                self.gamma = None
                self.gate()
                keep = inputs.keep_targets_layer(h, seed + 20, l) if self.layers > 1 else inputs.keep_targets_uniform(h, seed + 20)
                self.gammas.append(inputs.calibrate_gamma(self.scores, keep, sh.tau).to(dev))
                self.gamma = self.gammas[l]
                self.gate()
                self.kv_project_cache()
                self.prefill()
                self.out_project()
            self.set_layer(0)
            self.gamma = self.gammas[0]
        elif self.has_gate:
            if self.layers > 1:
                # per layer: mean eviction 10 % (first) ... 90 % (last), gamma calibrated on the layer's
                # own scores at gamma = 0
                self.gammas = []
                for l in range(self.layers):
                    self.set_layer(l)
                    self.gamma = None
                    self.gate()
                    self.gammas.append(inputs.calibrate_gamma(self.scores, inputs.keep_targets_layer(h, seed + 20, l),
                                                              sh.tau).to(dev))
                self.set_layer(0)
            else:
                self.gate()
                keep = inputs.keep_targets_uniform(h, seed + 20) if name != "tiny" else [0.5] * h
                self.gammas = [inputs.calibrate_gamma(self.scores, keep, sh.tau).to(dev)]
            self.gamma = self.gammas[0]
        elif self.has_prefill:
            f, empty = inputs.deep_layer_flags(sh, seed + 20)
            self.flags.copy_(f.to(dev))
            for q in self.dq:
                q[3][:, torch.from_numpy(empty).to(dev)] = 0     # fully evicted heads stay empty

    def set_layer(self, layer):
        """Point the calls at the inputs of layer `layer` (a stack; a single layer has only layer 0)."""
        self.layer = layer
        self.dq = self.dqs[layer]
        if self.chain:
            self.X = self.X0 if layer == 0 else self.Xbuf[(layer - 1) % 2]
            self.X_next = self.Xbuf[layer % 2]
            self.W = self.Ws[layer]
        elif self.layers > 1 and self.has_gate:
            self.X, self.W, self.Q, self.K, self.V = self.layer_in[layer]

    def out_project(self):
        """The layer's output (Eq. 1) with the skip connection: the next layer's hidden states."""
        self.ag.ag_out_project(self.desc, self.O, self.W["Wo"], self.X, self.X_next)

    def gate(self, flags_out=None):
        W, ag = self.W, self.ag
        ag.ag_gate_forward(self.desc, self.X, W["Wq_g"], W["Wk_g"], W["Wv_g"], W["Wo_g"], self.gamma,
                           self.scores, self.flags if flags_out is None else flags_out, self.ws[ag.AG_CALL_GATE])

    def gate_linear(self):
        """The local gate (Sec. 3.4): same X, one [d, h] weight; timed on its own, not part of a step."""
        if not hasattr(self, "W_lin"):
            self.W_lin = inputs.linear_gate_weight(self.shape, 2900, self.X.device)
            self.flags_lin = torch.empty_like(self.flags)
        self.ag.ag_gate_linear_forward(self.desc, self.X, self.W_lin, None, self.scores, self.flags_lin)

    def kv_project_cache(self):
        """Eq. 2's key/value projection with the retained rows written straight into the cache
        (ag_kv_project_cache): what a layer that owns its K/V projection runs in place of
        projection + compaction; timed on its own, not part of a step."""
        ag = self.ag
        if not hasattr(self, "K2"):
            self.K2, self.V2 = torch.empty_like(self.K), torch.empty_like(self.V)
        if self.project:           # the layer owns its whole Q, K, V projection
            return ag.ag_qkv_project_cache(self.desc, self.X, self.W["Wq"], self.W["Wk"], self.W["Wv"], self.cur_flags,
                                           self.cache, self.prefix, None, self.Q, self.K2, self.V2, self.status)
        ag.ag_kv_project_cache(self.desc, self.X, self.W["Wk"], self.W["Wv"], self.cur_flags, self.cache, self.prefix,
                               None, self.K2, self.V2, self.status)

    def _group(self, g):
        """Descriptor and cache view of the heads g = (first, last + 1) of a batch-1 layer (the calls
        of a layer work on any subset of its heads: every (sequence, head) is independent)."""
        if g not in self._groups:
            assert self.shape.batch == 1 and self.shape.kv_heads == 0 and self.shape.recent_window <= 1
            ag, c = self.ag, self.cache
            view = ag.RaggedCache(c.k_rows, c.v_rows, c.row_off[g[0]:g[1]], c.cap[g[0]:g[1]], c.len[g[0]:g[1]], c.max_cap)
            self._groups[g] = (ag.make_desc(self.shape.with_(heads=g[1] - g[0])), view)
        return self._groups[g]

    def compact(self, g=None):
        ag = self.ag
        if g is not None:
            desc, cache = self._group(g)
            return ag.ag_compact_kv(desc, self.K[:, g[0]:g[1]], self.V[:, g[0]:g[1]], self.cur_flags[:, g[0]:g[1]], cache,
                                    self.prefix[:, g[0]:g[1]], None, self.status, self.ws[ag.AG_CALL_COMPACT])
        ag.ag_compact_kv(self.desc, self.K, self.V, self.cur_flags, self.cache, self.prefix, None, self.status,
                         self.ws[ag.AG_CALL_COMPACT])

    def prefill(self, g=None):
        ag = self.ag
        if g is not None:
            desc, cache = self._group(g)
            return ag.ag_prefill_attn(desc, self.Q[:, g[0]:g[1]], self.K[:, g[0]:g[1]], self.V[:, g[0]:g[1]],
                                      self.cur_flags[:, g[0]:g[1]], cache, self.prefix[:, g[0]:g[1]], 0.0,
                                      self.O[:, g[0]:g[1]], self.ws[ag.AG_CALL_PREFILL])
        ag.ag_prefill_attn(self.desc, self.Q, self.K, self.V, self.cur_flags, self.cache, self.prefix, 0.0, self.O,
                           self.ws[ag.AG_CALL_PREFILL])

    def decode(self, s):
        ag = self.ag
        q, kn, vn, fn = self.dq[s]
        # attention + conditional append of the step in one call
        ag.ag_decode_step(self.desc, q, kn, vn, fn, self.cache, 0.0, self.o, self.status, self.ws[ag.AG_CALL_DECODE])

    def step(self, ev=None, start=None):
        """One pass; ev (optional) = dict of lists of (start, end) CUDA events per call.  The calls of a
        pass run back to back on one stream, so the end mark of a call is the start mark of the next
        (start = the event the caller recorded just before the pass): one event per call."""
        chain = not self.first_gated                 # the guided stack runs its gates on a second stream
        prev = [start if chain else None]

        def timed(key, fn, *a):
            if ev is None:
                return fn(*a)
            s = prev[0]
            if s is None:
                s = torch.cuda.Event(enable_timing=True)
                s.record()
            fn(*a)
            e = torch.cuda.Event(enable_timing=True)
            e.record()
            ev[key].append((s, e))
            prev[0] = e if chain else None
        if self.first_gated:
            return self._step_guided_by_previous_layer(timed)
        for layer in range(self.layers):
            self.set_layer(layer)
            if self.has_gate:
                self.gamma = self.gammas[layer]
                timed("gate", self.gate)
            if self.project:
                timed("project", self.kv_project_cache)
                timed("prefill", self.prefill)
                if self.chain:
                    timed("out_project", self.out_project)
            elif self.has_prefill:
                timed("compact", self.compact)
                timed("prefill", self.prefill)
            else:
                self.cache.len.copy_(self.len0)      # every pass starts from the same cache
            timed("decode", self.decode_all)

    def _step_guided_by_previous_layer(self, timed):
        """Layer l runs under the flags of layer l-1's gate (Sec. 4.4, setting (4-1)); the gate passes
        run on a second stream, each beside the compaction, prefill and decode of its own layer."""
        if not hasattr(self, "schedule"):
            from paper_2410_12876_b200.schedule import PreviousLayerGate
            ones = torch.ones_like(self.flags)
            self.schedule = PreviousLayerGate(self.first_gated, [self.flags, torch.empty_like(self.flags)], ones, self.dev)

        def gate(layer, flags_out):
            # the module of layer `layer` on that layer's hidden states; its flags guide layer + 1
            keep = (self.layer, self.X, self.W)
            self.X, self.W = self.layer_in[layer][0], self.layer_in[layer][1]
            self.gamma = self.gammas[layer]
            timed("gate", self.gate, flags_out)
            self.layer, self.X, self.W = keep

        def attend(layer, flags):
            self.set_layer(layer)
            self.cur_flags = flags
            timed("compact", self.compact)
            timed("prefill", self.prefill)
            timed("decode", self.decode_all)
        self.schedule.run(self.layers, gate, attend)

    def decode_all(self):
        """All decode steps of a pass.  They are dozens of small launches, so they are
        replayed from one CUDA graph (captured once, on first use) unless disabled."""
        if not self.use_graph:
            for s in range(self.decode_steps):
                self.decode(s)
            return
        if self.layer not in self.graphs:
            len_before = self.cache.len.clone()
            for s in range(self.decode_steps):       # warm-up outside capture
                self.decode(s)
            self.cache.len.copy_(len_before)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for s in range(self.decode_steps):
                    self.decode(s)
            self.cache.len.copy_(len_before)         # capture does not run the kernels
            self.graphs[self.layer] = g
        self.graphs[self.layer].replay()

    def tokens_per_step(self):
        return self.shape.batch * ((self.shape.seq if self.has_prefill else 0) + self.decode_steps) * self.layers

    def launches_per_step(self):
        gates = (self.layers - self.first_gated) if self.has_gate else 0      # the last guided layer's gate has no consumer
        window = 2 if self.shape.recent_window > 1 else 0      # the ring fill after compaction, the band pass after prefill
        return gates * LAUNCHES["gate"] + self.layers * (
            (LAUNCHES["compact"] + LAUNCHES["prefill"] + window + (1 if self.chain else 0) if self.has_prefill else 0)
            + self.decode_steps * self.decode_launches())

    def decode_launches(self):
        slabs = self.shape.batch * self.shape.heads
        return 1 if slabs <= DECODE_CLUSTER_MAX_SLABS else LAUNCHES["decode"]

    def work_per_call(self):
        """Algorithmic work of one call, averaged over the layers of a pass (untimed extra pass):
        effective prefill FLOPs 4 D sum_j (1 + P[j]) (QK^T and PV over visible (query, key) pairs
        only), retained rows, and the bytes one decode step must move (every valid cache row once,
        K and V, plus q, k_new, v_new, o; lengths grow linearly over the decode steps)."""
        e = 2 if self.shape.dtype == "bf16" else 4
        D, slabs = self.shape.head_dim, self.shape.batch * self.shape.heads
        appended = float(np.mean([sum(q[3].to(torch.float64).sum().item() for q in dq) for dq in self.dqs]))
        f_eff, kept = [], []
        for layer in range(self.layers):
            self.set_layer(layer)
            if self.first_gated:
                if layer < self.first_gated:
                    self.cur_flags = torch.ones_like(self.flags)
                else:
                    self.gamma, self.cur_flags = self.gammas[layer - 1], self.flags
                    self.X, self.W = self.layer_in[layer - 1][0], self.layer_in[layer - 1][1]
                    self.gate()
                    self.set_layer(layer)
            elif self.has_gate:
                self.gamma = self.gammas[layer]
                self.gate()
            if self.has_prefill:
                if self.project:
                    self.kv_project_cache()
                else:
                    self.compact()
                if self.chain:
                    self.prefill()
                    self.out_project()
                P = self.prefix[:, :, :-1].to(torch.float64)
                f_eff.append(float(4.0 * D * (P.sum() + P.numel())))
                kept.append(float(self.prefix[:, :, -1].to(torch.float64).sum().item()))
            else:
                kept.append(float(self.len0.to(torch.float64).sum().item()))
        mean_kept = float(np.mean(kept))
        mean_len = mean_kept + appended * (self.decode_steps - 1) / (2.0 * self.decode_steps)
        return {"prefill_flops": float(np.mean(f_eff)) if f_eff else 0.0, "kept_rows": mean_kept,
                "decode_bytes": 2.0 * mean_len * D * e + 4.0 * slabs * D * e}

    def gate_flops(self):
        sh = self.shape
        GD = sh.gate_heads * sh.gate_head_dim
        rows = sh.batch * sh.seq
        return (2.0 * rows * sh.hidden * 3 * GD + 4.0 * sh.gate_head_dim * sh.gate_heads * sh.batch * sh.seq * (sh.seq + 1) / 2
                + 2.0 * rows * GD * sh.heads)


def max_over_ranks(values, dist, device):
    """Replicas share nothing on the data path; the only exchange of a multi-GPU run is this
    max-reduction of the per-rank timings (the job is as slow as its slowest rank)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_value(tokens_per_rank_step, world, steps, total_ms):
    """Whole-job tokens/s of `world` weak-scaled replicas timed as max over ranks."""
    return tokens_per_rank_step * world * steps / (total_ms * 1e-3)


def flush_l2(buf):
    buf.zero_()


CALLS = ("gate", "compact", "project", "prefill", "out_project", "decode")


def timed_passes(run, n_passes, l2buf):
    """n_passes passes of the whole path, each bracketed by CUDA events on the launching stream with
    the L2 flushed (outside the events) before it.  Returns (total ms, mean ms per call)."""
    ev = {k: [] for k in CALLS}
    pass_ev = []
    for _ in range(n_passes):
        flush_l2(l2buf)
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        run.step(ev, s)
        e.record()
        pass_ev.append((s, e))
    torch.cuda.synchronize()
    total_ms = sum(s.elapsed_time(e) for s, e in pass_ev)
    per_call_ms = {k: float(np.mean([s.elapsed_time(e) for s, e in v])) * len(v) / n_passes / run.layers
                   for k, v in ev.items() if v}
    return total_ms, per_call_ms


def rooflines_of(run, per_call_ms, peaks, workload):
    """Achieved rate of every call of a pass against its bound: algorithmic work of the call (from the
    flags / lengths the run produced) over its CUDA-event time (mean per layer)."""
    sh = run.shape
    e = 2 if sh.dtype == "bf16" else 4
    out = {}
    work = run.work_per_call()

    def entry(bound, kernel, amount, ms, key):
        unit, peak = ("TFLOP/s", peaks["bf16_tflops"]) if bound == "tensor" else ("GB/s", peaks["hbm_gbs"])
        rate = amount / (ms * 1e-3) / (1e12 if bound == "tensor" else 1e9)
        r = {"bound": bound, "kernel": kernel, "achieved": rate, "peak": peak, "unit": unit, "frac": rate / peak,
             "traffic": TRAFFIC.get((workload, key)), "peak_source": peaks["source"], "ms": ms, "workload": workload}
        r["algorithmic_flops" if bound == "tensor" else "algorithmic_bytes"] = amount
        return r

    dec_ms = per_call_ms["decode"] / run.decode_steps
    out["decode"] = entry("hbm", "ag_decode_step", work["decode_bytes"], dec_ms, "decode")
    if work["decode_bytes"] < L2_BYTES:
        # the cache of the step fits in L2 and has just been written by compaction and read by prefill:
        # the replayed decode steps stream it from L2, and a few microseconds per step do not depend on
        # its length at all.  The rate is reported, but it is no measurement of HBM bandwidth.
        out["decode"]["bound"] = "l2/latency"
        out["decode"]["note"] = ("cache of %.0f MB per step stays in L2 (126 MB): rate against the HBM copy peak for "
                                 "scale only; the HBM-bound decode figure is the decode_ragged workload's"
                                 % (work["decode_bytes"] / 1e6))
    if run.has_prefill:
        out["prefill"] = entry("tensor", "ag_prefill_attn", work["prefill_flops"], per_call_ms["prefill"], "prefill")
        if "compact" in per_call_ms:
            cb = 2.0 * (2.0 * work["kept_rows"] * sh.head_dim * e) + sh.batch * sh.heads * sh.seq * 9.0
            out["compact"] = entry("hbm", "ag_compact_kv", cb, per_call_ms["compact"], "compact")
        if "project" in per_call_ms:
            kf = 2.0 * sh.batch * sh.seq * sh.hidden * (2 * sh.kvh + sh.heads) * sh.head_dim
            out["project"] = entry("tensor", "ag_qkv_project_cache", kf, per_call_ms["project"], "project")
        if "out_project" in per_call_ms:
            of = 2.0 * sh.batch * sh.seq * sh.heads * sh.head_dim * sh.hidden
            out["out_project"] = entry("tensor", "ag_out_project", of, per_call_ms["out_project"], "out_project")
    if run.has_gate:
        out["gate"] = entry("tensor", "ag_gate_forward", run.gate_flops(), per_call_ms["gate"], "gate")
    return out


def timed_alone(fn, n, l2buf):
    """Mean CUDA-event time (ms) of n calls of fn, L2 flushed before each, after 3 warm-up calls."""
    evs = []
    for i in range(3 + n):
        flush_l2(l2buf)
        s_, e_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s_.record()
        fn()
        e_.record()
        if i >= 3:
            evs.append((s_, e_))
    torch.cuda.synchronize()
    return float(np.mean([a_.elapsed_time(b_) for a_, b_ in evs]))


def near_threshold_fractions(run):
    """Share of the (head, token) gate scores that lie within 1e-3 of the threshold, in the two units
    the tolerance can be read in: score units |s + gamma - logit(tau)| < 1e-3 (what the parity tests
    exclude from the bit-exact flag comparison) and probability units |Sigmoid(s + gamma) - tau| < 1e-3.
    Counted on the scores the last gate pass of the run produced."""
    tau = float(run.shape.tau)
    z = run.scores.double() + run.gamma.double().view(1, -1, 1)
    logit = float(np.log(tau / (1.0 - tau)))
    return {"score_units": float(((z - logit).abs() < 1e-3).double().mean().item()),
            "probability_units": float(((torch.sigmoid(z) - tau).abs() < 1e-3).double().mean().item())}


# The other full-size workloads, timed briefly after the headline workload in the default invocation:
# name -> (warm-up passes, timed passes).  One pass of decode_ragged is 256 graph-replayed decode steps
# over 2.4 GB of cache each; one of deep_layer is compaction + prefill of 16384 tokens + 128 decode
# steps; one of stack7b is 32 layers of gate + compaction + prefill + 256 decode steps at batch 8.
EXTRA_WORKLOADS = {"decode_ragged": (1, 3), "deep_layer": (3, 20), "stack7b": (1, 2)}


def measure_extra(name, dev, l2buf, peaks):
    warm, passes = EXTRA_WORKLOADS[name]
    run = LayerRun(name, 2000, dev)
    for _ in range(warm):
        run.step()
    torch.cuda.synchronize()
    total_ms, per_call_ms = timed_passes(run, passes, l2buf)
    assert int(run.status.item()) == 0, "device reported a cache overflow"
    roofs = rooflines_of(run, per_call_ms, peaks, name)
    info = {"ms_per_pass": total_ms / passes, "passes": passes, "tokens_per_s": run.tokens_per_step() * passes / (total_ms * 1e-3),
            "per_call_ms_per_layer": per_call_ms, "launches": run.launches_per_step() * passes,
            "mean_keep": float(run.flags.float().mean().item()) if run.has_prefill else None}
    del run
    torch.cuda.empty_cache()
    return roofs, info


def run_ours(args, rank, world, dev):
    torch.cuda.set_device(dev)
    run = LayerRun(args.workload, 2000 + 100 * rank, dev, args.recent_window)
    run.use_graph = not args.no_graph
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
    # A step is `passes` passes of the whole path over the batch, enough of them that the timed region
    # (steps x passes) lasts about MIN_TIMED_S: a few milliseconds of work would leave the clock
    # sampler, and whoever watches the GPU from outside, with a sample or two.
    t_probe, _ = timed_passes(run, 2, l2buf)
    est_pass_ms, = max_over_ranks([t_probe / 2], dist, dev)
    passes = args.passes if args.passes > 0 else max(1, int(np.ceil(MIN_TIMED_S * 1e3 / (args.steps * est_pass_ms))))
    sampler = ClockSampler(torch.cuda.current_device())
    if rank == 0:
        sampler.start()
    barrier()
    total_ms, per_call_ms = timed_passes(run, args.steps * passes, l2buf)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    assert int(run.status.item()) == 0, "device reported a cache overflow"
    timeouts = run.ag.ag_device_wait_timeouts()
    assert timeouts == 0, f"{timeouts} bounded device waits expired"

    # end to end: pinned host inputs in, results out, through the same calls
    sh = run.shape
    stack = run.layers > 1 and run.has_gate
    if run.chain:
        dev_in = [run.X0] + run.dq_flat
    elif stack:
        dev_in = [t for (X, W, Q, K, V), flat in zip(run.layer_in, run.dq_flat) for t in [X, Q, K, V, flat]]
    elif run.project:
        dev_in = [run.X]                                     # Q, K and V are made on the device
    elif run.has_gate:
        dev_in = [run.X, run.Q, run.K, run.V]
    elif run.has_prefill:
        dev_in = [run.Q, run.K, run.V, run.flags]
    else:
        dev_in = []
    if not stack and not run.chain:
        dev_in += run.dq_flat
    dev_out = ([run.O, run.flags] if run.has_prefill else []) + [run.o]
    host_in = [t.detach().cpu().pin_memory() for t in dev_in]
    host_out = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in dev_out]
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = sum(t.numel() * t.element_size() for t in host_out)
    e2e_steps = max(1, min(args.steps, 10 if not stack else 1))
    # One layer with a gate: the copies run on their own streams, each call waits only for the inputs
    # it reads (X -> gate; a head group's K, V, Q -> its compaction and prefill; the decode tokens ->
    # decode), and the flags and each group's O go back to the host while later groups come in.
    # Other workloads: copy in, step, copy out, in order.
    overlap = run.has_gate and run.has_prefill and run.layers == 1
    if run.chain:
        dev_out.append(run.Xbuf[(run.layers - 1) % 2])      # the stack's final hidden states
        host_out.append(torch.empty(run.X0.shape, dtype=run.X0.dtype).pin_memory())
        d2h = sum(t.numel() * t.element_size() for t in host_out)
    if overlap and run.project:
        main = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    elif overlap:
        main = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        n_dq = len(dev_in) - 4
        # head groups of the pipelined copies: the heads of a sequence are contiguous only when batch = 1
        hg = sh.heads // 4                       # heads per group; every group's slices must start on 16-byte boundaries
        n_groups = 4 if (sh.batch == 1 and sh.kv_heads == 0 and sh.heads % 4 == 0 and sh.recent_window <= 1
                         and (hg * (sh.seq + 1) * 4) % 16 == 0 and (hg * sh.seq) % 16 == 0) else 1
        groups = [(g * sh.heads // n_groups, (g + 1) * sh.heads // n_groups) for g in range(n_groups)]
    O_step = run.O.clone() if run.has_prefill else None      # what the device-resident steps produced
    barrier()
    t_e2e = 0.0
    for _ in range(e2e_steps):
        flush_l2(l2buf)
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        if overlap and run.project:
            # X -> gate, the projection and prefill; the decode tokens -> decode
            s_in.wait_stream(main)
            s_out.wait_stream(main)
            ready = []
            with torch.cuda.stream(s_in):
                for group in ([0], list(range(1, len(dev_in)))):
                    for i in group:
                        dev_in[i].copy_(host_in[i], non_blocking=True)
                    ev_ = torch.cuda.Event()
                    ev_.record(s_in)
                    ready.append(ev_)
            run.gamma = run.gammas[0]
            main.wait_event(ready[0]); run.gate()
            flags_done = torch.cuda.Event(); flags_done.record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(flags_done)
                host_out[1].copy_(run.flags, non_blocking=True)
            run.kv_project_cache()
            run.prefill()
            if run.chain:
                run.set_layer(0)
                run.out_project()
            o_done = torch.cuda.Event(); o_done.record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(o_done)
                host_out[0].copy_(run.O, non_blocking=True)
            main.wait_event(ready[1]); run.decode_all()
            host_out[2].copy_(run.o, non_blocking=True)
            if run.chain:
                host_out[3].copy_(run.Xbuf[0], non_blocking=True)     # the layer's output hidden states
            main.wait_stream(s_out)
        elif overlap:
            s_in.wait_stream(main)
            s_out.wait_stream(main)
            ready = []                                       # events: X, decode inputs (small), one per head group (its K, V, Q)
            with torch.cuda.stream(s_in):
                for group in ([(0, None)], [(i, None) for i in range(4, 4 + n_dq)],
                              *[[(2, g), (3, g), (1, g)] for g in groups]):
                    for i, g in group:
                        if g is None:
                            dev_in[i].copy_(host_in[i], non_blocking=True)
                        else:
                            dev_in[i][:, g[0]:g[1]].copy_(host_in[i][:, g[0]:g[1]], non_blocking=True)
                    ev_ = torch.cuda.Event()
                    ev_.record(s_in)
                    ready.append(ev_)
            run.gamma = run.gammas[0]
            main.wait_event(ready[0]); run.gate()
            flags_done = torch.cuda.Event(); flags_done.record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(flags_done)
                host_out[1].copy_(run.flags, non_blocking=True)
            for gi, g in enumerate(groups):
                # compaction and prefill attention of a head group as soon as its K, V, Q are in; its O
                # goes back while the next groups are still coming in (the link carries both directions)
                main.wait_event(ready[2 + gi])
                gg = g if n_groups > 1 else None
                run.compact(gg); run.prefill(gg)
                o_done = torch.cuda.Event(); o_done.record(main)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(o_done)
                    host_out[0][:, g[0]:g[1]].copy_(run.O[:, g[0]:g[1]], non_blocking=True)
            main.wait_event(ready[1]); run.decode_all()
            host_out[2].copy_(run.o, non_blocking=True)
            main.wait_stream(s_out)
        else:
            for d, hsrc in zip(dev_in, host_in):
                d.copy_(hsrc, non_blocking=True)
            run.step()
            for hdst, d in zip(host_out, dev_out):
                hdst.copy_(d, non_blocking=True)
        e.record()
        e.synchronize()
        t_e2e += s.elapsed_time(e)
    barrier()
    if O_step is not None:
        assert torch.equal(host_out[0], O_step.cpu()), "the end-to-end pass and the device-resident step disagree"

    total_ms, t_e2e = max_over_ranks([total_ms, t_e2e], dist, dev)
    if rank != 0:
        return None
    tokens = run.tokens_per_step() * world
    peaks = _peaks()
    near = near_threshold_fractions(run) if run.has_gate else None     # on the scores of the step's own gate pass
    rooflines = rooflines_of(run, per_call_ms, peaks, args.workload)
    if run.has_gate and run.layers == 1:
        # the local gate variant, timed apart from the step (L2 flushed before each call)
        lin_ms = timed_alone(run.gate_linear, min(args.steps, 20), l2buf)
        e = 2 if sh.dtype == "bf16" else 4
        lb = float(sh.batch * sh.seq * sh.hidden * e + sh.hidden * sh.heads * e + sh.batch * sh.heads * sh.seq * 5)
        gbs = lb / (lin_ms * 1e-3) / 1e9
        rooflines["gate_linear"] = {"bound": "hbm", "kernel": "ag_gate_linear_forward (not part of the step)",
                                    "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                    "frac": gbs / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
                                    "algorithmic_bytes": lb, "ms": lin_ms, "workload": args.workload}
        if (sh.dtype == "bf16" and sh.head_dim == 128 and sh.seq % 128 == 0 and sh.recent_window <= 1
                and not run.project):
            # the fused key/value projection, timed apart from the step like the local gate
            kv_ms = timed_alone(run.kv_project_cache, min(args.steps, 20), l2buf)
            kf = 2.0 * sh.batch * sh.seq * sh.hidden * 2 * sh.kvh * sh.head_dim
            tf = kf / (kv_ms * 1e-3) / 1e12
            rooflines["kv_project_cache"] = {"bound": "tensor",
                                             "kernel": "ag_kv_project_cache (not part of the step)",
                                             "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                             "frac": tf / peaks["bf16_tflops"],
                                             "traffic": TRAFFIC.get((args.workload, "kv_project_cache")),
                                             "peak_source": peaks["source"], "algorithmic_flops": kf, "ms": kv_ms,
                                             "workload": args.workload}
    head = "prefill" if run.has_prefill else "decode"
    n_timed = args.steps * passes
    ms_pass = total_ms / n_timed
    out = {
        "metric": METRIC, "value": aggregate_value(run.tokens_per_step(), world, n_timed, total_ms), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if sh.dtype == "bf16" else "f32", "data": "synthetic",
        "config": config_of(args.workload, sh, run.decode_steps, run.desc_text),
        "timing": {"passes_per_step": passes, "ms_per_pass": ms_pass,
                   "step": f"{passes} passes of the whole path over the batch, L2 flushed before each pass (outside its events)",
                   "recent_window": max(1, sh.recent_window),
                   "mean_keep": float(run.flags.float().mean().item()) if run.has_prefill else None,
                   "near_threshold": near,
                   "replicas": world,
                   "decode_launch": "one CUDA graph per pass" if run.use_graph else "individual launches"},
        "clocks": clocks,
        "e2e": {"value": tokens * e2e_steps / (t_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps, "passes_per_step": 1},
        "gpu_launches": run.launches_per_step() * n_timed,
        "roofline": rooflines[head],
        "rooflines": rooflines,
        "per_call_ms": per_call_ms,
        "dominant_call": max(per_call_ms, key=per_call_ms.get),
        "decode_tokens_per_s": sh.batch * run.decode_steps / (per_call_ms["decode"] * 1e-3),
    }
    if run.has_prefill:
        pre_ms = sum(per_call_ms.get(k, 0.0) for k in ("gate", "compact", "project", "prefill", "out_project"))
        out["prefill_tokens_per_s"] = sh.batch * sh.seq / (pre_ms * 1e-3)
    if args.workload == "prefill7b" and world == 1 and not args.no_extra and args.recent_window <= 1:
        # the other full-size workloads, briefly: their rooflines ride in the same line
        out["workloads"] = {}
        del host_in, host_out
        for name in EXTRA_WORKLOADS:
            roofs, info = measure_extra(name, dev, l2buf, peaks)
            out["workloads"][name] = info
            for k, r in roofs.items():
                rooflines[f"{name}.{k}"] = r
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
    if name == "prefill7b_proj":                 # the layer owns its projection (Eq. 2)
        Qd = orc.project_q(Xd, f64(Wsub["Wq"]), hs)
        Kd, Vd = orc.project_kv(Xd, f64(Wsub["Wk"]), f64(Wsub["Wv"]), hs)
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
    return {"value": tokens / est, "unit": UNIT, "cores": int(cores), "kind": "oracle", "sample_s": t_gate + t_heads + t_dec,
            "sample": f"full gate + {hs} of {shape.heads} heads of compaction/prefill + {ds} of {dsteps} decode steps, "
                      f"scaled to the whole step (gate {t_gate:.2f}s, heads {t_heads:.2f}s, decode {t_dec:.3f}s)",
            "est_step_s": est}


def run_reference(args, rank, world):
    if rank != 0:
        return None
    shape, dsteps, text = WORKLOADS[args.workload]
    # each step is one bounded oracle sample (seconds of CPU work); the number of samples is capped so
    # that the whole run stays within a few minutes whatever --steps asks for
    vals, walls, t_start, budget_s = [], [], time.perf_counter(), 150.0
    for k in range(args.warmup + args.steps):
        t_k = time.perf_counter()
        r = oracle_sample(args.workload, 2000, n_heads_sample=1, decode_steps=1)
        if k >= args.warmup:
            vals.append(r)
            walls.append(r["sample_s"])
        per = (time.perf_counter() - t_start) / (k + 1)
        if vals and time.perf_counter() - t_start + per > budget_s:
            break
    est = float(np.mean([r["est_step_s"] for r in vals]))
    tokens = shape.batch * (shape.seq + dsteps)
    v = tokens / est
    base = dict(vals[-1])
    base["value"] = v
    base.pop("est_step_s", None)
    base.pop("sample_s", None)
    # ms_per_step is the measured time of one step of THIS arm (one bounded sample); `value` is the
    # whole-layer rate that sample extrapolates to (est_layer_ms)
    return {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": world, "steps": len(vals),
            "steps_requested": args.steps,
            "warmup": args.warmup, "ms_per_step": float(np.mean(walls)) * 1e3, "est_layer_ms": est * 1e3,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(args.workload, shape, dsteps, text),
            "cpu_baseline": base,
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def config_of(workload, sh, decode_steps, text):
    """The keys of `config` both arms print alike."""
    return {"workload": workload, "description": text, "batch": sh.batch, "seq": sh.seq, "hidden": sh.hidden,
            "heads": sh.heads, "head_dim": sh.head_dim, "gate_heads": sh.gate_heads, "gate_head_dim": sh.gate_head_dim,
            "decode_steps_per_pass": decode_steps,
            "l2": "GPU arm: flushed before every pass (256 MiB write, outside the pass's events); the CPU arm has no GPU cache"}


def replica_command(n_gpus, argv, port):
    """The command line that runs this script as n_gpus replicas, one process per GPU, on this node."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def spawn_replicas(n_gpus, argv):
    port = 29500 + os.getpid() % 2000
    return subprocess.call(replica_command(n_gpus, argv, port))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="prefill7b", choices=list(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--recent-window", type=int, default=0,
                    help="recent tokens always visible, the current one included (0 or 1: the method as published)")
    ap.add_argument("--no-graph", action="store_true", help="launch the decode steps one by one instead of replaying a CUDA graph")
    ap.add_argument("--passes", type=int, default=0,
                    help="passes of the whole path per step (0: as many as make the timed region last about 0.6 s)")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the brief measurements of the other full-size workloads after the headline one")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand with --gpus N: become N replicas, one process per GPU
        raise SystemExit(spawn_replicas(args.gpus, sys.argv[1:]))
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
        if not args.no_cpu_baseline and world == 1 and args.workload in ("prefill7b", "prefill7b_proj", "tiny"):
            cb = oracle_sample(args.workload, 2000, n_heads_sample=WORKLOADS[args.workload][0].heads, decode_steps=16)
            cb.pop("est_step_s", None)
            cb.pop("sample_s", None)
            out["cpu_baseline"] = cb
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
