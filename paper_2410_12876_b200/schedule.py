"""Stream schedule of a stack of AG-gated layers whose eviction is guided by the previous layer
(Sec. 4.4, ablation settings (4-1) and (4-2)).

In the default method layer l's gate pass must finish before layer l's compaction and attention
can start.  When layer l instead evicts by the flags that layer l-1's AG module computed from layer
l-1's hidden states, the gate pass of a layer has no consumer inside that layer: it runs on a second
stream beside the layer's own compaction, prefill attention and decode steps, and only the NEXT
layer waits for it.  This module holds that ordering and nothing else: the work itself is the
caller's two callables, which enqueue the library's calls on the current stream.

    gate(l, flags_out)   enqueue layer l's gate pass (its AG module, its hidden states) -> flags_out
    attend(l, flags)     enqueue layer l's compaction, prefill attention and decode steps under flags
"""
import torch


class PreviousLayerGate:
    """first_gated: the first layer that evicts (1 in setting (4-1), 2 in (4-2)); the layers before
    it run under `ones` (all retained).  flag_bufs: two flag tensors used in turn, so that a gate
    pass may write one while the attention of the layer beside it reads the other."""

    def __init__(self, first_gated, flag_bufs, ones, device=None):
        if first_gated < 1:
            raise ValueError("the first layer has no previous layer to take flags from")
        if len(flag_bufs) != 2:
            raise ValueError("two flag buffers are needed")
        self.first_gated, self.flag_bufs, self.ones = first_gated, flag_bufs, ones
        self.gate_stream = torch.cuda.Stream(device)
        self.flags_ready = [torch.cuda.Event(), torch.cuda.Event()]
        self.flags_read = [torch.cuda.Event(), torch.cuda.Event()]

    def run(self, n_layers, gate, attend):
        """Enqueues the whole stack; returns with the current stream waiting on all of it."""
        main = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(main)
        self.gate_stream.wait_event(start)            # inputs written on the caller's stream are visible
        written = [False, False]                      # buffer holds flags some layer still has to read
        for l in range(n_layers):
            nxt = l + 1
            if self.first_gated <= nxt < n_layers:
                b = nxt % 2
                with torch.cuda.stream(self.gate_stream):
                    if written[b]:
                        self.gate_stream.wait_event(self.flags_read[b])   # layer l-1 is done reading it
                    gate(l, self.flag_bufs[b])
                    self.flags_ready[b].record(self.gate_stream)
                written[b] = True
            if l >= self.first_gated:
                b = l % 2
                main.wait_event(self.flags_ready[b])
                attend(l, self.flag_bufs[b])
                self.flags_read[b].record(main)
            else:
                attend(l, self.ones)
        done = torch.cuda.Event()
        done.record(self.gate_stream)
        main.wait_event(done)


class ChainedLayerBuffers:
    """Device buffers one layer of a chained stack works in (shared by all layers of the stack: a
    layer's Q, K, V, O, flags and cache are dead once its output has been projected, except for the
    cache when decode steps follow)."""

    def __init__(self, ag, shape, extra_rows=0, device="cuda"):
        import torch as _t
        B, h, hk, n, D = shape.batch, shape.heads, shape.kvh, shape.seq, shape.head_dim
        dt = shape.torch_dtype
        self.desc = ag.make_desc(shape)
        self.scores = _t.empty(B, hk, n, dtype=_t.float32, device=device)
        self.flags = _t.empty(B, hk, n, dtype=_t.uint8, device=device)
        self.prefix = _t.empty(B, hk, n + 1, dtype=_t.int32, device=device)
        self.Q = _t.empty(B, h, n, D, dtype=dt, device=device)
        self.K = _t.empty(B, hk, n, D, dtype=dt, device=device)
        self.V = _t.empty(B, hk, n, D, dtype=dt, device=device)
        self.O = _t.empty(B, h, n, D, dtype=dt, device=device)
        self.cache = ag.RaggedCache.allocate(shape, [n + extra_rows] * (B * hk), device)
        self.status = _t.zeros(1, dtype=_t.int32, device=device)
        self.ws_gate = ag.workspace(self.desc, ag.AG_CALL_GATE, device)
        self.ws_prefill = ag.workspace(self.desc, ag.AG_CALL_PREFILL, device)


def chained_layer(ag, buf, X, W, gamma, X_next, after=None):
    """Enqueues one layer of a chained stack of attention layers on the current stream: the gate on
    the layer's hidden states X (Sec. 3.3), the Q, K, V projection of Eq. 2 that writes the retained
    rows into the cache, prefill attention under the eviction mask (Eq. 5), and the output
    projection of Eq. 1 with the skip connection, X_next = X + [H_1 .. H_h] W^O: the next layer's
    hidden states.  Nothing normalises and no feed-forward block sits between two layers.
    W: dict with Wq, Wk, Wv, Wo and the gate's Wq_g, Wk_g, Wv_g, Wo_g.  after (optional) is called
    between the layer's calls with the name of the call just enqueued (for timing marks)."""
    mark = after if after is not None else (lambda name: None)
    ag.ag_gate_forward(buf.desc, X, W["Wq_g"], W["Wk_g"], W["Wv_g"], W["Wo_g"], gamma, buf.scores, buf.flags,
                       buf.ws_gate)
    mark("gate")
    ag.ag_qkv_project_cache(buf.desc, X, W["Wq"], W["Wk"], W["Wv"], buf.flags, buf.cache, buf.prefix, None, buf.Q,
                            buf.K, buf.V, buf.status)
    mark("project")
    ag.ag_prefill_attn(buf.desc, buf.Q, buf.K, buf.V, buf.flags, buf.cache, buf.prefix, 0.0, buf.O, buf.ws_prefill)
    mark("prefill")
    ag.ag_out_project(buf.desc, buf.O, W["Wo"], X, X_next)
    mark("out_project")
