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
