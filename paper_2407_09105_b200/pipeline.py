"""Host-to-host runs of the path, one packed stream (pack / mini-batch) at a time.

The packs of a step are independent, so the copy of pack i+1 to the device, the kernels of pack i
and the copy of pack i-1's results back to the host can run at the same time on three CUDA
streams (PCIe is full duplex).  Plumbing only: every computation happens in the library calls
the caller passes in as ``compute``."""
from __future__ import annotations

from typing import Callable, List, Sequence

import torch


class HostPipeline:
    """``host_in[i]`` / ``dev_in[i]`` and ``dev_out[i]`` / ``host_out[i]`` are matching lists of
    tensors of pack i (host tensors pinned); ``compute(i, stream)`` enqueues pack i's kernels."""

    def __init__(self, host_in: Sequence[Sequence[torch.Tensor]], dev_in, dev_out, host_out,
                 compute: Callable[[int, torch.cuda.Stream], None]):
        self.host_in, self.dev_in, self.dev_out, self.host_out = host_in, dev_in, dev_out, host_out
        self.compute = compute
        self.n = len(host_in)
        self.s_in, self.s_c, self.s_out = (torch.cuda.Stream() for _ in range(3))
        mk = lambda: [torch.cuda.Event() for _ in range(self.n)]
        self.ev_in, self.ev_c, self.ev_out = mk(), mk(), mk()
        self.primed = False

    def step(self, after: torch.cuda.Stream) -> None:
        """One pass over all packs; starts after the work already queued on ``after`` and is
        joined back into it (so events recorded on ``after`` bracket the whole pass)."""
        start = torch.cuda.Event()
        start.record(after)
        for s in (self.s_in, self.s_c, self.s_out):
            s.wait_event(start)
        for i in range(self.n):
            if self.primed:                       # the device buffers of pack i are reused
                self.s_in.wait_event(self.ev_c[i])      # inputs: last pass's kernels are done
                self.s_c.wait_event(self.ev_out[i])     # outputs: last pass's copy-out is done
            with torch.cuda.stream(self.s_in):
                for h, d in zip(self.host_in[i], self.dev_in[i]):
                    d.copy_(h, non_blocking=True)
                self.ev_in[i].record(self.s_in)
            self.s_c.wait_event(self.ev_in[i])
            self.compute(i, self.s_c)
            self.ev_c[i].record(self.s_c)
            self.s_out.wait_event(self.ev_c[i])
            with torch.cuda.stream(self.s_out):
                for d, h in zip(self.dev_out[i], self.host_out[i]):
                    h.copy_(d, non_blocking=True)
                self.ev_out[i].record(self.s_out)
        self.primed = True
        for s in (self.s_in, self.s_c, self.s_out):
            done = torch.cuda.Event()
            done.record(s)
            after.wait_event(done)
