"""Several compressors (one per shape class of a model's matrix stack) stepped concurrently.

Each handle gets a CUDA stream of its own: the small finishing kernels of one shape class (Cholesky,
Q_i = W_i T', ...) and the ragged last wave of its big kernel overlap the streaming kernel of the next
class instead of leaving SMs idle.  The handles share nothing (own workspace, own tensor maps), so no
ordering is needed between them inside a step; a step starts after everything queued before it on the
caller's stream and is complete, for the caller's stream, when `step` returns.
"""
from __future__ import annotations


class StreamedStack:
    def __init__(self, handles, device=None):
        import torch

        self.torch = torch
        self.handles = list(handles)
        self.device = torch.device(device if device is not None else self.handles[0].device)
        self.streams = [torch.cuda.Stream(self.device) for _ in self.handles]
        self._fork = torch.cuda.Event()
        self._join = [torch.cuda.Event() for _ in self.handles]

    def step(self, G_list, force_refresh=False):
        """One compression step of every handle on its own stream; G_list[i] belongs to handles[i]."""
        torch = self.torch
        main = torch.cuda.current_stream(self.device)
        self._fork.record(main)
        for h, g, s, e in zip(self.handles, G_list, self.streams, self._join):
            s.wait_event(self._fork)
            h.step(g, stream=s, force_refresh=force_refresh)
            e.record(s)
        for e in self._join:
            main.wait_event(e)

    def step_host(self, G_host, G_stage, P_hat_host, Q_host):
        """The host-buffer entry point of every handle on its own stream (copies of one class overlap
        the kernels of another)."""
        torch = self.torch
        main = torch.cuda.current_stream(self.device)
        self._fork.record(main)
        for h, gh, st, ph, qh, s, e in zip(self.handles, G_host, G_stage, P_hat_host, Q_host, self.streams, self._join):
            s.wait_event(self._fork)
            h.step_host(gh, st, ph, qh, stream=s)
            e.record(s)
        for e in self._join:
            main.wait_event(e)
