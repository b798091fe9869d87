"""Data parallelism proper: every process holds some of the nodes, the means of Algorithm 2 cross the processes.

Algorithm 2 averages three arrays over the nodes: P, Q and, when t mod tau = 0, the error-compensated gradient itself.
Each handle forms the mean over the nodes it holds (`psgd_exchange_begin / _orth / _end`); this module lays the arrays
of all handles of a model side by side in ONE flat buffer per exchange and averages each buffer over the processes with
a single all-reduce (NCCL over NVLink on GPUs).  Every process then factorises the same averaged array with the same
deterministic kernels, so P~ and Q agree bit for bit without being broadcast.

Nothing here computes anything of the method: the handles do (CUDA), `torch.distributed` moves the bytes.  The class
takes any objects with the four `exchange_*` methods, which is how the CPU tests drive it over gloo.
"""
from __future__ import annotations

ALIGN_FLOATS = 64    # every slot starts on a 256-byte boundary (the library asks for 16)


def slot_offsets(sizes, align=ALIGN_FLOATS):
    """Start of each slot in a flat buffer, every start a multiple of `align` elements; returns (offsets, total)."""
    offsets, pos = [], 0
    for s in sizes:
        if s < 0:
            raise ValueError("negative slot size")
        offsets.append(pos)
        pos += -(-int(s) // align) * align
    return offsets, pos


class ExchangedStack:
    """Handles of one model stepped together, their node means averaged over the processes of `group`.

    All processes must build the same handles in the same order (same shapes, seeds, options and nodes per handle)."""

    def __init__(self, handles, group=None, device=None, dist=None, dtype=None):
        import torch

        self.torch = torch
        self.handles = list(handles)
        if dist is None:
            import torch.distributed as dist
        self.dist = dist
        self.group = group
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.device = torch.device(device if device is not None else self.handles[0].device)
        self.dtype = dtype if dtype is not None else torch.float32     # the library's arrays are float32
        self._buf = {}          # (which exchange, floats) -> flat buffer; at most two sizes of the first (P or Delta) and one of the second
        self.exchanges = 0      # all-reduces issued so far (two per step)
        self.bytes_exchanged = 0

    def _flat(self, which, floats):
        key = (which, floats)
        if key not in self._buf:
            self._buf[key] = self.torch.zeros((max(floats, 1),), dtype=self.dtype, device=self.device)   # gaps between slots stay zero
        return self._buf[key]

    def _mean_over_processes(self, buf):
        self.exchanges += 1
        self.bytes_exchanged += buf.numel() * buf.element_size()
        if self.world == 1:
            return
        dist = self.dist
        backend = dist.get_backend(self.group)
        if backend == "nccl":
            dist.all_reduce(buf, op=dist.ReduceOp.AVG, group=self.group)
        else:                     # gloo has no mean: sum, then scale
            dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=self.group)
            buf.mul_(1.0 / self.world)

    def step(self, G_list, force_refresh=False):
        """One iteration of every handle; G_list[i] holds the gradients of the nodes of handles[i] on this process."""
        hs = self.handles
        plans = [h.exchange_plan(force_refresh) for h in hs]
        off1, tot1 = slot_offsets([p[1] for p in plans])
        off2, tot2 = slot_offsets([p[2] for p in plans])
        first, second = self._flat(0, tot1), self._flat(1, tot2)
        s1 = [first[o:o + p[1]] for o, p in zip(off1, plans)]
        s2 = [second[o:o + p[2]] for o, p in zip(off2, plans)]
        for h, g, a in zip(hs, G_list, s1):
            h.exchange_begin(g, a, force_refresh=force_refresh)
        self._mean_over_processes(first)
        for h, a, b in zip(hs, s1, s2):
            h.exchange_orth(a, b)
        self._mean_over_processes(second)
        for h, b in zip(hs, s2):
            h.exchange_end(b)
        return [p[0] for p in plans]
