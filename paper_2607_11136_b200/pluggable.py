"""Static-memory runtime for ordinary PyTorch code: PyTorch's allocator is replaced by the
library's plug-in (CUDAPluggableAllocator), one step is recorded, laid out by Algorithm 1
(xema_plan_arena) and then replayed with every allocation answered from the planned arena.

    from paper_2607_11136_b200 import pluggable
    pluggable.install()                   # before the process makes its first CUDA allocation
    rt = pluggable.StaticRuntime()
    rt.warm_up(step)                      # one-time workspaces are allocated outside the plan
    rt.record(step)                       # logs sizes and lifetimes of one step
    rt.plan()                             # offsets + one arena of exactly the planned peak
    out = rt.replay(step)                 # allocation = table lookup

`step` must release everything it allocates before it returns (copy results out), and must issue
the same allocation sequence every time (template-static execution).
"""
from __future__ import annotations

import torch

from . import binding as xb

_installed = False


def install():
    """Routes every CUDA allocation of this process through the library (pass-through mode).
    PyTorch accepts this only before its own allocator has been used."""
    global _installed
    if _installed:
        return
    alloc = torch.cuda.memory.CUDAPluggableAllocator(xb.LIB_PATH, "xema_pluggable_malloc", "xema_pluggable_free")
    torch.cuda.memory.change_current_allocator(alloc)
    xb.lib()
    _installed = True


class StaticRuntime:
    def __init__(self, device="cuda:0"):
        if not _installed:
            raise RuntimeError("call pluggable.install() first")
        self.device = torch.device(device)
        self.requests, self.offsets, self.peak_bytes, self.max_live_bytes = None, None, None, None
        self.arena = None

    def warm_up(self, step, times: int = 2):
        xb.xema_pluggable_mode(xb.ALLOC_PASSTHROUGH)
        out = None
        for _ in range(times):
            out = step()
        torch.cuda.synchronize(self.device)
        return out

    def record(self, step):
        torch.cuda.synchronize(self.device)
        xb.xema_pluggable_mode(xb.ALLOC_RECORD)
        try:
            out = step()
            torch.cuda.synchronize(self.device)
        finally:
            xb.xema_pluggable_mode(xb.ALLOC_PASSTHROUGH)
        self.requests, self.n_events = xb.xema_pluggable_recorded()
        return out

    def plan(self):
        """Algorithm 1 over the recorded lifetimes; allocates the arena (pass-through mode)."""
        if not self.requests:
            raise RuntimeError("nothing recorded")
        self.offsets, self.peak_bytes, self.max_live_bytes = xb.xema_plan_arena(self.requests)
        # PyTorch keys its own bookkeeping by address, so no planned tensor may start at the
        # address of the tensor that holds the arena: the plan starts 256 bytes in
        self.arena = torch.empty(self.peak_bytes + 256, dtype=torch.uint8, device=self.device)
        self.base = self.arena.data_ptr() + 256
        xb.xema_pluggable_set_plan(self.base, self.peak_bytes, self.offsets)
        return self.peak_bytes

    def replay(self, step):
        xb.xema_pluggable_mode(xb.ALLOC_REPLAY)
        try:
            xb.xema_pluggable_step_begin()
            out = step()
            torch.cuda.synchronize(self.device)
        finally:
            xb.xema_pluggable_mode(xb.ALLOC_PASSTHROUGH)
        return out

    def contains(self, t: torch.Tensor) -> bool:
        return self.base <= t.data_ptr() and t.data_ptr() + t.numel() * t.element_size() <= self.base + self.peak_bytes
