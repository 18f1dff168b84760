"""Device-side plumbing around the C ABI: torch owns the arena, the weights and the RoPE
table; the library gets raw pointers.  No arithmetic of the block happens here."""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch

from . import binding as xb


def _dev_u16(bits: np.ndarray, device) -> torch.Tensor:
    """uint16 bf16 bit patterns -> device tensor of the same bits (viewed as int16)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device, non_blocking=False)


class BlockSession:
    """One bound plan: arena + weights + RoPE table on `device`, ready for forward calls.

    template: object with the xema_config field names (e.g. xema_inputs.Template).
    weights:  list (one per block) of dicts name -> uint16 bf16 bit patterns (numpy), or of
              dicts name -> torch tensors already on the device.
    Either `chunks` (one count, or a triple of per-phase counts) or `budget_bytes` selects
    the chunking; with a budget, `per_phase` picks between the per-phase search (chunk only
    the phases whose trace exceeds the budget) and one count for the whole block.
    """

    def __init__(self, template, weights: Sequence[dict], chunks=None,
                 budget_bytes: Optional[int] = None, max_chunks: int = 64, device="cuda:0",
                 arena: Optional[torch.Tensor] = None, per_phase: bool = True):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU fallback)")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.template = template
        self.cfg = xb.make_config(template)
        if chunks is None:
            if budget_bytes is None:
                raise ValueError("give chunks or budget_bytes")
            search = xb.xema_phase_chunks_for_budget if per_phase else xb.xema_chunks_for_budget
            chunks, _ = search(self.cfg, int(budget_bytes), max_chunks)
            if chunks is None:
                raise xb.XemaError(xb.XEMA_EBUDGET, search.__name__)
        self.budget_bytes = budget_bytes
        self.plan = xb.Plan(self.cfg, chunks)
        self.chunks = chunks
        self.phase_chunks = self.plan.phase_chunks
        if budget_bytes is not None and self.plan.peak_bytes > budget_bytes:
            raise xb.XemaError(xb.XEMA_EBUDGET, "plan peak exceeds the budget")
        if len(weights) != template.n_blocks:
            raise ValueError("need one weight dict per block")
        self.weights = []
        ptrs = []
        for w in weights:
            dev = {k: (v if isinstance(v, torch.Tensor) else _dev_u16(v, self.device)) for k, v in w.items()}
            self.weights.append(dev)
            ptrs.append({k: v.data_ptr() for k, v in dev.items()})
        self.rope = torch.from_numpy(xb.xema_rope_table(self.cfg)).to(self.device)
        # the arena is exactly the planned peak: the library cannot touch anything else
        if arena is None:
            arena = torch.empty(self.plan.peak_bytes, dtype=torch.uint8, device=self.device)
        if arena.numel() < self.plan.peak_bytes:
            raise xb.XemaError(xb.XEMA_ENOSPC, "arena")
        self.arena = arena
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.plan.bind(self.arena.data_ptr(), self.arena.numel(), ptrs, self.rope.data_ptr(), self.status.data_ptr())
        self.seq = template.s_text + template.grid_t * template.grid_h * template.grid_w

    # ---- views into the arena ---------------------------------------------------------
    def view(self, name: str, dtype=torch.int16, shape=None) -> torch.Tensor:
        off, nbytes = self.plan.tensor(name)
        v = self.arena[off:off + nbytes].view(dtype)
        if shape is not None:
            n = int(np.prod(shape))
            v = v[:n].view(*shape)
        return v

    def hid_in(self) -> torch.Tensor:
        t = self.template
        return self.view("hid0", torch.int16, (t.batch, self.seq, t.hidden))

    def temb(self) -> torch.Tensor:
        t = self.template
        return self.view("temb", torch.int16, (t.batch, t.temb_dim))

    def hid_out(self) -> torch.Tensor:
        t = self.template
        return self.view("hid%d" % t.n_blocks, torch.int16, (t.batch, self.seq, t.hidden))

    # ---- data movement ------------------------------------------------------------------
    def set_inputs(self, x_bits, temb_bits, non_blocking: bool = False):
        """x_bits / temb_bits: uint16 numpy arrays or int16 torch tensors (host or device)."""
        for dst, src in ((self.hid_in(), x_bits), (self.temb(), temb_bits)):
            if isinstance(src, np.ndarray):
                src = torch.from_numpy(np.ascontiguousarray(src).view(np.int16))
            dst.copy_(src.view(dst.shape), non_blocking=non_blocking)

    def forward(self, stream: Optional[torch.cuda.Stream] = None):
        s = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        if self.template.n_blocks == 1:
            self.plan.block_forward(s)
        else:
            self.plan.step_forward(s)

    def output_bits(self) -> np.ndarray:
        """Synchronises and returns the output hidden state as uint16 bf16 bit patterns."""
        out = self.hid_out().cpu().numpy().view(np.uint16)
        self.check_status()
        return out

    def check_status(self):
        code = int(self.status.item())
        if code != 0:
            raise xb.XemaError(xb.XEMA_ETIMEOUT, "device status word 0x%08x" % (code & 0xFFFFFFFF))
