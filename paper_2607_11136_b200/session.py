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
    the phases whose trace exceeds the budget) and one count for the whole block; `serialize`
    lets that search split a phase into sub-batches instead of row chunks where the batch allows
    it (temporary serialization).  `axes` gives the split axis per phase for explicit `chunks`.
    `shard` = (p, P) binds the plan of one sequence-parallel shard (explicit `chunks` only): the
    session's input and output are then the shard's own token rows, and `forward_sharded` runs the
    step with the caller's exchange of keys and values in the middle of every block.
    `guard_bytes` > 0 binds the debug layout with a guard band after every tensor (explicit
    `chunks` only); `forward_guarded` then runs op by op and checks the bands.
    """

    def __init__(self, template, weights: Sequence[dict], chunks=None,
                 budget_bytes: Optional[int] = None, max_chunks: int = 64, device="cuda:0",
                 arena: Optional[torch.Tensor] = None, per_phase: bool = True, axes=None, serialize: bool = False,
                 shard=None, guard_bytes: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU fallback)")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.template = template
        self.cfg = xb.make_config(template)
        if chunks is None:
            if budget_bytes is None:
                raise ValueError("give chunks or budget_bytes")
            if serialize:
                chunks, axes, _ = xb.xema_mitigation_for_budget(self.cfg, int(budget_bytes), max_chunks)
                search = xb.xema_mitigation_for_budget
            else:
                search = xb.xema_phase_chunks_for_budget if per_phase else xb.xema_chunks_for_budget
                chunks, _ = search(self.cfg, int(budget_bytes), max_chunks)
            if chunks is None:
                raise xb.XemaError(xb.XEMA_EBUDGET, search.__name__)
        self.budget_bytes = budget_bytes
        if shard is not None and budget_bytes is not None:
            raise ValueError("a sharded session takes explicit chunks")
        if guard_bytes and budget_bytes is not None:
            raise ValueError("a guarded session takes explicit chunks")
        self.plan = xb.Plan(self.cfg, chunks, axes, shard, guard_bytes)
        self.chunks = chunks
        self.phase_chunks = self.plan.phase_chunks
        self.axes = self.plan.axes
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
        self.seq_all = template.s_text + template.grid_t * template.grid_h * template.grid_w
        self.seq = self.plan.rows          # token rows of this session's tensors (all of them unless sharded)

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

    def kv(self, block: int = 0) -> torch.Tensor:
        """Keys and values of `block`, [B, S, 2D] over ALL token rows (K half first per row)."""
        t = self.template
        _, off = self.plan.gather_point(block)
        n = 2 * t.batch * self.seq_all * 2 * t.hidden
        return self.arena[off:off + n].view(torch.int16).view(t.batch, self.seq_all, 2 * t.hidden)

    def forward_sharded(self, exchange, stream: Optional[torch.cuda.Stream] = None):
        """The forward pass of a sequence-parallel shard: for every block, the ops up to its
        gather point, then `exchange(block)` -- which must leave the other shards' rows of
        `self.kv(block)` in place, ordered after the enqueued work on `stream` and before what is
        enqueued next -- then on to the next gather point."""
        s = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        at = 0
        for l in range(self.template.n_blocks):
            op, _ = self.plan.gather_point(l)
            self.plan.forward_range(at, op, s)
            exchange(l)
            at = op
        self.plan.forward_range(at, self.plan.n_ops, s)

    GUARD_PATTERN = 0xA5

    def _guard(self, d) -> torch.Tensor:
        g = self.plan.guard_bytes
        return self.arena[d["offset"] + d["bytes"]:d["offset"] + d["bytes"] + g]

    def forward_guarded(self, stream: Optional[torch.cuda.Stream] = None, exchange=None):
        """The forward pass one op at a time over the guarded layout: the guard band of a tensor
        is filled with a pattern just before the op that gives birth to it (for the inputs: now,
        so call this after set_inputs) and checked after every op for as long as the tensor
        lives.  Returns the violations as (op index, op name, tensor name, damaged bytes): a
        kernel that writes past the end of its tensor is caught at the op that did it.  An empty
        list means every band stayed intact.  `exchange(block)`: as in forward_sharded."""
        if not self.plan.guard_bytes:
            raise ValueError("the session was not created with guard_bytes")
        st = stream or torch.cuda.current_stream(self.device)
        tensors = self.plan.tensors()
        gather = {self.plan.gather_point(l)[0]: l for l in range(self.template.n_blocks)} if exchange else {}
        bad = []
        with torch.cuda.stream(st):
            for k in range(self.plan.n_ops):
                for d in tensors:
                    if d["birth"] == k:
                        self._guard(d).fill_(self.GUARD_PATTERN)
                if k in gather:
                    exchange(gather[k])
                self.plan.forward_range(k, k + 1, st.cuda_stream)
                name = self.plan.op(k)["name"]
                for d in tensors:
                    if d["birth"] <= k < d["death"]:
                        n = int((self._guard(d) != self.GUARD_PATTERN).sum().item())
                        if n:
                            bad.append((k, name, d["name"], n))
        return bad

    def capture(self, stream: Optional[torch.cuda.Stream] = None) -> "torch.cuda.CUDAGraph":
        """Records one forward pass into a CUDA graph (every address is static, so the graph
        stays valid for as long as the session lives); `graph.replay()` then costs one launch on
        the host instead of one per kernel.  The first call warms the kernels up eagerly."""
        st = stream or torch.cuda.Stream(self.device)
        st.wait_stream(torch.cuda.current_stream(self.device))
        with torch.cuda.stream(st):
            self.forward(st)                      # one-time function attributes are set outside capture
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            self.forward(st)
        torch.cuda.current_stream(self.device).wait_stream(st)
        return g

    def output_bits(self) -> np.ndarray:
        """Synchronises and returns the output hidden state as uint16 bf16 bit patterns."""
        out = self.hid_out().cpu().numpy().view(np.uint16)
        self.check_status()
        return out

    def check_status(self):
        code = int(self.status.item())
        if code != 0:
            raise xb.XemaError(xb.XEMA_ETIMEOUT, "device status word 0x%08x" % (code & 0xFFFFFFFF))

    # ---- host-to-host pipeline ----------------------------------------------------------
    def run_pipelined(self, x_hosts, temb_hosts, out_hosts, stream: Optional[torch.cuda.Stream] = None):
        """One forward per (x, temb) pair of pinned host tensors, results into the pinned
        `out_hosts`; the host->device copy of step i+1 and the device->host copy of step i-1
        run on their own streams while step i computes.  The arena itself cannot take the next
        input early (its input slot is reused inside the block), so the copies go through one
        staging buffer per direction, outside the arena; `staging_bytes` says how large they
        are.  Returns after everything was enqueued; synchronise `stream` and the returned
        event before reading `out_hosts`."""
        compute = stream or torch.cuda.current_stream(self.device)
        if not hasattr(self, "_pipe"):
            self._pipe = {
                "h2d": torch.cuda.Stream(self.device), "d2h": torch.cuda.Stream(self.device),
                "x": torch.empty_like(self.hid_in()), "temb": torch.empty_like(self.temb()),
                "y": torch.empty_like(self.hid_out()),
            }
        pp = self._pipe
        # staging input consumed by the arena copy / staging output read back by the host copy;
        # carried over from an earlier call, whose last copies may still be in flight
        in_free, out_free = pp.get("in_free"), pp.get("out_free")
        if in_free is None:
            in_free, out_free = torch.cuda.Event(), torch.cuda.Event()
            in_free.record(compute)
            out_free.record(compute)
        done = None
        for x_h, t_h, y_h in zip(x_hosts, temb_hosts, out_hosts):
            ready = torch.cuda.Event()
            with torch.cuda.stream(pp["h2d"]):
                pp["h2d"].wait_event(in_free)
                pp["x"].copy_(x_h.view(pp["x"].shape), non_blocking=True)
                pp["temb"].copy_(t_h.view(pp["temb"].shape), non_blocking=True)
                ready.record(pp["h2d"])
            with torch.cuda.stream(compute):
                compute.wait_event(ready)
                self.hid_in().copy_(pp["x"], non_blocking=True)
                self.temb().copy_(pp["temb"], non_blocking=True)
                in_free = torch.cuda.Event()
                in_free.record(compute)
                self.forward(compute)
                compute.wait_event(out_free)
                pp["y"].copy_(self.hid_out(), non_blocking=True)
                produced = torch.cuda.Event()
                produced.record(compute)
            with torch.cuda.stream(pp["d2h"]):
                pp["d2h"].wait_event(produced)
                y_h.view(pp["y"].shape).copy_(pp["y"], non_blocking=True)
                out_free = torch.cuda.Event()
                out_free.record(pp["d2h"])
                done = out_free
        pp["in_free"], pp["out_free"] = in_free, out_free
        return done

    @property
    def staging_bytes(self) -> int:
        t = self.template
        return 2 * (2 * t.batch * self.seq * t.hidden) + 2 * t.batch * t.temb_dim


def all_gather_rows(full: torch.Tensor, row_ranges, group=None):
    """The exchange of sequence parallelism on a [B, S, W] tensor every rank holds in full size:
    rank r has filled rows row_ranges[r] = (first row, rows) of every batch element; afterwards
    every rank holds all rows.  One broadcast per (rank, batch element) -- the row ranges differ
    in size by up to one row, which a plain all-gather of equal parts cannot express -- straight
    into the tensor itself (for a session: into its own arena); no peer memory is ever read by a
    kernel.  Works on CPU tensors (gloo) and CUDA tensors (NCCL)."""
    import torch.distributed as dist
    for r, (r0, n) in enumerate(row_ranges):
        for b in range(full.shape[0]):
            dist.broadcast(full[b, r0:r0 + n], src=dist.get_global_rank(group, r) if group is not None else r, group=group)
