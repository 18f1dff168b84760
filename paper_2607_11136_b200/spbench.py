"""Sequence-parallel shards of a block or step, timed.

  python -m paper_2607_11136_b200.spbench --workload cogvideox --shards 4 --chunks 1,1,2

One process, one GPU: the P shards of the paper's sequence parallelism (section "Execution
Configurations": the latent sequence split across GPUs) run one after the other, each in its own
planned arena; the exchange of keys and values between them is a device-to-device copy of every
shard's rows into every other shard's kv tensor (what an all-gather into the ranks' own arenas
leaves behind).  What this measures is the COMPUTE of one rank of a P-GPU group -- how evenly the
block's work divides -- not the group: the exchange over NVLink is not run, only its byte count
is reported, with the time those bytes take at a stated link rate.  The outputs are checked to
be the bits of the unsharded run.

Under torchrun with P ranks (one GPU each) rank r runs shard (r, P) and the exchange is
`session.all_gather_rows` over NCCL; the time is the slowest rank's.  That path has only been run
with two gloo ranks on CPU for its bookkeeping; it has not been timed on more than one GPU.

Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from xema_inputs import make_activations, make_block_weights, template

from . import binding as xb
from .session import BlockSession, all_gather_rows

LINK_GBS = 770.0   # measured peer-copy rate per direction on this machine's NVLink 5 (nominal 900)


def _events(n):
    return [torch.cuda.Event(enable_timing=True) for _ in range(n)]


def _segments(sess):
    """Op ranges of a shard between the gather points: [(first, end), ...], one more than blocks."""
    pts = [sess.plan.gather_point(l)[0] for l in range(sess.template.n_blocks)]
    edges = [0] + pts + [sess.plan.n_ops]
    return [(edges[i], edges[i + 1]) for i in range(len(edges) - 1)]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="cogvideox")
    ap.add_argument("--shards", type=int, default=4)
    ap.add_argument("--chunks", default="1,1,2", help="per-phase chunk counts of every shard and of the unsharded run")
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    a = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    chunks = tuple(int(v) for v in a.chunks.split(","))
    t = template(a.workload)
    weights = [make_block_weights(t, l) for l in range(t.n_blocks)]
    x, temb = make_activations(t)
    x_dev = torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to(dev)
    temb_dev = torch.from_numpy(np.ascontiguousarray(temb).view(np.int16)).to(dev)
    stream = torch.cuda.current_stream(dev)
    kv_bytes_block = 2 * t.batch * t.seq * 2 * t.hidden           # bf16 [B, S, 2D]

    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        P = world
        sess = BlockSession(t, weights, chunks=chunks, shard=(rank, P), device=dev)
        ranges = [xb.xema_shard_rows(sess.cfg, p, P) for p in range(P)]
        x_own = x_dev[:, sess.plan.row0:sess.plan.row0 + sess.plan.rows].contiguous()
        segs = _segments(sess)

        def step():
            sess.set_inputs(x_own, temb_dev, non_blocking=True)
            for i, (lo, hi) in enumerate(segs):
                sess.plan.forward_range(lo, hi, stream.cuda_stream)
                if i < t.n_blocks:
                    all_gather_rows(sess.kv(i), ranges)
        for _ in range(a.warmup):
            step()
        ev = _events(2)
        dist.barrier()
        torch.cuda.synchronize()
        ev[0].record(stream)
        for _ in range(a.steps):
            step()
        ev[1].record(stream)
        torch.cuda.synchronize()
        ms = torch.tensor([ev[0].elapsed_time(ev[1]) / a.steps], dtype=torch.float64, device=dev)
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        sess.check_status()
        if rank == 0:
            print(json.dumps({"workload": a.workload, "shards": P, "chunks": list(chunks), "mode": "one rank per GPU, NCCL",
                              "ms_per_step": float(ms.item()), "arena_bytes_per_shard": int(sess.plan.peak_bytes),
                              "kv_bytes_received_per_rank_per_block": int(kv_bytes_block * (P - 1) / P)}), flush=True)
        dist.destroy_process_group()
        return

    P = a.shards
    full = BlockSession(t, weights, chunks=chunks, device=dev)
    dev_w = full.weights

    def full_step():
        full.set_inputs(x_dev, temb_dev, non_blocking=True)
        full.forward(stream)
    for _ in range(a.warmup):
        full_step()
    ev = _events(2)
    torch.cuda.synchronize()
    ev[0].record(stream)
    for _ in range(a.steps):
        full_step()
    ev[1].record(stream)
    torch.cuda.synchronize()
    ms_full = ev[0].elapsed_time(ev[1]) / a.steps
    want = full.output_bits().copy()
    full_peak = int(full.plan.peak_bytes)
    del full

    shards = [BlockSession(t, dev_w, chunks=chunks, shard=(p, P), device=dev) for p in range(P)]
    x_own = [x_dev[:, s.plan.row0:s.plan.row0 + s.plan.rows].contiguous() for s in shards]
    segs = _segments(shards[0])
    n_seg = len(segs)
    per_shard_ms = np.zeros(P)
    exchange_ms = 0.0

    def sp_step(timed):
        nonlocal exchange_ms
        evs = [[_events(2) for _ in range(n_seg)] for _ in range(P)] if timed else None
        ex = [_events(2) for _ in range(t.n_blocks)] if timed else None
        for p, s in enumerate(shards):
            s.set_inputs(x_own[p], temb_dev, non_blocking=True)
        for i, (lo, hi) in enumerate(segs):
            for p, s in enumerate(shards):
                assert _segments(s)[i] == (lo, hi)
                if timed:
                    evs[p][i][0].record(stream)
                s.plan.forward_range(lo, hi, stream.cuda_stream)
                if timed:
                    evs[p][i][1].record(stream)
            if i < t.n_blocks:
                if timed:
                    ex[i][0].record(stream)
                for src in shards:
                    r0, n = src.plan.row0, src.plan.rows
                    for dst in shards:
                        if dst is not src:
                            dst.kv(i)[:, r0:r0 + n].copy_(src.kv(i)[:, r0:r0 + n], non_blocking=True)
                if timed:
                    ex[i][1].record(stream)
        if timed:
            torch.cuda.synchronize()
            for p in range(P):
                per_shard_ms[p] += sum(e0.elapsed_time(e1) for e0, e1 in evs[p])
            exchange_ms += sum(e0.elapsed_time(e1) for e0, e1 in ex)

    for _ in range(a.warmup):
        sp_step(False)
    for _ in range(a.steps):
        sp_step(True)
    per_shard_ms /= a.steps
    exchange_ms /= a.steps
    for s in shards:
        s.check_status()
    got = np.concatenate([s.output_bits() for s in shards], axis=1)
    recv = kv_bytes_block * (P - 1) / P
    out = {
        "workload": a.workload, "shards": P, "chunks": list(chunks),
        "mode": "P shards in turn on one GPU; exchange emulated by device copies and not part of the shard times",
        "ms_unsharded": ms_full,
        "ms_shard": [float(v) for v in per_shard_ms], "ms_shard_max": float(per_shard_ms.max()),
        # how evenly the work divides: 1.0 = every rank does exactly 1/P of the unsharded step
        "compute_partition_efficiency": ms_full / (P * float(per_shard_ms.max())),
        "arena_bytes_unsharded": full_peak, "arena_bytes_per_shard": [int(s.plan.peak_bytes) for s in shards],
        "kv_bytes_received_per_rank_per_block": int(recv),
        "exchange_ms_per_block_at_link_rate": recv / (LINK_GBS * 1e9) * 1e3, "link_rate_gbs": LINK_GBS,
        "exchange_emulated_on_device_ms_per_step": exchange_ms,
        "bit_identical_to_unsharded": bool(got.shape == want.shape and np.array_equal(got, want)),
    }
    est = out["ms_shard_max"] + t.n_blocks * out["exchange_ms_per_block_at_link_rate"]
    out["estimated_step_ms_exchange_not_overlapped"] = est
    out["estimated_speedup_over_one_gpu"] = ms_full / est
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
