"""Replays the block's tensor-lifetime trace through PyTorch's caching allocator and compares what
it reserves with the planned arena (the paper's layout experiment: reserved memory of the caching
allocator, of `expandable_segments`, and of the static layout against the active peak).

  python -m paper_2607_11136_b200.alloc_replay --sequence cogvideox:1,1,2 flux:1 cogvideox:8 --rounds 3
  python -m paper_2607_11136_b200.alloc_replay --sequence step:1,1,2 --expandable

Every tensor of the trace becomes one `torch.empty(bytes, uint8)` at its birth op and is dropped at
its death op, in op order (deaths before births at the same op), so the allocator sees exactly the
request stream an eager framework would issue for this block.  No kernel runs.  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import contextlib
import json
import os
import subprocess
import sys

from . import binding as xb


def alloc_events(tensors, n_ops):
    """[(op, 'free' | 'alloc', tensor index)] in replay order: at every op first the tensors whose
    lifetime ended, then the ones born there (in id order).  Tensors still live after the last op
    are freed at op == n_ops."""
    by_birth, by_death = {}, {}
    for i, d in enumerate(tensors):
        by_birth.setdefault(d["birth"], []).append(i)
        by_death.setdefault(d["death"], []).append(i)
    ev = []
    for op in range(n_ops + 1):
        ev += [(op, "free", i) for i in by_death.get(op, [])]
        ev += [(op, "alloc", i) for i in by_birth.get(op, [])]
    return ev


def parse_item(item: str):
    name, _, ch = item.partition(":")
    c = [int(v) for v in ch.split(",")] if ch else [1]
    return name, (c[0] if len(c) == 1 else tuple(c))


def replay(sequence, rounds: int, device: str = "cuda:0") -> dict:
    import torch
    from xema_inputs import template
    torch.cuda.set_device(device)
    torch.cuda.empty_cache()
    torch.cuda.reset_peak_memory_stats()
    # whatever the process already holds (weights of earlier work, say) is not this replay's
    base_alloc = torch.cuda.memory_allocated()
    base_reserved = torch.cuda.memory_reserved()
    plans = []
    for name, chunks in sequence:
        cfg = xb.make_config(template(name))
        triple = (chunks,) * 3 if isinstance(chunks, int) else chunks
        tensors, n_ops = xb.xema_trace_phases(cfg, triple)
        _, peak, live = xb.xema_plan_arena(tensors)
        plans.append({"workload": name, "chunks": list(triple), "arena_peak_bytes": peak, "max_live_bytes": live,
                      "tensors": len(tensors), "events": alloc_events(tensors, n_ops), "sizes": [d["bytes"] for d in tensors]})
    # The replay allocates from a memory pool of its own: segments that the process already holds
    # (partly used ones keep their free space through empty_cache) would otherwise take the
    # replay's tensors without the reserved figure moving at all.
    pool = None
    scope = contextlib.nullcontext()
    if hasattr(torch.cuda, "MemPool") and hasattr(torch.cuda, "use_mem_pool"):
        try:
            pool = torch.cuda.MemPool()
            scope = torch.cuda.use_mem_pool(pool)
        except RuntimeError:
            pool, scope = None, contextlib.nullcontext()
    reserved_peak = 0
    with scope:
        for _ in range(rounds):
            for p in plans:
                held = {}
                for _, kind, i in p["events"]:
                    if kind == "alloc":
                        held[i] = torch.empty(p["sizes"][i], dtype=torch.uint8, device=device)
                    else:
                        del held[i]
                assert not held
                if pool is not None:      # a pool's segments stay until it is destroyed: the sum is its peak
                    reserved_peak = max(reserved_peak, sum(seg["total_size"] for seg in pool.snapshot()))
    if pool is None:
        reserved_peak = torch.cuda.max_memory_reserved() - base_reserved
    out = {
        "sequence": [{k: p[k] for k in ("workload", "chunks", "arena_peak_bytes", "max_live_bytes", "tensors")} for p in plans],
        "rounds": rounds,
        "static_arena_bytes": max(p["arena_peak_bytes"] for p in plans),
        "active_peak_bytes": max(p["max_live_bytes"] for p in plans),
        "torch_allocated_peak_bytes": torch.cuda.max_memory_allocated() - base_alloc,
        "torch_reserved_peak_bytes": reserved_peak,
        "allocator": os.environ.get("PYTORCH_CUDA_ALLOC_CONF", "default (caching allocator)"),
    }
    out["utilisation_torch"] = out["active_peak_bytes"] / max(out["torch_reserved_peak_bytes"], 1)
    out["utilisation_static"] = out["active_peak_bytes"] / out["static_arena_bytes"]
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--sequence", nargs="+", default=["cogvideox:1,1,2"],
                    help="items workload[:C | :CA,CB,CC], replayed in this order")
    ap.add_argument("--rounds", type=int, default=3)
    ap.add_argument("--expandable", action="store_true", help="run with expandable_segments:True")
    a = ap.parse_args()
    if a.expandable and "expandable_segments" not in os.environ.get("PYTORCH_CUDA_ALLOC_CONF", ""):
        env = dict(os.environ, PYTORCH_CUDA_ALLOC_CONF="expandable_segments:True")
        argv = [sys.executable, "-m", "paper_2607_11136_b200.alloc_replay"] + sys.argv[1:]
        raise SystemExit(subprocess.call(argv, env=env))
    print(json.dumps(replay([parse_item(s) for s in a.sequence], a.rounds)), flush=True)


if __name__ == "__main__":
    main()
