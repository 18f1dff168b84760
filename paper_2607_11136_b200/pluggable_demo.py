"""A plain eager-PyTorch DiT block (library kernels of torch, none of this repository's) run on
the static-memory runtime: warm-up, record, plan, replay; checks that replay serves every request
from the planned arena and reproduces the recorded step bit for bit.  Prints one JSON line.

    python -m paper_2607_11136_b200.pluggable_demo [--tokens 4096 --hidden 1024 --heads 16 --chunks 2]
    python -m paper_2607_11136_b200.pluggable_demo --caching     # the same step on torch's own allocator
"""
from __future__ import annotations

import argparse
import json

import torch
import torch.nn.functional as F


def make_step(a, dev):
    g = torch.Generator(device="cpu").manual_seed(0)
    D, H, S, Fd = a.hidden, a.heads, a.tokens, 4 * a.hidden
    rnd = lambda *shape, s=0.02: (torch.randn(*shape, generator=g) * s).to(torch.bfloat16)
    host = {"x": rnd(1, S, D, s=1.0), "w_qkv": rnd(3 * D, D), "b_qkv": rnd(3 * D), "w_o": rnd(D, D), "b_o": rnd(D),
            "w_1": rnd(Fd, D), "b_1": rnd(Fd), "w_2": rnd(D, Fd), "b_2": rnd(D)}
    state = {}

    def load():
        # parameters and the input are long-lived: allocated before recording starts
        for k, v in host.items():
            state[k] = v.to(dev)

    def step():
        W = state
        x = W["x"]
        h = F.layer_norm(x, (D,))
        qkv = F.linear(h, W["w_qkv"], W["b_qkv"]).view(1, S, 3, H, D // H).permute(2, 0, 3, 1, 4)
        del h
        o = F.scaled_dot_product_attention(qkv[0], qkv[1], qkv[2])
        del qkv
        res = x + F.linear(o.transpose(1, 2).reshape(1, S, D), W["w_o"], W["b_o"])
        del o
        y = torch.empty_like(res)
        for rows in torch.arange(S, device="cpu").chunk(a.chunks):       # sequence-chunked FFN
            r0, r1 = int(rows[0]), int(rows[-1]) + 1
            h2 = F.layer_norm(res[:, r0:r1], (D,))
            gact = F.gelu(F.linear(h2, W["w_1"], W["b_1"]), approximate="tanh")
            del h2
            y[:, r0:r1] = res[:, r0:r1] + F.linear(gact, W["w_2"], W["b_2"])
            del gact
        out = y.cpu()                # copy the result out; everything allocated here dies here
        del y, res
        return out

    return load, step


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--tokens", type=int, default=4096)
    ap.add_argument("--hidden", type=int, default=1024)
    ap.add_argument("--heads", type=int, default=16)
    ap.add_argument("--chunks", type=int, default=2)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--caching", action="store_true", help="torch's caching allocator instead of the plug-in")
    a = ap.parse_args()
    dev = torch.device("cuda:0")
    if a.caching:
        load, step = make_step(a, dev)
        load()
        base = torch.cuda.memory_allocated()
        for _ in range(2):
            step()
        torch.cuda.synchronize()
        torch.cuda.reset_peak_memory_stats()
        base_reserved = torch.cuda.memory_reserved()
        for _ in range(a.steps):
            step()
        torch.cuda.synchronize()
        print(json.dumps({"allocator": "torch caching allocator",
                          "step_allocated_peak_bytes": torch.cuda.max_memory_allocated() - base,
                          "reserved_peak_bytes": torch.cuda.max_memory_reserved(),
                          "reserved_before_bytes": base_reserved, "parameter_bytes": base}), flush=True)
        return
    from . import binding as xb
    from . import pluggable
    pluggable.install()
    load, step = make_step(a, dev)
    load()
    rt = pluggable.StaticRuntime(dev)
    rt.warm_up(step)
    want = rt.record(step)
    peak = rt.plan()
    served0, fallback0, _ = xb.xema_pluggable_stats()
    identical = True
    for _ in range(a.steps):
        got = rt.replay(step)
        identical = identical and bool(torch.equal(got, want))
    served, fallback, nxt = xb.xema_pluggable_stats()
    # a tensor allocated in replay mode sits at its planned offset
    xb.xema_pluggable_mode(xb.ALLOC_REPLAY)
    xb.xema_pluggable_step_begin()
    first = torch.empty(rt.requests[0]["bytes"], dtype=torch.uint8, device=dev) if rt.requests else None
    at_offset = first is not None and first.data_ptr() == rt.base + rt.offsets[0] and rt.contains(first)
    del first
    xb.xema_pluggable_mode(xb.ALLOC_PASSTHROUGH)
    sizes = [r["bytes"] for r in rt.requests]
    print(json.dumps({
        "allocator": "xema plug-in", "requests_per_step": len(rt.requests), "events": rt.n_events,
        "sum_of_request_bytes": sum(sizes), "largest_request_bytes": max(sizes),
        "arena_peak_bytes": peak, "max_live_bytes": rt.max_live_bytes,
        "served": served - served0, "fallback": fallback - fallback0, "next_index_after_step": nxt,
        "replay_identical_to_record": identical, "first_request_at_planned_offset": bool(at_offset),
        "finite": bool(torch.isfinite(want.float()).all()),
    }), flush=True)


if __name__ == "__main__":
    main()
