#!/usr/bin/env python
"""Benchmark of the chunked, arena-placed DiT block on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cogvideox] [--budget-mib M]
  python bench.py --impl reference ...        # times the CPU oracle instead

One step = one pass of the whole hot path (modulation, LayerNorm+modulate, QKV GEMMs, RMSNorm +
RoPE, attention, gated projection, FFN) over one batch of seeded synthetic input, sequence-
chunked only in the phases whose memory trace exceeds the byte budget (per-phase chunk counts;
--uniform-chunks uses one count for the whole block instead).  Prints ONE JSON
line (see the keys below).  Under torchrun every rank runs the same workload on its own GPU
(independent replicas, no data-path collective); the value is the sum over ranks divided by the
slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from xema_inputs import bits_to_f64, make_activations, make_block_weights, sample_rows, template  # noqa: E402

METRIC = "DiT block TFLOP/s (bf16 in, fp32 accumulate) at a memory budget; block latency in ms_per_step"
UNIT = "TFLOP/s"
CPU_SAMPLE_ROWS = 1024


def block_flops(t) -> float:
    """Algorithmic flops of one block: the five GEMMs plus attention (4*S^2*D per batch element)."""
    S, D, F, B = t.seq, t.hidden, t.ffn, t.batch
    return B * (2.0 * S * D * (3 * D + D + 2 * F) + 4.0 * S * S * D) * t.n_blocks


def sample_flops(t, n_rows) -> float:
    """Flops the row-sampled oracle performs: k and v for every token, everything else for the
    sampled rows only."""
    S, D, F, B = t.seq, t.hidden, t.ffn, t.batch
    return B * (2.0 * S * D * 2 * D + n_rows * (2.0 * D * (2 * D + 2 * F) + 4.0 * S * D))


def load_peaks():
    """Measured roofline denominators written by the driver; else the pool's fallback numbers."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_burst": float(p["bf16_tflops"]),
                "bf16_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


def max_over_ranks(ms: float, dist, device) -> float:
    """Slowest rank's time (all ranks call this); identity without a process group."""
    if dist is None:
        return ms
    import torch
    tt = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def whole_job_tflops(flops_per_replica: float, world: int, ms: float) -> float:
    """Replicas are independent: the job did world x flops in the slowest rank's time."""
    return world * flops_per_replica / (ms * 1e-3) / 1e12


# DRAM traffic of one attention launch (dram__bytes_read.sum + dram__bytes_write.sum under ncu, see
# profiles/attention_dh64_rows2222_keys17776_h48.md).  Captured inside this bench at the full 17776
# query rows: 422.9 MB (329.0 read + 93.9 written; algorithmic 440.3 -- q is still in L2 from the Q
# projection).  Captured alone at 2222 rows: 266.6 MB (algorithmic 246.2), of which k and v (4*S*D
# bytes, independent of the number of query rows) are read once and the rest scales with the query
# rows; other row counts are scaled from that capture.  Not measured in the timed run.
def attention_traffic_bytes(t, rows: int) -> float:
    if (t.seq, t.hidden, t.head_dim) != (17776, 3072, 64):
        return None
    if rows == t.seq:
        return 422.9e6
    kv = 4.0 * t.seq * t.hidden
    return kv + (266.6e6 - kv) * rows / 2222.0


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU while the timed region runs: NVML
    polled every few milliseconds from a thread (read-only queries), else nvidia-smi at its
    fastest period."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NVML_REASONS = ((0x8, "hw_slowdown"), (0x40, "hw_thermal_slowdown"), (0x20, "sw_thermal_slowdown"),
                    (0x4, "sw_power_cap"))

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.nvml, self.stop_flag = index, [], None, None, False
        self.samples = []

    def _nvml_handle(self):
        import pynvml
        pynvml.nvmlInit()
        try:
            import torch
            uuid = str(torch.cuda.get_device_properties(self.index).uuid)
            h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
        except Exception:
            h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
        return pynvml, h

    def start(self):
        try:
            self.nvml, self.handle = self._nvml_handle()
            self.sm_max = float(self.nvml.nvmlDeviceGetMaxClockInfo(self.handle, self.nvml.NVML_CLOCK_SM))
            try:
                self.power_limit = self.nvml.nvmlDeviceGetEnforcedPowerLimit(self.handle) / 1000.0   # read-only
            except Exception:
                self.power_limit = None
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _poll(self):
        n, h = self.nvml, self.handle
        while not self.stop_flag:
            try:
                self.samples.append((float(n.nvmlDeviceGetClockInfo(h, n.NVML_CLOCK_SM)),
                                     n.nvmlDeviceGetPowerUsage(h) / 1000.0,
                                     int(n.nvmlDeviceGetCurrentClocksEventReasons(h))))
            except Exception:
                pass
            time.sleep(0.005)

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.nvml is not None:
            self.stop_flag = True
            self.thread.join(timeout=2)
            sm = [s[0] for s in self.samples]
            reasons = sorted({name for s in self.samples for bit, name in self.NVML_REASONS if s[2] & bit})
            return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                    "sm_max_mhz": self.sm_max, "power_w_max": max((s[1] for s in self.samples), default=None),
                    "power_limit_w": self.power_limit,
                    "samples": len(sm), "source": "nvml, 5 ms period", "reasons": reasons}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no clock source available"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); power.append(float(r[2]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "source": "nvidia-smi",
                "reasons": sorted(reasons)}


def oracle_inputs(t):
    w = {k: bits_to_f64(v) for k, v in make_block_weights(t, 0).items()}
    x, temb = make_activations(t)
    return w, bits_to_f64(x), bits_to_f64(temb)


def time_oracle_sample(t, n_rows=CPU_SAMPLE_ROWS, inputs=None):
    """Times the float64 oracle, as it stands, on a bounded sample of the workload: keys and
    values of every token, then the complete block for `n_rows` seeded token rows."""
    from oracle import block as ob
    w, x, temb = inputs or oracle_inputs(t)
    rows = sample_rows(t, n_random=n_rows)
    t0 = time.perf_counter()
    ob.block_forward(t, w, x, temb, rows=rows)
    dt = time.perf_counter() - t0
    return dt, len(rows)


def run_reference(args):
    """`--impl reference`: the CPU oracle on the host cores, on the same config and metric."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    t = template(args.workload).with_(n_blocks=1)
    cores = len(os.sched_getaffinity(0))
    times, n_rows = [], 0
    inputs = oracle_inputs(t)
    for i in range(args.warmup + args.steps):
        dt, n_rows = time_oracle_sample(t, min(args.cpu_rows, 256), inputs)
        if i >= args.warmup:
            times.append(dt)
    mean = float(np.mean(times))
    value = sample_flops(t, n_rows) / mean / 1e12
    sample = ("k, v for all %d tokens plus the complete block for %d seeded token rows of one block "
              "(%.3g of %.3g flop)" % (t.seq, n_rows, sample_flops(t, n_rows), block_flops(t)))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "batch": t.batch, "tokens": t.seq, "hidden": t.hidden, "heads": t.heads,
                   "head_dim": t.head_dim, "ffn": t.ffn, "n_blocks": 1, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="xema", choices=["xema", "reference"])
    ap.add_argument("--workload", default="cogvideox", choices=["tiny", "cogvideox", "flux", "longvideo", "step"])
    ap.add_argument("--budget-mib", type=float, default=640.0,
                    help="activation byte budget; the least chunking whose arena peak fits is used")
    ap.add_argument("--chunks", default="", help="force a chunk count C, or per-phase counts CA,CB,CC, "
                                                 "instead of a budget")
    ap.add_argument("--uniform-chunks", action="store_true",
                    help="budget search over one chunk count for all three phases")
    ap.add_argument("--cpu-rows", type=int, default=CPU_SAMPLE_ROWS)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="also time chunk counts 1, 2, 4, 8 (outside the timed region)")
    ap.add_argument("--sustained-seconds", type=float, default=3.0,
                    help="length of the extra sustained leg (after 2 s of pre-heat); 0 skips it")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)

    import torch
    from paper_2607_11136_b200 import binding as xb
    from paper_2607_11136_b200.session import BlockSession

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    t = template(args.workload)
    cfg = xb.make_config(t)
    forced = None
    if args.chunks:
        c = [int(v) for v in args.chunks.split(",")]
        forced = c[0] if len(c) == 1 else tuple(c)
    budget = None if forced else int(args.budget_mib * (1 << 20))
    weights = [make_block_weights(t, l) for l in range(t.n_blocks)]
    x_bits, temb_bits = make_activations(t)
    sess = BlockSession(t, weights, chunks=forced, budget_bytes=budget, device=dev,
                        per_phase=not args.uniform_chunks)
    n_launch = sess.plan.n_ops            # logical ops of the trace (fused ones launch nothing)
    n_kernels = sess.plan.launch_count()  # kernels actually launched per step
    ops = [sess.plan.op(i) for i in range(n_launch)]
    flops = block_flops(t)
    stream = torch.cuda.current_stream(dev)
    sess.set_inputs(x_bits, temb_bits)
    # The arena reuses the slots of the block input and of temb inside the block, so every step
    # has to be given its input again: device-resident copies, restored by a device-to-device copy
    # at the start of each step (inside the timed region; without it every step after the first
    # would run on leftovers -- NaNs -- and draw less power than real data does).
    x_dev = sess.hid_in().clone()
    temb_dev = sess.temb().clone()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # ---- device-resident timing: K steps, events on the launching stream -----------------------
    def timed_steps(n_steps, bracket=None):
        """n_steps steps, each restoring the inputs and issuing every op; clocks sampled
        meanwhile.  `bracket` = indices of the ops that get an event on either side (None: every
        op); the ops between two events go out in one call.  An event between two kernels costs
        about a microsecond of idle GPU, so the headline leg brackets only the dominant kernel
        (its duration is what the roofline needs) and the table of all ops comes from a pass of
        its own.  Returns (total ms, sorted per-step ms, restore ms, per-op dict of the bracketed
        ops, clocks)."""
        marks = set(range(n_launch)) if bracket is None else set(bracket)
        cuts = sorted({0, n_launch} | marks | {i + 1 for i in marks})
        segs = list(zip(cuts[:-1], cuts[1:]))
        sampler = ClockSampler(local)
        sampler.start()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(cuts))] for _ in range(n_steps)]
        ev_in = [torch.cuda.Event(enable_timing=True) for _ in range(n_steps)]
        barrier()
        for k in range(n_steps):
            ev_in[k].record(stream)
            sess.set_inputs(x_dev, temb_dev, non_blocking=True)
            for j, (lo, hi) in enumerate(segs):
                ev[k][j].record(stream)
                sess.plan.forward_range(lo, hi, stream.cuda_stream)
            ev[k][len(segs)].record(stream)
        barrier()
        clk = sampler.stop()
        total = ev_in[0].elapsed_time(ev[-1][len(segs)])
        steps_sorted = sorted(ev_in[k].elapsed_time(ev[k][len(segs)]) for k in range(n_steps))
        restore = sum(ev_in[k].elapsed_time(ev[k][0]) for k in range(n_steps)) / n_steps
        ops_t = {}
        for j, (lo, hi) in enumerate(segs):
            if hi != lo + 1 or lo not in marks:
                continue
            op = ops[lo]
            d = ops_t.setdefault(op["name"], {"ms": 0.0, "flops": 0.0, "bytes": 0.0, "launches": 0})
            d["ms"] += sum(ev[k][j].elapsed_time(ev[k][j + 1]) for k in range(n_steps)) / n_steps
            d["flops"] += op["flops"]; d["bytes"] += op["bytes"]; d["launches"] += 1
        return total, steps_sorted, restore, ops_t, clk

    for _ in range(args.warmup):
        sess.set_inputs(x_dev, temb_dev, non_blocking=True)
        sess.forward(stream)
    barrier()
    # which kernel dominates: a short pass with an event around every op, before the timed region
    _, _, _, calib, _ = timed_steps(max(2, min(args.warmup, 5)))
    dom_name = max(calib, key=lambda n_: calib[n_]["ms"])
    dom_ops = [i for i, op in enumerate(ops) if op["name"] == dom_name]
    free_before, _ = torch.cuda.mem_get_info(dev)
    total_ms, step_ms, restore_ms, dom_op, clocks = timed_steps(args.steps, bracket=dom_ops)
    free_after, _ = torch.cuda.mem_get_info(dev)
    sess.check_status()
    # the table of all ops: the same K steps again with an event around every op (not the headline)
    per_op_total_ms, _, _, per_op, per_op_clocks = timed_steps(args.steps)
    total_ms = max_over_ranks(total_ms, dist, dev)
    ms_per_step = total_ms / args.steps
    out_finite = bool(torch.isfinite(sess.hid_out().view(torch.bfloat16).float()).all().item())
    value = whole_job_tflops(flops, world, ms_per_step)

    # ---- sustained leg: the same loop after a pre-heat, long enough for the power governor --------
    sustained = None
    if args.sustained_seconds > 0:
        est = max(ms_per_step, 1e-3)
        for _ in range(max(1, int(2000.0 / est))):            # about 2 s of pre-heat, untimed
            sess.set_inputs(x_dev, temb_dev, non_blocking=True)
            sess.forward(stream)
        n_sus = max(3, int(args.sustained_seconds * 1000.0 / est))
        s_total, s_steps, _, s_dom, s_clk = timed_steps(n_sus, bracket=dom_ops)
        # the table of all ops in the same regime: a shorter pass right behind, an event around every op
        n_tab = max(3, n_sus // 4)
        s_tab_total, _, _, s_ops, s_tab_clk = timed_steps(n_tab)
        sess.check_status()
        s_total = max_over_ranks(s_total, dist, dev)
        sustained = {"steps": n_sus, "preheat_seconds": 2.0, "ms_per_step": s_total / n_sus,
                     "ms_median": s_steps[len(s_steps) // 2], "value": whole_job_tflops(flops, world, s_total / n_sus),
                     "clocks": s_clk, "per_op_raw": s_ops, "dom_raw": s_dom,
                     "per_op_pass": {"steps": n_tab, "ms_per_step": s_tab_total / n_tab, "clocks": s_tab_clk}}
        if s_clk.get("sm_mhz"):       # time x median clock: how the step depends on the clock it ran at
            sustained["sm_mcycles_per_step"] = sustained["ms_per_step"] * s_clk["sm_mhz"] / 1e3

    # ---- end to end through the public API: pinned host -> arena, forward, output -> host ------
    x_host = torch.from_numpy(x_bits.view(np.int16)).pin_memory()
    temb_host = torch.from_numpy(temb_bits.view(np.int16)).pin_memory()
    out_host = torch.empty_like(x_host).pin_memory()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def e2e_step():
        # the C ABI's host-buffer call: both copies and every launch on this stream, arena only
        sess.plan.forward_host(x_host.data_ptr(), temb_host.data_ptr(), out_host.data_ptr(), stream.cuda_stream)

    for _ in range(3):
        e2e_step()
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_serial_ms = max_over_ranks(e0.elapsed_time(e1), dist, dev) / args.steps
    # the same K steps with the copies of neighbouring steps overlapped with compute
    done = sess.run_pipelined([x_host] * 3, [temb_host] * 3, [out_host] * 3, stream)
    barrier()
    done.synchronize()
    e0.record(stream)
    done = sess.run_pipelined([x_host] * args.steps, [temb_host] * args.steps, [out_host] * args.steps, stream)
    stream.wait_event(done)
    e1.record(stream)
    barrier()
    sess.check_status()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), dist, dev) / args.steps
    h2d = int(x_host.numel() * 2 + temb_host.numel() * 2)
    d2h = int(out_host.numel() * 2)

    sweep = None
    if args.sweep and rank == 0:
        sweep = {}
        dev_w = sess.weights
        for C in (1, 2, 4, 8, (1, 1, 2), (1, 1, 3)):
            s2 = BlockSession(t, dev_w, chunks=C, device=dev)
            for _ in range(3):
                s2.set_inputs(x_dev, temb_dev, non_blocking=True)
                s2.forward(stream)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(dev)
            a.record(stream)
            for _ in range(10):
                s2.set_inputs(x_dev, temb_dev, non_blocking=True)
                s2.forward(stream)
            b.record(stream)
            torch.cuda.synchronize(dev)
            ms = a.elapsed_time(b) / 10
            sweep[str(C).replace(" ", "")] = {"ms": ms, "tflops": flops / ms / 1e9, "arena_bytes": s2.plan.peak_bytes}
            del s2
            torch.cuda.empty_cache()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel ---------------------------------------------------------
    peaks = load_peaks()
    TENSOR_OPS = ("KV", "Q", "ATTN", "PROJ", "FFN1", "FFN2")

    def regime_of(clk):
        """A kernel is compared with the sustained peak only when it was timed in that regime: the
        median SM clock more than 5 % below its maximum AND the board's power reading within 10 % of
        its limit.  A short leg whose clock has begun to fall while the (averaged) power reading is
        still far below the limit is compared with the burst peak, the larger denominator."""
        fast = clk.get("sm_mhz") and clk.get("sm_max_mhz") and clk["sm_mhz"] >= 0.95 * clk["sm_max_mhz"]
        limit = clk.get("power_limit_w") or 1000.0
        hot = clk.get("power_w_max") is not None and clk["power_w_max"] >= 0.9 * limit
        return "sustained" if (not fast and hot) else "burst"

    def roofline_of(ops_t, clk):
        dom = max(ops_t, key=lambda n: ops_t[n]["ms"])
        d = ops_t[dom]
        per_launch_s = d["ms"] * 1e-3 / d["launches"]
        regime = regime_of(clk)
        if dom in TENSOR_OPS:
            achieved = d["flops"] / d["launches"] / per_launch_s / 1e12
            peak = peaks["bf16_burst"] if regime == "burst" else peaks["bf16_sustained"]
            unit, bound = "TFLOP/s", "tensor"
        else:
            achieved = d["bytes"] / d["launches"] / per_launch_s / 1e9
            peak, unit, bound = peaks["hbm_gbs"], "GB/s", "hbm"
        r = {"kernel": dom, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
             "peak_source": "%s (%s: median SM clock %s of %s MHz, power up to %s of %s W)" % (
                 peaks["source"], regime if bound == "tensor" else "copy", clk.get("sm_mhz"), clk.get("sm_max_mhz"),
                 clk.get("power_w_max"), clk.get("power_limit_w")),
             "ms_per_launch": per_launch_s * 1e3, "launches_per_step": d["launches"]}
        if bound == "tensor":
            r["frac_of_burst"] = achieved / peaks["bf16_burst"]
            r["frac_of_sustained"] = achieved / peaks["bf16_sustained"]
            r["frac_of_nominal_2250"] = achieved / 2250.0
            r["peak_burst"], r["peak_sustained"] = peaks["bf16_burst"], peaks["bf16_sustained"]
        r["traffic"] = None
        if dom == "ATTN":
            r["traffic"] = attention_traffic_bytes(t, t.seq * t.n_blocks // d["launches"])
            r["traffic_source"] = ("not measured in this run: dram__bytes_read.sum + dram__bytes_write.sum of one ncu "
                                   "capture, see profiles/attention_dh64_*.md" if r["traffic"] else None)
        return r

    def breakdown_of(ops_t, step_ms_):
        return {n: {"ms": round(v["ms"], 4), "share": round(v["ms"] / step_ms_, 4),
                    "tflops": round(v["flops"] / (v["ms"] * 1e-3) / 1e12, 1) if v["ms"] > 0 else None,
                    "gbs": round(v["bytes"] / (v["ms"] * 1e-3) / 1e9, 1) if v["ms"] > 0 else None}
                for n, v in ops_t.items()}

    def tensor_ops_of(ops_t):
        ms = sum(v["ms"] for n, v in ops_t.items() if n in TENSOR_OPS)
        fl = sum(v["flops"] for n, v in ops_t.items() if n in TENSOR_OPS)
        tf = fl / (ms * 1e-3) / 1e12
        return {"tflops": tf, "ms": ms, "frac_of_burst": tf / peaks["bf16_burst"],
                "frac_of_sustained": tf / peaks["bf16_sustained"], "frac_of_nominal_2250": tf / 2250.0}

    roofline = roofline_of(dom_op, clocks)
    dom = roofline["kernel"]
    if dom == "ATTN" and t.head_dim == 64 and clocks.get("sm_max_mhz"):
        # context: with 64-wide heads there is one exponential per 4 * 64 flop and an SM retires 16 ex2 per
        # clock; three eighths of the exponentials run as a polynomial on the FMA pipe instead
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        mufu = 16.0 * sms * clocks["sm_max_mhz"] * 1e6 * 4 * t.head_dim / 1e12
        roofline["exp_rate_ceiling_tflops"] = {"all_on_mufu_at_max_clock": mufu, "five_eighths_on_mufu": mufu / 0.625}
    breakdown = breakdown_of(per_op, per_op_total_ms / args.steps)
    if sustained is not None:
        s_ops = sustained.pop("per_op_raw")
        sustained["roofline"] = roofline_of(sustained.pop("dom_raw"), sustained["clocks"])
        sustained["tensor_ops"] = tensor_ops_of(s_ops)
        sustained["per_op"] = breakdown_of(s_ops, sustained["per_op_pass"]["ms_per_step"])

    cpu = None
    if not args.no_cpu_baseline:
        dt, n_rows = time_oracle_sample(t.with_(n_blocks=1), args.cpu_rows)
        cpu = {"value": sample_flops(t, n_rows) / dt / 1e12, "unit": UNIT, "cores": len(os.sched_getaffinity(0)),
               "kind": "oracle", "seconds": dt,
               "sample": "k, v for all %d tokens plus the complete block for %d seeded token rows of one block"
                         % (t.seq, n_rows)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "ms_median": step_ms[len(step_ms) // 2],
        "ms_min": step_ms[0], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "batch": t.batch, "tokens": t.seq, "hidden": t.hidden,
                   "heads": t.heads, "head_dim": t.head_dim, "ffn": t.ffn, "n_blocks": t.n_blocks,
                   "budget_bytes": budget, "chunks": list(sess.phase_chunks),
                   "chunk_search": "forced" if forced else ("uniform" if args.uniform_chunks else "per_phase"),
                   "arena_bytes": sess.plan.peak_bytes,
                   "trace_max_live_bytes": sess.plan.max_live_bytes,
                   # the paper keeps a dynamic region of 5 % above the static reserved peak; this library has
                   # no dynamic allocations, the figure is reported for comparison only
                   "arena_bytes_plus_5pct_dynamic_region": int(sess.plan.peak_bytes * 1.05),
                   "device_bytes_allocated_by_forward": int(free_before - free_after),
                   "l2": "inputs larger than L2 (weights 245 MB + arena per block)",
                   "input_restore": "device-to-device copy of the block input and temb at the start of every step, "
                                    "inside the timed region (%.3f ms per step)" % restore_ms,
                   "output_finite": out_finite,
                   "parallelism": "replicas x%d" % world},
        "clocks": clocks,
        "regime": regime_of(clocks),
        "sm_mcycles_per_step": (ms_per_step * clocks["sm_mhz"] / 1e3) if clocks.get("sm_mhz") else None,
        # End to end through the C ABI's host-buffer call (xema_forward_host): pinned host -> arena ->
        # pinned host, nothing on the device outside the budgeted arena.  The pipelined
        # figure overlaps the copies of neighbouring steps with compute through staging buffers that
        # are NOT part of the budget, so it is the extra, not the value.
        "e2e": {"value": whole_job_tflops(flops, world, e2e_serial_ms), "unit": UNIT, "ms_per_step": e2e_serial_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "how": "xema_forward_host: pinned host -> arena, forward, arena -> pinned host; the output of a finished "
                       "feed-forward piece is copied out while the next piece runs (plan-owned copy stream)",
                "device_bytes": sess.plan.peak_bytes, "fits_budget": budget is None or sess.plan.peak_bytes <= budget,
                "pipelined": {"value": whole_job_tflops(flops, world, e2e_ms), "ms_per_step": e2e_ms,
                              "how": "BlockSession.run_pipelined: copies of neighbouring steps overlap compute",
                              "staging_bytes_outside_arena": sess.staging_bytes,
                              "device_bytes": sess.plan.peak_bytes + sess.staging_bytes,
                              "fits_budget": budget is None or sess.plan.peak_bytes + sess.staging_bytes <= budget}},
        "gpu_launches": n_kernels * args.steps,
        "roofline": roofline,
        "tensor_ops": tensor_ops_of(per_op),
        "per_op": breakdown,
        # the per-op table comes from a second pass of the same K steps with an event around every op;
        # the timed region of `value` carries events only around each step and the dominant kernel
        "per_op_pass": {"steps": args.steps, "ms_per_step": per_op_total_ms / args.steps, "clocks": per_op_clocks},
        "sustained": sustained,
        "cpu_baseline": cpu,
    }
    if sweep:
        line["by_chunks"] = sweep
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
