"""The N > 1 path of bench.py shards nothing and exchanges nothing on the data path: every rank
runs a replica, the ranks meet at a barrier and the slowest rank's time is used.  That host
logic is exercised here with two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    out[rank] = (ms, bench.whole_job_tflops(1e12, world, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, tflops = res[0]
    assert ms == 15.0
    assert abs(tflops - 2 * 1e12 / 15e-3 / 1e12) < 1e-9


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    from xema_inputs import template
    t = template("cogvideox")
    assert abs(bench.block_flops(t) - 7.910e12) / 7.910e12 < 1e-3
    assert bench.attention_traffic_bytes(t, 2222) == 266.6e6


def test_reference_arm_runs_on_rank_zero_only():
    """Under torchrun the reference arm is printed by rank 0 alone; every other rank exits 0
    without output and without work."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def _sp_worker(rank, world, port, out):
    """One rank of a sequence-parallel pair: plans its own shard (host code only), takes part in
    the exchange of keys and values on a CPU stand-in for the kv tensor, and reports what it
    ended up with."""
    sys.path.insert(0, ROOT)
    from paper_2607_11136_b200 import binding as xb
    from paper_2607_11136_b200.session import all_gather_rows
    from xema_inputs import template
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    t = template("tiny", batch=2)
    cfg = xb.make_config(t)
    plan = xb.Plan(cfg, (1, 2, 1), shard=(rank, world))
    mine = (plan.row0, plan.rows)
    ranges = [None] * world
    dist.all_gather_object(ranges, mine)
    points = [None] * world
    dist.all_gather_object(points, (plan.gather_point(0)[0], plan.tensor("kv0")[1], plan.n_ops))
    # the kv tensor of block 0, [B, S, 2D]: this rank fills its own rows with (rank, batch, row, column)
    S, W = t.seq, 2 * t.hidden
    kv = torch.full((t.batch, S, W), -1, dtype=torch.int32)
    r0, n = mine
    b_idx = torch.arange(t.batch).view(-1, 1, 1)
    r_idx = torch.arange(r0, r0 + n).view(1, -1, 1)
    c_idx = torch.arange(W).view(1, 1, -1)
    kv[:, r0:r0 + n] = (rank << 28) + (b_idx << 24) + (r_idx << 12) + c_idx
    all_gather_rows(kv, ranges)
    owner = torch.empty(S, dtype=torch.int64)
    for r, (q0, qn) in enumerate(ranges):
        owner[q0:q0 + qn] = r
    want = (owner.view(1, -1, 1) << 28) + (b_idx << 24) + (torch.arange(S).view(1, -1, 1) << 12) + c_idx
    out[rank] = {"ranges": ranges, "points": points, "gathered_ok": bool(torch.equal(kv.long(), want)),
                 "peak": plan.peak_bytes, "hid_bytes": plan.tensor("hid0")[1]}
    dist.barrier()
    dist.destroy_process_group()


def test_sequence_parallel_pair_plans_and_exchanges():
    """Two gloo ranks as a sequence-parallel pair: their row ranges partition the sequence, both
    see the same gather point and the same full-size kv tensor, and after the exchange every rank
    holds every row of every batch element exactly where the owner wrote it."""
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_sp_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0]["ranges"] == res[1]["ranges"] == [(0, 144), (144, 144)]
    assert res[0]["points"] == res[1]["points"] and res[0]["points"][0] == res[0]["points"][1]
    first_op, kv_bytes, n_ops = res[0]["points"][0]
    assert (first_op, n_ops) == (4, 17) and kv_bytes == 2 * 2 * 288 * 2 * 512      # kv stays full-size: B*S*2D bf16
    assert res[0]["gathered_ok"] and res[1]["gathered_ok"]
    assert res[0]["hid_bytes"] == res[1]["hid_bytes"] == 2 * 2 * 144 * 512         # the hidden state is the owned rows
    assert res[0]["peak"] == res[1]["peak"]
