"""Bit-exact parity of the library's host planner with the oracle (CPU only)."""
import math

import numpy as np
import pytest

from oracle import arena as o_arena
from oracle import block as o_block
from oracle import trace as o_trace
from paper_2607_11136_b200 import binding as xb
from xema_inputs import template

CASES = [("tiny", 1), ("cogvideox", 1), ("flux", 1), ("flux", 4), ("longvideo", 1), ("longvideo", 2)]


@pytest.mark.parametrize("name,batch", CASES)
def test_trace_offsets_peak_bit_exact(name, batch):
    t = template(name, batch=batch)
    cfg = xb.make_config(t)
    for C in list(range(1, 17)) + [31, 64]:
        want, want_ops = o_trace.trace(t, C)
        got, got_ops = xb.xema_trace(cfg, C)
        assert got_ops == want_ops
        assert got == want, (name, C)
        offs, peak, live = xb.xema_plan_arena(got)
        w_offs, w_peak = o_arena.plan_arena(want)
        assert offs == w_offs and peak == w_peak
        assert live == o_arena.max_live_bytes(want, want_ops)


@pytest.mark.parametrize("C", [1, 2, 3, 4, 8])
def test_step_trace_bit_exact(C):
    t = template("step")
    want, want_ops = o_trace.trace(t, C)
    got, got_ops = xb.xema_trace(xb.make_config(t), C)
    assert (got, got_ops) == (want, want_ops)
    offs, peak, _ = xb.xema_plan_arena(got)
    w_offs, w_peak = o_arena.plan_arena(want)
    assert offs == w_offs and peak == w_peak


def test_plan_object_agrees_with_free_functions():
    t = template("cogvideox")
    cfg = xb.make_config(t)
    p = xb.Plan(cfg, 4)
    ts, n_ops = xb.xema_trace(cfg, 4)
    offs, peak, live = xb.xema_plan_arena(ts)
    assert (p.peak_bytes, p.max_live_bytes, p.n_ops, p.n_tensors, p.chunks) == (peak, live, n_ops, len(ts), 4)
    for d, off in zip(p.tensors(), offs):
        assert d["offset"] == off
        assert p.tensor(d["name"]) == (off, d["bytes"])
    p.close()


def test_plan_arena_on_random_traces():
    rng = np.random.default_rng(5)
    for _ in range(200):
        n = int(rng.integers(1, 40))
        ts = []
        for _ in range(n):
            b = int(rng.integers(0, 30))
            ts.append({"bytes": 256 * int(rng.integers(1, 50)), "birth": b, "death": b + int(rng.integers(1, 12))})
        offs, peak, live = xb.xema_plan_arena(ts)
        w_offs, w_peak = o_arena.plan_arena(ts)
        assert offs == w_offs and peak == w_peak and live == o_arena.max_live_bytes(ts)
        assert o_arena.overlapping_pairs(ts, offs) == []


def test_chunks_for_budget_bit_exact():
    GiB = 1 << 30
    sweeps = [
        ("cogvideox", 1, [764583936, 764583935, 657074688, 657074687, 601613568, 573883136, 560 << 20, 1 << 40]),
        ("flux", 1, [24 * GiB]), ("flux", 4, [24 * GiB, 700 << 20]),
        ("longvideo", 1, [8 * GiB, 16 * GiB, 32 * GiB, 4 * GiB, int(3.5 * GiB), int(3.25 * GiB)]),
        ("longvideo", 2, [8 * GiB, 16 * GiB]), ("longvideo", 4, [8 * GiB, 16 * GiB, 32 * GiB]),
        ("step", 1, [768 << 20, 640 << 20, 576 << 20]),
        ("tiny", 1, [2076672, 1786368, 1561856, 1500000]),
    ]
    for name, batch, budgets in sweeps:
        t = template(name, batch=batch)
        cfg = xb.make_config(t)
        for budget in budgets:
            assert xb.xema_chunks_for_budget(cfg, budget, 16) == o_arena.chunks_for_budget(t, budget, 16), (name, budget)


def test_rope_table_against_oracle_angles():
    for name in ("tiny", "flux"):
        t = template(name)
        tab = xb.xema_rope_table(xb.make_config(t))
        ang = o_block.rope_angles(t)
        assert tab.shape == (t.seq, t.head_dim // 2, 2)
        assert np.array_equal(tab[..., 0], np.cos(ang).astype(np.float32))
        assert np.array_equal(tab[..., 1], np.sin(ang).astype(np.float32))
    # text tokens are left unrotated
    assert np.all(tab[:t.s_text, :, 0] == 1.0) and np.all(tab[:t.s_text, :, 1] == 0.0)


# ---- per-phase chunk counts ---------------------------------------------------------------

PHASE_TRIPLES = [(1, 1, 1), (1, 1, 2), (1, 1, 3), (2, 1, 3), (3, 2, 1), (1, 4, 2), (5, 3, 7), (16, 1, 9)]


@pytest.mark.parametrize("name,batch", CASES + [("step", 1)])
def test_phase_trace_offsets_peak_bit_exact(name, batch):
    t = template(name, batch=batch)
    cfg = xb.make_config(t)
    for counts in PHASE_TRIPLES if name != "step" else PHASE_TRIPLES[:4]:
        want, want_ops = o_trace.trace(t, counts)
        got, got_ops = xb.xema_trace_phases(cfg, counts)
        assert got_ops == want_ops and got == want, (name, counts)
        offs, peak, live = xb.xema_plan_arena(got)
        w_offs, w_peak = o_arena.plan_arena(want)
        assert offs == w_offs and peak == w_peak
        plan = xb.Plan(cfg, counts)
        assert plan.phase_chunks == counts and plan.chunks == max(counts)
        assert plan.peak_bytes == w_peak and plan.n_ops == want_ops
        assert [d["offset"] for d in plan.tensors()] == w_offs
        plan.close()


def test_phase_trace_uniform_equals_trace():
    t = template("cogvideox")
    cfg = xb.make_config(t)
    for C in (1, 2, 5):
        assert xb.xema_trace_phases(cfg, (C, C, C)) == xb.xema_trace(cfg, C)
        a, b = xb.Plan(cfg, C), xb.Plan(cfg, (C, C, C))
        assert (a.peak_bytes, a.n_ops, a.phase_chunks) == (b.peak_bytes, b.n_ops, b.phase_chunks)


def test_phase_trace_rejects_bad_counts():
    t = template("tiny")
    cfg = xb.make_config(t)
    for bad in [(0, 1, 1), (1, -1, 1), (1, 1, t.seq + 1)]:
        with pytest.raises(xb.XemaError) as e:
            xb.xema_trace_phases(cfg, bad)
        assert e.value.status == xb.XEMA_EINVAL
        with pytest.raises(xb.XemaError):
            xb.Plan(cfg, bad)
    got, n_ops = xb.xema_trace_phases(cfg, (t.seq, 1, t.seq))
    assert n_ops == 1 + 3 * t.seq + 5 + 3 * t.seq


def test_phase_chunks_for_budget_bit_exact():
    GiB = 1 << 30
    sweeps = [
        ("cogvideox", 1, [764583936, 764583935, 657074688, 600760320, 600760319, 549565440, 549565439,
                          525 << 20, 1 << 40, 1]),
        ("flux", 1, [24 * GiB, 150 << 20, 142073856, 142073855]), ("flux", 4, [24 * GiB, 700 << 20]),
        ("longvideo", 1, [8 * GiB, 4 * GiB, int(3.5 * GiB), int(3.25 * GiB), 3 * GiB]),
        ("longvideo", 2, [8 * GiB, 16 * GiB]),
        ("step", 1, [768 << 20, 640 << 20, 576 << 20]),
        ("tiny", 1, [2076672, 1786368, 1634304, 1634303, 1496064, 1496063]),
    ]
    for name, batch, budgets in sweeps:
        t = template(name, batch=batch)
        cfg = xb.make_config(t)
        for budget in budgets:
            got = xb.xema_phase_chunks_for_budget(cfg, budget, 16)
            assert got == o_arena.phase_chunks_for_budget(t, budget, 16), (name, budget)
    with pytest.raises(xb.XemaError):
        xb.xema_phase_chunks_for_budget(xb.make_config(template("tiny")), 1 << 30, 0)


def test_alloc_replay_event_order_reproduces_the_live_trace():
    """The allocator replay issues frees before allocations at an op and its running byte count
    equals the oracle's live-byte trace at every op."""
    from paper_2607_11136_b200.alloc_replay import alloc_events, parse_item
    assert parse_item("cogvideox:1,1,2") == ("cogvideox", (1, 1, 2)) and parse_item("flux:3") == ("flux", 3)
    assert parse_item("tiny") == ("tiny", 1)
    t = template("tiny")
    for counts in [(1, 1, 1), (2, 1, 3), (3, 3, 3)]:
        tensors, n_ops = o_trace.trace(t, counts)
        live = o_arena.live_per_op(tensors, n_ops)
        ev = alloc_events(tensors, n_ops)
        assert sorted(i for _, k, i in ev if k == "alloc") == list(range(len(tensors)))
        assert sorted(i for _, k, i in ev if k == "free") == list(range(len(tensors)))
        cur, seen = 0, {}
        for op, kind, i in ev:
            cur += tensors[i]["bytes"] if kind == "alloc" else -tensors[i]["bytes"]
            seen[op] = cur                      # value after the last event of this op
        got, last = [], 0
        for op in range(n_ops):                 # ops without an event keep the running value
            last = seen.get(op, last)
            got.append(last)
        assert got == live and cur == 0


# ---- temporary serialization (sub-batch pieces) ------------------------------------------------

def test_mitigated_trace_and_search_bit_exact():
    cases = [("flux", 4), ("tiny", 3), ("longvideo", 2), ("tiny", 1), ("cogvideox", 1)]
    for name, batch in cases:
        t = template(name, batch=batch)
        cfg = xb.make_config(t)
        for counts, axes in [((1, 1, 2), (0, 0, 1)), ((2, 1, 1), (1, 0, 0)), ((1, 2, 2), (0, 1, 1)),
                             ((2, 2, 2), (1, 1, 1)), ((3, 1, 2), (0, 0, 1)), ((1, 1, 3), (0, 0, 1)), ((2, 3, 4), (0, 0, 0))]:
            if any(c > batch for c, a in zip(counts, axes) if a):
                with pytest.raises(xb.XemaError) as e:
                    xb.xema_trace_mitigated(cfg, counts, axes)
                assert e.value.status == xb.XEMA_EINVAL
                continue
            want, want_ops = o_trace.trace(t, counts, axes)
            got, got_ops = xb.xema_trace_mitigated(cfg, counts, axes)
            assert got_ops == want_ops and got == want, (name, batch, counts, axes)
            plan = xb.Plan(cfg, counts, axes)
            w_offs, w_peak = o_arena.plan_arena(want)
            assert plan.peak_bytes == w_peak and plan.axes == axes and plan.phase_chunks == counts
            assert [d["offset"] for d in plan.tensors()] == w_offs
        p1 = o_arena.plan_arena(o_trace.trace(t, 1)[0])[1]
        for frac in (1.0, 0.9, 0.8, 0.76, 0.74, 0.5):
            budget = int(p1 * frac)
            assert xb.xema_mitigation_for_budget(cfg, budget, 16) == o_arena.mitigation_for_budget(t, budget, 16)
    with pytest.raises(xb.XemaError):
        xb.xema_trace_mitigated(xb.make_config(template("tiny", batch=2)), (1, 1, 2), (0, 0, 5))


def test_pressure_ranges_bit_exact():
    rng = np.random.default_rng(3)
    for _ in range(50):
        n_ops = int(rng.integers(1, 12))
        ts = []
        for _ in range(int(rng.integers(0, 8))):
            b = int(rng.integers(0, n_ops))
            ts.append({"bytes": int(rng.integers(1, 9)) * 256, "birth": b, "death": int(rng.integers(b + 1, n_ops + 1))})
        for budget in (0, 256, 1024, 2048, 1 << 20):
            assert xb.xema_pressure_ranges(ts, n_ops, budget) == o_arena.pressure_ranges(ts, n_ops, budget)
    for name, counts in (("cogvideox", (1, 1, 1)), ("cogvideox", (1, 1, 2)), ("step", (1, 1, 1))):
        t = template(name)
        ts, n_ops = o_trace.trace(t, counts)
        for budget in (640 << 20, 560 << 20, 549565439, 1 << 40, 0):
            assert xb.xema_pressure_ranges(ts, n_ops, budget) == o_arena.pressure_ranges(ts, n_ops, budget)
    with pytest.raises(xb.XemaError):
        xb.xema_pressure_ranges([{"bytes": 256, "birth": 2, "death": 2}], 4, 0)


def test_sharded_trace_and_plan_bit_exact():
    """Sequence-parallel shards: the library's trace, offsets, peak and row ranges equal the
    oracle's for every shard of several shard counts, chunkings and split axes."""
    cases = [("tiny", 1, (1, 1, 1), None), ("tiny", 1, (2, 3, 1), None), ("tiny", 2, (1, 2, 2), (0, 1, 1)),
             ("cogvideox", 1, (1, 1, 2), None), ("flux", 4, (1, 2, 4), (0, 0, 1)), ("step", 1, (1, 1, 2), None)]
    for name, batch, counts, axes in cases:
        t = template(name, batch=batch)
        cfg = xb.make_config(t)
        for P in (1, 2, 3, 8):
            if name == "step" and P not in (2, 8):
                continue
            for p in range(P):
                want, want_ops = o_trace.trace(t, counts, axes or (0, 0, 0), shard=(p, P))
                got, n_ops = xb.xema_trace_sharded(cfg, counts, axes, p, P)
                assert n_ops == want_ops and len(got) == len(want)
                for g, w in zip(got, want):
                    assert all(g[k] == w[k] for k in ("name", "kind", "dtype", "block", "chunk", "bytes", "birth", "death")), (g, w)
                assert xb.xema_shard_rows(cfg, p, P) == o_trace.shard_rows(t, (p, P))
                if name == "step" and p not in (0, P - 1):
                    continue
                pl = xb.Plan(cfg, counts, axes, shard=(p, P))
                w_offs, w_peak = o_arena.plan_arena(want)
                assert [d["offset"] for d in pl.tensors()] == w_offs and pl.peak_bytes == w_peak
                assert pl.max_live_bytes == o_arena.max_live_bytes(want, want_ops)
                assert (pl.shard, (pl.row0, pl.rows)) == ((p, P), o_trace.shard_rows(t, (p, P)))
                ca, cb, cc = counts
                for l in range(t.n_blocks if name != "step" else 2):
                    op, off = pl.gather_point(l)
                    assert op == l * (1 + 3 * ca + 5 * cb + 3 * cc) + 1 + 3 * ca
                    assert off == pl.tensor("kv%d" % l)[0]
                pl.close()
    cfg = xb.make_config(template("tiny"))
    for bad in ((2, 2), (-1, 2), (0, 0), (0, 289)):
        with pytest.raises(xb.XemaError):
            xb.xema_shard_rows(cfg, *bad)
    with pytest.raises(xb.XemaError):
        xb.Plan(cfg, (1, 200, 1), shard=(0, 2))            # more chunks than owned rows (144)
