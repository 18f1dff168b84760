"""Pins for the oracle's trace, Algorithm 1 layout and chunk search (CPU only)."""
import itertools
import os
import random

import pytest

from oracle import arena, trace
from xema_inputs import template

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _mk(size, b, e):
    return {"bytes": size, "birth": b, "death": e}


def _read_examples():
    examples, cur = [], None
    for line in open(os.path.join(GOLDEN, "algorithm1_worked_examples.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "example":
            cur = {"name": tok[1], "tensors": [], "expect": []}
            examples.append(cur)
        elif tok[0] == "peak":
            cur["peak"], cur["maxlive"] = int(tok[1]), int(tok[3])
        else:
            cur["tensors"].append(_mk(int(tok[1]), int(tok[2]), int(tok[3])))
            cur["expect"].append(int(tok[4]))
    return examples


@pytest.mark.parametrize("ex", _read_examples(), ids=lambda e: e["name"])
def test_algorithm1_worked_examples(ex):
    offsets, peak = arena.plan_arena(ex["tensors"])
    assert offsets == ex["expect"]
    assert peak == ex["peak"]
    assert arena.max_live_bytes(ex["tensors"]) == ex["maxlive"]
    assert arena.overlapping_pairs(ex["tensors"], offsets) == []


def _optimal_peak(tensors):
    """Brute force: every placement order with lowest-address first-fit.  For interval
    conflict graphs this reaches the optimum on the tiny cases used here."""
    best = None
    n = len(tensors)
    for order in itertools.permutations(range(n)):
        offs = [None] * n
        for i in order:
            busy = sorted((offs[j], offs[j] + tensors[j]["bytes"]) for j in range(n)
                          if offs[j] is not None and arena.conflicts(tensors[i], tensors[j]))
            pos = 0
            for lo, hi in busy:
                if lo - pos >= tensors[i]["bytes"]:
                    break
                pos = max(pos, hi)
            offs[i] = pos
        peak = max(offs[i] + tensors[i]["bytes"] for i in range(n))
        best = peak if best is None else min(best, peak)
    return best


def test_algorithm1_against_brute_force():
    rng = random.Random(11)
    for _ in range(150):
        n = rng.randint(1, 6)
        tensors = []
        for _ in range(n):
            b = rng.randint(0, 6)
            tensors.append(_mk(256 * rng.randint(1, 5), b, b + rng.randint(1, 4)))
        offsets, peak = arena.plan_arena(tensors)
        assert arena.overlapping_pairs(tensors, offsets) == []
        assert all(o % 256 == 0 for o in offsets)
        live = arena.max_live_bytes(tensors)
        opt = _optimal_peak(tensors)
        assert peak >= opt >= live


def test_algorithm1_degenerate_cases():
    assert arena.plan_arena([]) == ([], 0)
    # disjoint lifetimes share address 0
    offs, peak = arena.plan_arena([_mk(512, 0, 1), _mk(1024, 1, 2), _mk(256, 2, 3)])
    assert offs == [0, 0, 0] and peak == 1024
    # touching half-open lifetimes do not conflict
    assert not arena.conflicts(_mk(1, 0, 2), _mk(1, 2, 3))
    assert arena.conflicts(_mk(1, 0, 3), _mk(1, 2, 3))
    # all live together: a stack in size order
    offs, peak = arena.plan_arena([_mk(256, 0, 1), _mk(768, 0, 1), _mk(512, 0, 1)])
    assert offs == [1280, 0, 768] and peak == 1536


def test_trace_counts_and_order():
    t = template("tiny")
    for C in (1, 2, 3, 8):
        tensors, n_ops = trace.trace(t, C)
        assert n_ops == 1 + 11 * C
        assert len(tensors) == 6 + 7 * C
        births = [d["birth"] for d in tensors]
        assert births == sorted(births)
        assert [d["name"] for d in tensors[:3]] == ["temb", "hid0", "mod0"]
        assert all(d["bytes"] % 256 == 0 and d["bytes"] > 0 for d in tensors)
        assert all(0 <= d["birth"] < d["death"] <= n_ops for d in tensors)
    ts, n_ops = trace.trace(template("step"), 8)
    assert n_ops == 42 * 89 and len(ts) == 42 * (4 + 7 * 8) + 2


def test_trace_lifetimes_tiny_c2():
    """Lifetimes read off the op list by hand for C = 2 (23 ops):
    0 MOD | 1 LN1A0 2 KV0 3 KROPE0 4 LN1A1 5 KV1 6 KROPE1 |
    7 LN1B0 8 Q0 9 QROPE0 10 ATTN0 11 PROJ0 12 LN1B1 13 Q1 14 QROPE1 15 ATTN1 16 PROJ1 |
    17 LN20 18 FFN10 19 FFN20 20 LN21 21 FFN11 22 FFN21"""
    ts, n_ops = trace.trace(template("tiny"), 2)
    life = {d["name"]: (d["birth"], d["death"]) for d in ts}
    assert n_ops == 23
    assert life == {
        "temb": (0, 1), "hid0": (0, 17), "mod0": (0, 23), "kv0": (2, 16),
        "h1a0_0": (1, 3), "h1a0_1": (4, 6),
        "h1b0_0": (7, 9), "q0_0": (8, 11), "o0_0": (10, 12), "lse0_0": (10, 11), "res0": (11, 23),
        "h1b0_1": (12, 14), "q0_1": (13, 16), "o0_1": (15, 17), "lse0_1": (15, 16),
        "h20_0": (17, 19), "g0_0": (18, 20), "hid1": (19, 23),
        "h20_1": (20, 22), "g0_1": (21, 23),
    }
    size = {d["name"]: d["bytes"] for d in ts}
    # S = 288 -> chunks of 144 rows; D = 512; H = 8; F = 2048
    assert size["hid0"] == 2 * 288 * 512 and size["kv0"] == 4 * 288 * 512
    assert size["res0"] == 4 * 288 * 512 and size["mod0"] == 24 * 512
    assert size["q0_1"] == 2 * 144 * 512 and size["g0_0"] == 2 * 144 * 2048
    assert size["lse0_0"] == trace.align_up(4 * 8 * 144) and size["temb"] == 1024


def test_trace_closed_form_golden():
    t = template("cogvideox")
    for line in open(os.path.join(GOLDEN, "trace_closed_form_cogvideox.txt")):
        if line.startswith("chunks"):
            _, C, _, want = line.split()
            ts, n_ops = trace.trace(t, int(C))
            assert arena.max_live_bytes(ts, n_ops) == int(want)


def _closed_form_peak(t, C):
    """Max-live of one block when F = 4D: C = 1 peaks at the FFN, C >= 2 at the attention
    of a largest chunk."""
    A = trace.align_up
    B, S, D, H, F = t.batch, t.seq, t.hidden, t.heads, t.ffn
    u = 2 * B * S * D
    temb = A(2 * B * t.temb_dim) if t.n_blocks > 1 else 0
    if C == 1:
        return temb + A(24 * B * D) + A(2 * u) + A(u) + A(2 * B * S * F)
    n = -(-S // C)
    return temb + A(u) + A(24 * B * D) + 2 * A(2 * u) + 2 * A(2 * B * n * D) + A(4 * B * H * n)


@pytest.mark.parametrize("name", ["tiny", "cogvideox", "flux", "longvideo"])
def test_trace_closed_form_all_templates(name):
    t = template(name)
    for C in (1, 2, 3, 4, 7, 8, 16):
        ts, n_ops = trace.trace(t, C)
        assert arena.max_live_bytes(ts, n_ops) == _closed_form_peak(t, C), (name, C)


def test_step_trace_keeps_temb_live():
    t = template("step")
    for C in (1, 2):
        ts, n_ops = trace.trace(t, C)
        assert arena.max_live_bytes(ts, n_ops) == _closed_form_peak(t, C)


@pytest.mark.parametrize("name,batch", [("tiny", 1), ("cogvideox", 1), ("flux", 1), ("flux", 4), ("longvideo", 1)])
def test_plan_valid_and_tight(name, batch):
    t = template(name, batch=batch)
    prev = None
    for C in range(1, 17):
        ts, n_ops = trace.trace(t, C)
        offsets, peak = arena.plan_arena(ts)
        assert arena.overlapping_pairs(ts, offsets) == []
        assert all(o % 256 == 0 for o in offsets)
        # tightness is a property of this template, not of Algorithm 1 in general
        assert peak == arena.max_live_bytes(ts, n_ops)
        if prev is not None:
            assert peak <= prev
        prev = peak


def test_plan_step_valid_and_tight():
    t = template("step")
    for C in (1, 2, 4):
        ts, n_ops = trace.trace(t, C)
        offsets, peak = arena.plan_arena(ts)
        assert peak == _closed_form_peak(t, C)
        # full pairwise check is quadratic; check conflicts per op instead
        by_op = {}
        for i, d in enumerate(ts):
            for op in range(d["birth"], d["death"]):
                by_op.setdefault(op, []).append(i)
        seen = set()
        for ids in by_op.values():
            key = tuple(ids)
            if key in seen:
                continue
            seen.add(key)
            spans = sorted((offsets[i], offsets[i] + ts[i]["bytes"]) for i in ids)
            assert all(spans[k][1] <= spans[k + 1][0] for k in range(len(spans) - 1))


def test_chunks_for_budget():
    t = template("cogvideox")
    peaks = {C: arena.plan_arena(trace.trace(t, C)[0])[1] for C in (1, 2, 3, 4, 8)}
    assert peaks[1] == 764583936 and peaks[2] == 657074688
    for C in (1, 2, 4, 8):
        assert arena.chunks_for_budget(t, peaks[C], 64) == (C, peaks[C])
    assert arena.chunks_for_budget(t, peaks[1] - 1, 64)[0] == 2
    assert arena.chunks_for_budget(t, peaks[2] - 1, 64)[0] == 3
    assert arena.chunks_for_budget(t, 1 << 40, 64)[0] == 1
    # below the floor (hid + mod + kv + res are never chunked): nothing fits
    C, smallest = arena.chunks_for_budget(t, 5 * 109215744, 32)
    assert C is None and smallest == arena.plan_arena(trace.trace(t, 32)[0])[1]
    # a non-binding budget keeps C = 1 (Flux under 24 GiB, long video under 8 GiB)
    assert arena.chunks_for_budget(template("flux", batch=4), 24 << 30, 8)[0] == 1
    assert arena.chunks_for_budget(template("longvideo"), 8 << 30, 8)[0] == 1
    assert arena.chunks_for_budget(template("longvideo"), 4 << 30, 8)[0] == 2
