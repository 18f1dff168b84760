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


def test_overlap_checker_reports_hand_made_collisions():
    """Negative control for the validity checker behind every "no overlaps" assertion: layouts
    written by hand with known collisions must come back with exactly the offending pairs."""
    ts = [_mk(1024, 0, 4), _mk(512, 0, 2), _mk(512, 1, 4), _mk(256, 2, 4)]
    good = [0, 1024, 1536, 1024]                 # worked example (i): D reuses B's hole
    assert arena.overlapping_pairs(ts, good) == []
    # D moved up to 1536: it now shares [1536, 1792) with C, which is live with it
    assert arena.overlapping_pairs(ts, [0, 1024, 1536, 1536]) == [(2, 3)]
    # B placed inside A while both are live; C one byte into A's last byte; D alone is fine
    assert arena.overlapping_pairs(ts, [0, 512, 1023, 2048]) == [(0, 1), (0, 2), (1, 2)]
    # same addresses, lifetimes that only touch ([0,2) then [2,4)) are no collision ...
    assert arena.overlapping_pairs([_mk(512, 0, 2), _mk(512, 2, 4)], [0, 0]) == []
    # ... one op of common life is
    assert arena.overlapping_pairs([_mk(512, 0, 3), _mk(512, 2, 4)], [0, 0]) == [(0, 1)]
    # address ranges that only touch ([0,512) and [512,768)) are no collision; one byte less is
    assert arena.overlapping_pairs([_mk(512, 0, 3), _mk(256, 0, 3)], [0, 512]) == []
    assert arena.overlapping_pairs([_mk(512, 0, 3), _mk(256, 0, 3)], [0, 511]) == [(0, 1)]
    # a tensor wholly inside another, and the order of the pair does not matter
    assert arena.overlapping_pairs([_mk(256, 1, 2), _mk(2048, 0, 5)], [512, 0]) == [(0, 1)]
    # a corrupted Algorithm 1 result is caught: shift one offset of a real plan onto a neighbour
    t = template("tiny")
    tensors, _ = trace.trace(t, 2)
    offsets, _ = arena.plan_arena(tensors)
    assert arena.overlapping_pairs(tensors, offsets) == []
    hit = 0
    for i in range(len(tensors)):
        for j in range(len(tensors)):
            if i != j and arena.conflicts(tensors[i], tensors[j]):
                moved = list(offsets)
                moved[i] = offsets[j]
                pairs = arena.overlapping_pairs(tensors, moved)
                assert (min(i, j), max(i, j)) in pairs
                hit += 1
    assert hit > 50


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


# ---- per-phase chunk counts ("Applying Mitigation Only Where Needed") ---------------------

def _closed_form_phase_live(t, counts):
    """Largest live-byte sum inside each phase of a single block, written out per op from the
    block's data flow (not from the recorder): which full-size tensors exist at that point
    plus the chunk-sized ones of the largest chunk."""
    A = trace.align_up
    B, S, D, H, F = t.batch, t.seq, t.hidden, t.heads, t.ffn
    ca, cb, cc = counts
    u, mod, kv, res = A(2 * B * S * D), A(24 * B * D), A(4 * B * S * D), A(4 * B * S * D)
    big = lambda C: -(-S // C)
    ck = lambda n, w: A(2 * B * n * w)
    # phase A peaks at a KV op: block input, modulation, the K/V tensor, the LN output chunk
    pa = max(A(2 * B * t.temb_dim) + u + mod, u + mod + kv + ck(big(ca), D))
    # phase B: ATTN holds q, o and lse of the chunk; res exists from the first PROJ on
    n = big(cb)
    attn = u + mod + kv + 2 * ck(n, D) + A(4 * B * H * n)
    if cb == 1:
        pb = max(attn, u + mod + ck(n, D) + res)
    else:
        pb = attn + res
    # phase C: FFN1 holds the LN output and the GELU output of the chunk; the next hidden
    # state exists from the first FFN2 on
    n = big(cc)
    if cc == 1:
        pc = mod + res + max(ck(n, D) + ck(n, F), ck(n, F) + u)
    else:
        pc = mod + res + u + ck(n, D) + ck(n, F)
    return pa, pb, pc


@pytest.mark.parametrize("name", ["tiny", "cogvideox", "flux", "longvideo"])
def test_phase_trace_closed_form(name):
    t = template(name)
    for counts in [(1, 1, 1), (1, 1, 2), (1, 1, 3), (2, 1, 1), (1, 2, 1), (3, 2, 5), (4, 4, 4), (2, 7, 3)]:
        ts, n_ops = trace.trace(t, counts)
        assert n_ops == 1 + 3 * counts[0] + 5 * counts[1] + 3 * counts[2]
        live = arena.live_per_op(ts, n_ops)
        got = [0, 0, 0]
        for op, b in enumerate(live):
            ph = arena.phase_of_op(t, counts, op)
            got[ph] = max(got[ph], b)
        assert tuple(got) == _closed_form_phase_live(t, counts), (name, counts)
        assert max(got) == arena.max_live_bytes(ts, n_ops)


def test_phase_trace_reduces_to_uniform():
    for name in ("tiny", "step"):
        t = template(name)
        for C in (1, 2, 3):
            assert trace.trace(t, (C, C, C)) == trace.trace(t, C)


def test_phase_trace_lifetimes_tiny():
    """(C_A, C_B, C_C) = (2, 1, 3) on the tiny template, op by op:
    0 MOD | 1 LN1A_0 2 KV_0 3 KROPE_0 4 LN1A_1 5 KV_1 6 KROPE_1 | 7 LN1B 8 Q 9 QROPE 10 ATTN
    11 PROJ | 12 LN2_0 13 FFN1_0 14 FFN2_0 15 LN2_1 16 FFN1_1 17 FFN2_1 18 LN2_2 19 FFN1_2
    20 FFN2_2."""
    t = template("tiny")
    ts, n_ops = trace.trace(t, (2, 1, 3))
    assert n_ops == 21
    life = {d["name"]: (d["birth"], d["death"]) for d in ts}
    assert life == {
        "temb": (0, 1), "hid0": (0, 12), "mod0": (0, 21),
        "h1a0_0": (1, 3), "kv0": (2, 11), "h1a0_1": (4, 6),
        "h1b0_0": (7, 9), "q0_0": (8, 11), "o0_0": (10, 12), "lse0_0": (10, 11), "res0": (11, 21),
        "h20_0": (12, 14), "g0_0": (13, 15), "hid1": (14, 21),
        "h20_1": (15, 17), "g0_1": (16, 18), "h20_2": (18, 20), "g0_2": (19, 21),
    }
    S = t.seq
    rows = {d["name"]: d["bytes"] for d in ts}
    assert rows["h1a0_0"] == trace.align_up(2 * t.batch * (S // 2) * t.hidden)
    assert rows["g0_1"] == trace.align_up(2 * t.batch * (2 * S // 3 - S // 3) * t.ffn)


@pytest.mark.parametrize("name", ["tiny", "cogvideox"])
def test_phase_plan_valid_and_tight(name):
    t = template(name)
    for counts in itertools.product((1, 2, 3), repeat=3):
        ts, n_ops = trace.trace(t, counts)
        offsets, peak = arena.plan_arena(ts)
        assert arena.overlapping_pairs(ts, offsets) == []
        assert peak == arena.max_live_bytes(ts, n_ops)


@pytest.mark.parametrize("name", ["tiny", "cogvideox", "flux"])
def test_phase_chunks_for_budget_is_minimal(name):
    """The search result fits, and no triple with a smaller total chunk count does (brute
    force over all triples up to 4 per phase)."""
    t = template(name)
    peaks = {c: arena.plan_arena(trace.trace(t, c)[0])[1] for c in itertools.product((1, 2, 3, 4), repeat=3)}
    p1 = peaks[(1, 1, 1)]
    for frac in (1.0, 0.95, 0.85, 0.79, 0.75, 0.73):
        budget = int(p1 * frac)
        counts, peak = arena.phase_chunks_for_budget(t, budget, 4)
        feasible = [c for c, p in peaks.items() if p <= budget]
        assert counts is not None and peak == peaks[counts] and peak <= budget
        assert sum(counts) == min(sum(c) for c in feasible), (name, frac, counts)
    # chunking the attention phase never helps: its floor is the unchunked attention peak
    assert min(peaks[(a, b, c)] for a, b, c in peaks if b > 1) > min(peaks.values())


def test_phase_chunks_for_budget_values():
    t = template("cogvideox")
    MiB = 1 << 20
    assert arena.phase_chunks_for_budget(t, 768 * MiB, 16) == ((1, 1, 1), 764583936)
    # 640 MiB: one count for the whole block needs C = 2 and reserves 657 074 688 bytes;
    # chunking the feed-forward phase alone reserves less with 3 fewer launches
    assert arena.chunks_for_budget(t, 640 * MiB, 16) == (2, 657074688)
    assert arena.phase_chunks_for_budget(t, 640 * MiB, 16) == ((1, 1, 2), 600760320)
    assert arena.phase_chunks_for_budget(t, 576 * MiB, 16) == ((1, 1, 2), 600760320)
    assert arena.phase_chunks_for_budget(t, 560 * MiB, 16) == ((1, 1, 3), 549565440)
    # 525 MiB is below every uniform plan up to 16 chunks but (1, 1, 3) fits
    assert arena.chunks_for_budget(t, 525 * MiB, 16)[0] is None
    assert arena.phase_chunks_for_budget(t, 525 * MiB, 16) == ((1, 1, 3), 549565440)
    # the floor: block input, K/V, q, o and lse of the unchunked attention
    assert arena.phase_chunks_for_budget(t, 549565440 - 1, 16)[0] is None
    # non-binding budgets stay unchunked
    assert arena.phase_chunks_for_budget(template("longvideo"), 8 << 30, 8)[0] == (1, 1, 1)
    assert arena.phase_chunks_for_budget(template("longvideo"), 4 << 30, 8)[0] == (1, 1, 2)
    # the 42-block step: same counts as one block (the budget binds inside a block)
    assert arena.phase_chunks_for_budget(template("step"), 640 * MiB, 16)[0] == (1, 1, 2)


# ---- temporary serialization: a phase split into sub-batches instead of row chunks -----------

def test_batch_split_trace_sizes_and_lifetimes():
    """Lifetimes do not depend on the split axis; piece sizes do: a sub-batch piece holds whole
    batch elements (all S rows), a row chunk holds all B elements of its rows."""
    t = template("tiny", batch=4)
    S, D, F, H = t.seq, t.hidden, t.ffn, t.heads
    rows, n_ops = trace.trace(t, (2, 2, 4))
    sub, n_ops2 = trace.trace(t, (2, 2, 4), (1, 1, 1))
    assert n_ops == n_ops2 and [(d["name"], d["birth"], d["death"]) for d in rows] == \
        [(d["name"], d["birth"], d["death"]) for d in sub]
    size = {d["name"]: d["bytes"] for d in sub}
    A = trace.align_up
    assert size["h1a0_0"] == size["q0_1"] == A(2 * 2 * S * D)          # 2 of 4 batch elements
    assert size["lse0_0"] == A(4 * 2 * H * S)
    assert size["g0_3"] == A(2 * 1 * S * F) and size["h20_0"] == A(2 * 1 * S * D)
    # 3 sub-batches of 4 elements: pieces of 1, 1, 2 elements
    sizes3 = [d["bytes"] for d in trace.trace(t, (1, 1, 3), (0, 0, 1))[0] if d["name"].startswith("g0_")]
    assert sizes3 == [A(2 * S * F), A(2 * S * F), A(2 * 2 * S * F)]
    # the same fraction along either axis gives the same piece size when both divide evenly
    assert {d["name"]: d["bytes"] for d in trace.trace(t, (2, 2, 2))[0]} == \
        {d["name"]: d["bytes"] for d in trace.trace(t, (2, 2, 2), (1, 1, 1))[0]}
    for bad in [((5, 1, 1), (1, 0, 0)), ((1, 1, 2), (0, 0, 2))]:
        with pytest.raises(ValueError):
            trace.trace(t, *bad)
    with pytest.raises(ValueError):
        trace.trace(template("tiny"), (1, 1, 2), (0, 0, 1))             # B = 1 cannot be serialized


def test_mitigation_for_budget_serializes_where_the_batch_allows():
    t = template("flux", batch=4)
    p1 = arena.plan_arena(trace.trace(t, 1)[0])[1]
    assert arena.mitigation_for_budget(t, p1, 16) == ((1, 1, 1), (0, 0, 0), p1)
    counts, axes, peak = arena.mitigation_for_budget(t, int(0.9 * p1), 16)
    assert (counts, axes) == ((1, 1, 2), (0, 0, 1)) and peak == arena.phase_chunks_for_budget(t, int(0.9 * p1), 16)[1]
    # three sub-batches of four elements still hold two elements in one piece: serialization
    # needs four pieces where row chunking needs three
    counts, axes, peak = arena.mitigation_for_budget(t, int(0.76 * p1), 16)
    assert (counts, axes) == ((1, 1, 4), (0, 0, 1))
    assert arena.phase_chunks_for_budget(t, int(0.76 * p1), 16) == ((1, 1, 3), peak)
    # beyond B pieces the search falls back to row chunks
    t2 = template("longvideo", batch=2)
    p1 = arena.plan_arena(trace.trace(t2, 1)[0])[1]
    assert arena.mitigation_for_budget(t2, int(0.9 * p1), 16)[:2] == ((1, 1, 2), (0, 0, 1))
    assert arena.mitigation_for_budget(t2, int(0.74 * p1), 16)[:2] == ((1, 1, 3), (0, 0, 0))
    # B = 1: identical to the per-phase search
    t1 = template("cogvideox")
    assert arena.mitigation_for_budget(t1, 640 << 20, 16) == ((1, 1, 2), (0, 0, 0), 600760320)
    # every plan the search returns is valid and tight on these templates
    for tt, frac in ((t, 0.9), (t, 0.76), (t2, 0.9)):
        p = arena.plan_arena(trace.trace(tt, 1)[0])[1]
        counts, axes, peak = arena.mitigation_for_budget(tt, int(frac * p), 16)
        ts, n_ops = trace.trace(tt, counts, axes)
        offs, pk = arena.plan_arena(ts)
        assert pk == peak == arena.max_live_bytes(ts, n_ops) and arena.overlapping_pairs(ts, offs) == []


def test_pressure_ranges():
    """Where the live bytes exceed the budget, as maximal op ranges."""
    mk = lambda size, b, e: {"bytes": size, "birth": b, "death": e}
    ts = [mk(4, 0, 6), mk(3, 1, 3), mk(2, 2, 5), mk(5, 4, 6)]      # live per op: 4 7 9 6 11 9
    assert arena.live_per_op(ts, 6) == [4, 7, 9, 6, 11, 9]
    assert arena.pressure_ranges(ts, 6, 11) == []
    assert arena.pressure_ranges(ts, 6, 8) == [(2, 3), (4, 6)]
    assert arena.pressure_ranges(ts, 6, 6) == [(1, 3), (4, 6)]
    assert arena.pressure_ranges(ts, 6, 3) == [(0, 6)]
    # CogVideoX-shaped block, unchunked, 640 MiB: only the two feed-forward GEMMs are over
    t = template("cogvideox")
    tensors, n_ops = trace.trace(t, 1)
    assert arena.pressure_ranges(tensors, n_ops, 640 << 20) == [(10, 12)]
    # with the feed-forward phase in two chunks nothing is over; at 560 MiB only FFN1 of the second
    # chunk is (the next hidden state exists by then, during the first chunk it does not)
    tensors, n_ops = trace.trace(t, (1, 1, 2))
    assert arena.pressure_ranges(tensors, n_ops, 640 << 20) == []
    assert arena.pressure_ranges(tensors, n_ops, 560 << 20) == [(13, 14)]
    # one byte below the attention peak the attention op joins the set
    assert arena.pressure_ranges(tensors, n_ops, 549565440 - 1) == [(7, 8), (13, 14)]


# ---- sequence-parallel shards (the paper's SP: the latent sequence split across GPUs) -----------

def test_shard_rows_partition_the_sequence():
    for name in ("tiny", "cogvideox", "longvideo"):
        t = template(name)
        for P in (1, 2, 3, 4, 7, 8):
            cuts = [trace.shard_rows(t, (p, P)) for p in range(P)]
            assert cuts[0][0] == 0 and cuts[-1][0] + cuts[-1][1] == t.seq
            assert all(cuts[p][0] + cuts[p][1] == cuts[p + 1][0] for p in range(P - 1))
            assert max(n for _, n in cuts) - min(n for _, n in cuts) <= 1
    with pytest.raises(ValueError):
        trace.shard_rows(template("tiny"), (2, 2))
    with pytest.raises(ValueError):
        trace.trace(template("tiny"), 1, shard=(0, 289))       # more shards than rows


def test_one_shard_is_the_unsharded_trace():
    t = template("tiny")
    for counts in (1, 3, (1, 2, 3)):
        assert trace.trace(t, counts, shard=(0, 1)) == trace.trace(t, counts)


def test_sharded_trace_keeps_lifetimes_and_splits_row_local_bytes():
    """Same ops and lifetimes as the unsharded trace; `kv`, `mod` and `temb` keep their size; every
    other tensor holds the owned rows only, so over the shards the row-local bytes add up to the
    unsharded ones (hidden width 3072: a row is a multiple of 256 bytes, nothing is lost to the
    rounding of sizes)."""
    t = template("cogvideox")
    full, n_ops = trace.trace(t, (1, 1, 1))
    by_name = {d["name"]: d for d in full}
    for P in (2, 3, 8):
        total = {}
        for p in range(P):
            ts, n = trace.trace(t, (1, 1, 1), shard=(p, P))
            assert n == n_ops and [d["name"] for d in ts] == [d["name"] for d in full]
            for d in ts:
                f = by_name[d["name"]]
                assert (d["birth"], d["death"], d["kind"], d["dtype"]) == (f["birth"], f["death"], f["kind"], f["dtype"])
                if d["name"] in ("kv0", "mod0", "temb"):
                    assert d["bytes"] == f["bytes"]
                total[d["name"]] = total.get(d["name"], 0) + d["bytes"]
        for name in ("hid0", "hid1", "res0", "h1a0_0", "h1b0_0", "q0_0", "o0_0", "h20_0", "g0_0"):
            assert total[name] == by_name[name]["bytes"], name


def test_sharded_peak_closed_form():
    """One block, every phase in one piece, P >= 2 shards of the CogVideoX-shaped template: the
    peak is at the attention (own hidden rows, modulation, ALL keys and values, own q, o, lse);
    the feed-forward phase, which sets the unsharded peak, shrinks with the shard.
    Hand check, shard 1 of 4 (4444 rows): 3 x 27 303 936 + 73 728 + 218 431 488 + 853 248."""
    t = template("cogvideox")
    A = trace.align_up
    B, S, D, H = t.batch, t.seq, t.hidden, t.heads
    ts, n_ops = trace.trace(t, (1, 1, 1), shard=(1, 4))
    assert arena.max_live_bytes(ts, n_ops) == 301270272
    for P in (2, 4, 8):
        for p in range(P):
            _, n = trace.shard_rows(t, (p, P))
            ts, n_ops = trace.trace(t, (1, 1, 1), shard=(p, P))
            want = 3 * A(2 * B * n * D) + A(24 * B * D) + A(4 * B * S * D) + A(4 * B * H * n)
            ffn = A(24 * B * D) + A(4 * B * n * D) + A(2 * B * n * D) + A(2 * B * n * t.ffn)
            assert want > ffn
            assert arena.max_live_bytes(ts, n_ops) == want
            # Algorithm 1 is a heuristic: with two shards it leaves a hole under the full-size kv
            # (reserved 436 936 704 against 384 035 328 live); from four shards on it is tight
            offsets, peak = arena.plan_arena(ts)
            assert arena.overlapping_pairs(ts, offsets) == []
            assert peak == (436936704 if P == 2 else want) >= want
    # chunks cut the owned rows: chunk sizes of shard 2 of 3 with C = 2 (5926 owned rows)
    r0, n = trace.shard_rows(t, (2, 3))
    assert (r0, n) == (11850, 5926)
    ts, _ = trace.trace(t, (1, 2, 1), shard=(2, 3))
    q = {d["name"]: d["bytes"] for d in ts}
    assert q["q0_0"] == A(2 * 2963 * D) and q["q0_1"] == A(2 * 2963 * D) and q["kv0"] == A(4 * S * D)
