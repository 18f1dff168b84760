"""Offline static layout (Algorithm 1 of the paper) and the chunk-count search
(test infrastructure only).

Algorithm 1: visit tensors in descending size; for each, collect the already
placed tensors whose lifetimes intersect its own, look at the address gaps those
leave, take the smallest gap that holds the tensor, and otherwise place it above
all of them.  Points the paper leaves open, fixed here:

  * equal sizes are visited by (birth, death, id) ascending;
  * lifetimes are half-open, [b_i, e_i) and [b_j, e_j) conflict iff
    b_i < e_j and b_j < e_i;
  * a gap is a finite hole between conflicting tensors in address order,
    including the one that starts at address 0; equal-sized holes resolve to the
    lowest address; the unbounded space above the highest conflict is not a gap
    but the fallback position.

Chunk search ("apply only as much mitigation as needed" with chunk count as the
intensity): the smallest C in 1..max_chunks whose laid-out (reserved) peak is
within the byte budget, found by a linear scan so no monotonicity is assumed.
"""
from __future__ import annotations

from . import trace as _trace


def conflicts(a, b):
    return a["birth"] < b["death"] and b["birth"] < a["death"]


def max_live_bytes(tensors, n_ops=None):
    """max over op index t of the bytes of tensors with birth <= t < death."""
    if not tensors:
        return 0
    n_ops = max(d["death"] for d in tensors) if n_ops is None else n_ops
    best = 0
    for t in range(n_ops):
        live = sum(d["bytes"] for d in tensors if d["birth"] <= t < d["death"])
        best = max(best, live)
    return best


def plan_arena(tensors):
    """Returns (offsets, peak).  offsets[i] belongs to tensors[i]."""
    n = len(tensors)
    order = sorted(range(n), key=lambda i: (-tensors[i]["bytes"], tensors[i]["birth"], tensors[i]["death"], i))
    offsets = [None] * n
    placed = []
    for i in order:
        ti = tensors[i]
        O = [j for j in placed if conflicts(ti, tensors[j])]
        O.sort(key=lambda j: (offsets[j], j))
        cursor = 0
        best = None                      # (gap size, bottom address)
        for j in O:
            if offsets[j] > cursor:
                gap = offsets[j] - cursor
                if gap >= ti["bytes"] and (best is None or gap < best[0]):
                    best = (gap, cursor)
            cursor = max(cursor, offsets[j] + tensors[j]["bytes"])
        offsets[i] = best[1] if best is not None else cursor
        placed.append(i)
    peak = max((offsets[i] + tensors[i]["bytes"] for i in range(n)), default=0)
    return offsets, peak


def overlapping_pairs(tensors, offsets):
    """All pairs that are live together and share an address -- must be empty."""
    bad = []
    for i in range(len(tensors)):
        for j in range(i + 1, len(tensors)):
            if conflicts(tensors[i], tensors[j]):
                a0, a1 = offsets[i], offsets[i] + tensors[i]["bytes"]
                b0, b1 = offsets[j], offsets[j] + tensors[j]["bytes"]
                if a0 < b1 and b0 < a1:
                    bad.append((i, j))
    return bad


def phase_of_op(t, counts, op):
    """0 / 1 / 2 for an op of the key-value / attention / feed-forward phase of its block; the
    MOD op belongs to phase 0."""
    ca, cb, cc = counts
    per_block = 1 + 3 * ca + 5 * cb + 3 * cc
    k = op % per_block
    if k < 1 + 3 * ca:
        return 0
    if k < 1 + 3 * ca + 5 * cb:
        return 1
    return 2


def live_per_op(tensors, n_ops):
    """Active-memory trace: bytes of the tensors live at every op."""
    out = [0] * n_ops
    for d in tensors:
        for op in range(d["birth"], d["death"]):
            out[op] += d["bytes"]
    return out


def pressure_ranges(tensors, n_ops, budget_bytes):
    """The memory-pressure set as maximal half-open op ranges [first, end) in which the
    active-memory trace exceeds the budget (the planner's step "locate where memory exceeds the
    budget": mitigation is applied to these ranges only)."""
    live = live_per_op(tensors, n_ops)
    out, start = [], None
    for op, b in enumerate(live):
        if b > budget_bytes and start is None:
            start = op
        if b <= budget_bytes and start is not None:
            out.append((start, op))
            start = None
    if start is not None:
        out.append((start, n_ops))
    return out


def phase_chunks_for_budget(t, budget_bytes, max_chunks):
    """Mitigation only where it is needed (the planner's stage "locating where memory exceeds
    the budget", with chunking as the mitigation): start unchunked; mark the phases in which
    the active-memory trace exceeds the budget at some op; raise the chunk count of exactly
    those phases by one; repeat until no phase is over.  The trace is then laid out; should the
    reserved peak still exceed the budget (Algorithm 1 is a heuristic), the phase holding the
    op with the most live bytes is raised as well.  Returns ((C_A, C_B, C_C), reserved peak),
    or (None, smallest reserved peak seen) when a phase would need more than max_chunks.
    (The per-op reserved memory is no guide here: the longest-lived tensors sit at the top of
    the arena, so every op reaches the peak address.)"""
    counts = [1, 1, 1]
    smallest = None
    limit = min(max_chunks, t.seq)
    while True:
        tensors, n_ops = _trace.trace(t, tuple(counts))
        _, peak = plan_arena(tensors)
        smallest = peak if smallest is None else min(smallest, peak)
        live = live_per_op(tensors, n_ops)
        over = {phase_of_op(t, counts, op) for op, b in enumerate(live) if b > budget_bytes}
        if not over:
            if peak <= budget_bytes:
                return tuple(counts), peak
            over = {phase_of_op(t, counts, max(range(n_ops), key=lambda op: (live[op], -op)))}
        for ph in sorted(over):
            counts[ph] += 1
            if counts[ph] > limit:
                return None, smallest


def serialization_axes(t, counts):
    """Temporary serialization where the batch allows it: a phase split C > 1 ways is split into
    sub-batches when C <= B, into row chunks otherwise (and when it is not split at all)."""
    return tuple(_trace.SPLIT_BATCH if 1 < c <= t.batch else _trace.SPLIT_ROWS for c in counts)


def mitigation_for_budget(t, budget_bytes, max_chunks):
    """phase_chunks_for_budget with the split axis chosen by serialization_axes at every step.
    Returns ((C_A, C_B, C_C), axes, reserved peak) or (None, None, smallest reserved peak seen)."""
    counts = [1, 1, 1]
    smallest = None
    limit = min(max_chunks, t.seq)
    while True:
        axes = serialization_axes(t, counts)
        tensors, n_ops = _trace.trace(t, tuple(counts), axes)
        _, peak = plan_arena(tensors)
        smallest = peak if smallest is None else min(smallest, peak)
        live = live_per_op(tensors, n_ops)
        over = {phase_of_op(t, counts, op) for op, b in enumerate(live) if b > budget_bytes}
        if not over:
            if peak <= budget_bytes:
                return tuple(counts), axes, peak
            over = {phase_of_op(t, counts, max(range(n_ops), key=lambda op: (live[op], -op)))}
        for ph in sorted(over):
            counts[ph] += 1
            if counts[ph] > limit:
                return None, None, smallest


def chunks_for_budget(t, budget_bytes, max_chunks):
    """Returns (chunks, peak) for the first C in 1..max_chunks whose arena peak fits,
    or (None, smallest peak seen) when none does."""
    smallest = None
    for C in range(1, min(max_chunks, t.seq) + 1):
        tensors, _ = _trace.trace(t, C)
        _, peak = plan_arena(tensors)
        if peak <= budget_bytes:
            return C, peak
        smallest = peak if smallest is None else min(smallest, peak)
    return None, smallest
