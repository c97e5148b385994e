"""CPU oracle for the arena plan: Greedy-by-Size, a validity checker, brute force. TEST ONLY.

Follows Algorithm 4 (Greedy-by-Size) and Sec. "Design", "Memory Allocation and Management":
tensors whose lifetimes do not overlap may share addresses inside one big block; tensors are
taken largest first and put into the first slot that holds them, else the block grows.

A record is (id, size, first, last): size in bytes, lifetime = the inclusive step interval
[first, last] of the linear sequence. Two records conflict iff first_a <= last_b and
first_b <= last_a.

Readings where Algorithm 4 is terse (the library implements the same ones):
  * "delete the available space of the tensor whose lifetime overlaps": the free slots for the
    current tensor are the gaps, from the header upward, between the address ranges of the
    already placed tensors that conflict with it.
  * the pseudo-code takes the first slot that is large enough (lowest offset); the prose says
    "most suitable": policy="best" picks the smallest adequate gap instead. Default "first".
  * "increase and allocate the last free available block": the tail slot starts at the highest
    end address among the conflicting placed tensors.
  * sort ties: earlier first step, then smaller id. Sizes are rounded up to `align` bytes and
    the first `header` bytes of the block are reserved.

Pins (tests/test_oracle_arena.py): closed forms (all-disjoint lifetimes -> max size; all
overlapping -> sum of sizes; chains), the independent pairwise checker below, the live-set lower
bound, and exhaustive search over placement orders for n <= 7.
"""
from __future__ import annotations

import itertools

ALIGN = 256
HEADER = 256


def round_up(n, a=ALIGN):
    return (n + a - 1) // a * a


def conflicts(a, b):
    return a[2] <= b[3] and b[2] <= a[3]


def _place(rec, placed, size, header, policy):
    """Offset for `rec` given {id: (offset, size, first, last)} already placed."""
    busy = sorted((o, o + s) for (o, s, f, l) in placed.values()
                  if f <= rec[3] and rec[2] <= l)
    gaps, cursor = [], header
    for lo, hi in busy:
        if lo - cursor >= size:
            gaps.append((cursor, lo - cursor))
        cursor = max(cursor, hi)
    if gaps:
        if policy == "best":
            return min(gaps, key=lambda g: (g[1], g[0]))[0]
        return gaps[0][0]
    return cursor


def greedy_by_size(records, align=ALIGN, header=HEADER, policy="first"):
    """Algorithm 4. Returns ({id: offset}, arena_bytes)."""
    order = sorted(records, key=lambda r: (-round_up(r[1], align), r[2], r[0]))
    placed = {}
    arena = header
    for rec in order:
        size = round_up(rec[1], align)
        off = _place(rec, placed, size, header, policy)
        placed[rec[0]] = (off, size, rec[2], rec[3])
        arena = max(arena, off + size)
    return {k: v[0] for k, v in placed.items()}, arena


def live_set_bound(records, align=ALIGN, header=HEADER):
    """header + the largest sum of sizes simultaneously alive at one step."""
    if not records:
        return header
    steps = sorted({r[2] for r in records} | {r[3] for r in records})
    return header + max(sum(round_up(r[1], align) for r in records if r[2] <= t <= r[3])
                        for t in steps)


def naive_sum(records, align=ALIGN, header=HEADER):
    return header + sum(round_up(r[1], align) for r in records)


def check_arena(records, offsets, arena_bytes, align=ALIGN, header=HEADER):
    """Independent O(n^2) validity check; returns a list of violation strings (empty = valid)."""
    bad = []
    top = header
    for r in records:
        off = offsets[r[0]]
        size = round_up(r[1], align)
        if off % align:
            bad.append(f"record {r[0]}: offset {off} not {align}-aligned")
        if off < header:
            bad.append(f"record {r[0]}: offset {off} inside the header")
        top = max(top, off + size)
    for a, b in itertools.combinations(records, 2):
        if conflicts(a, b):
            oa, ob = offsets[a[0]], offsets[b[0]]
            if oa < ob + round_up(b[1], align) and ob < oa + round_up(a[1], align):
                bad.append(f"records {a[0]} and {b[0]} overlap in lifetime and address")
    if arena_bytes != top:
        bad.append(f"arena_bytes {arena_bytes} != max(offset+size) {top}")
    if arena_bytes < live_set_bound(records, align, header):
        bad.append("arena smaller than the largest live set")
    if arena_bytes > naive_sum(records, align, header):
        bad.append("arena larger than one slice per tensor")
    return bad


def brute_force_arena(records, align=ALIGN, header=HEADER):
    """Smallest peak over every placement order with lowest-feasible-offset placement.

    Any packing can be turned into one of these without raising its peak (slide each block down
    in order of offset), so the minimum over orders is the optimum. n! orders: n <= 7 or so.
    """
    best = None
    for order in itertools.permutations(records):
        placed, arena = {}, header
        for rec in order:
            size = round_up(rec[1], align)
            off = _place(rec, placed, size, header, "first")
            placed[rec[0]] = (off, size, rec[2], rec[3])
            arena = max(arena, off + size)
            if best is not None and arena >= best:
                break
        else:
            best = arena if best is None else min(best, arena)
    return best if best is not None else header
