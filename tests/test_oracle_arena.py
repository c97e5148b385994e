"""Pins for the arena oracle (Algorithm 4): closed forms, independent checker, brute force."""
import numpy as np
import pytest

from oracle import arena as A

H = A.HEADER


def recs(sizes, lifetimes):
    return [(i, s, f, l) for i, (s, (f, l)) in enumerate(zip(sizes, lifetimes))]


def test_disjoint_lifetimes_share_one_slot():
    r = recs([1000, 5000, 300], [(0, 1), (2, 3), (4, 5)])
    off, peak = A.greedy_by_size(r)
    assert peak == H + A.round_up(5000) and set(off.values()) == {H}
    assert A.check_arena(r, off, peak) == []


def test_all_overlapping_need_the_sum():
    r = recs([256, 512, 1024, 100], [(0, 9)] * 4)
    off, peak = A.greedy_by_size(r)
    assert peak == H + 256 + 512 + 1024 + 256
    assert off[2] == H and off[1] == H + 1024 and off[0] == H + 1536 and off[3] == H + 1792
    assert A.check_arena(r, off, peak) == []


def test_chain_lower_bound_and_hand_example():
    # tensor i lives while tensor i+1 is produced: [i, i+1]
    sizes = [512, 2048, 256, 1024, 768]
    r = recs(sizes, [(i, i + 1) for i in range(5)])
    off, peak = A.greedy_by_size(r)
    pair = max(A.round_up(a) + A.round_up(b) for a, b in zip(sizes, sizes[1:]))
    assert A.live_set_bound(r) == H + pair
    assert peak >= H + pair and A.check_arena(r, off, peak) == []
    assert A.brute_force_arena(r) == H + pair
    # a hand-worked case: the gap under a short-lived big block is reused (first fit)
    r = [(0, 1024, 0, 1), (1, 512, 1, 3), (2, 512, 2, 3), (3, 256, 0, 0)]
    off, peak = A.greedy_by_size(r)
    assert off == {0: H, 1: H + 1024, 2: H, 3: H + 1024} and peak == H + 1536


def test_first_fit_versus_best_fit():
    # Hand-worked: P, Q, R, S are all alive at step 0, so they stack by size (ties: smaller id first):
    #   P 1024 @ H, Q 512 @ H+1024, R 512 @ H+1536, S 256 @ H+2048.
    # T (256 bytes, alive at step 2 only) conflicts with Q and S alone, which leaves it two gaps: P's old range
    # (1024 bytes at H) and R's old range (512 bytes at H+1536). The pseudo-code's first slot is the lower one;
    # the prose's "most suitable" slot is the tighter one. The two policies must therefore differ here.
    r = [(0, 1024, 0, 0), (1, 512, 0, 2), (2, 512, 0, 0), (3, 256, 0, 2), (4, 256, 2, 2)]
    off_f, peak_f = A.greedy_by_size(r, policy="first")
    off_b, peak_b = A.greedy_by_size(r, policy="best")
    assert off_f == {0: H, 1: H + 1024, 2: H + 1536, 3: H + 2048, 4: H}
    assert off_b == {0: H, 1: H + 1024, 2: H + 1536, 3: H + 2048, 4: H + 1536}
    assert peak_f == peak_b == H + 2304
    assert A.check_arena(r, off_f, peak_f) == [] and A.check_arena(r, off_b, peak_b) == []
    # equally tight gaps: best fit falls back to the lower offset
    r = [(0, 512, 0, 0), (1, 512, 0, 2), (2, 512, 0, 0), (3, 256, 0, 2), (4, 256, 2, 2)]
    off_b, _ = A.greedy_by_size(r, policy="best")
    assert off_b[4] == H


def test_sort_order_ties():
    r = [(5, 512, 3, 4), (2, 512, 0, 9), (7, 512, 0, 9)]
    off, _ = A.greedy_by_size(r)
    # same size: earlier first-step first, then smaller id -> record 2 gets the bottom slot
    assert off[2] == H and off[7] == H + 512 and off[5] == H + 1024


def test_checker_catches_violations():
    r = recs([512, 512], [(0, 2), (1, 3)])
    assert A.check_arena(r, {0: H, 1: H + 512}, H + 1024) == []
    assert any("overlap" in m for m in A.check_arena(r, {0: H, 1: H + 256}, H + 768))
    assert any("aligned" in m for m in A.check_arena(r, {0: H, 1: H + 513}, H + 1025))
    assert any("header" in m for m in A.check_arena(r, {0: 0, 1: H + 512}, H + 1024))
    assert any("arena_bytes" in m for m in A.check_arena(r, {0: H, 1: H + 512}, H + 2048))


@pytest.mark.parametrize("seed", range(20))
def test_random_small_sets_against_brute_force(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(3, 7))
    r = []
    for i in range(n):
        f = int(rng.integers(0, 8)); l = f + int(rng.integers(0, 4))
        r.append((i, int(rng.integers(1, 9)) * 256 - int(rng.integers(0, 200)), f, l))
    for policy in ("first", "best"):
        off, peak = A.greedy_by_size(r, policy=policy)
        assert A.check_arena(r, off, peak) == []
        opt = A.brute_force_arena(r)
        assert A.live_set_bound(r) <= opt <= peak <= A.naive_sum(r)


def test_empty():
    assert A.greedy_by_size([]) == ({}, H)
