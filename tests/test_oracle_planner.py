"""Pins for the layout-planner oracle (Algorithms 1-3, majority-vote merge)."""
import itertools
import math

import numpy as np
import pytest

from oracle import planner as P


def mk(ops):
    return [{"ins": list(i), "outs": list(o)} for i, o in ops]


def table_eval(seed, hi=20):
    """A deterministic, integer-valued stand-in for the measured cost function."""
    def ev(op, lay):
        key = (seed, op) + tuple(sorted(lay.items()))
        return float(np.random.default_rng(abs(hash(key)) % (2 ** 32)).integers(1, hi))
    return ev


CHAIN = mk([([0], [1]), ([1], [2]), ([2], [3]), ([3], [4])])
# a diamond with a long arm: 0 -> a -> b -> c -> join ; 0 -> d -> join
DIAMOND = mk([([0], [1]), ([1], [2]), ([2], [3]), ([3], [4]), ([1], [5]), ([4, 5], [6])])


def test_algorithm1_longest_distance_not_hop_count():
    f = P.Flow(DIAMOND)
    pos = {v: i for i, v in enumerate(f.linearise())}
    # op5 (join) is 2 hops from op0 via op4 but 4 via the long arm: the long arm must be taken
    assert P.find_longest_sequence(f, list(range(6)), pos) == [0, 1, 2, 3, 5]


def test_algorithm2_split_covers_every_node_once():
    f = P.Flow(DIAMOND)
    seqs = P.split(f)
    assert seqs == [[0, 1, 2, 3, 5], [4]]
    # two independent branches hanging off the main chain become separate sequences
    g = mk([([0], [1]), ([1], [2]), ([2], [3]), ([1], [4]), ([4], [5]), ([2], [6]), ([3, 5, 6], [7])])
    seqs = P.split(P.Flow(g))
    assert sorted(itertools.chain(*seqs)) == list(range(7))
    assert seqs[0] == [0, 1, 2, 6] and [3, 4] in seqs and [5] in seqs
    # remains that are still connected stay one sub-flow and are split recursively
    h = mk([([0], [1]), ([1], [2]), ([2], [3]), ([3], [4]), ([1], [5]), ([5], [6]), ([5], [7]), ([4, 6, 7], [8])])
    seqs = P.split(P.Flow(h))
    assert seqs[0] == [0, 1, 2, 3, 7] and seqs[1] == [4, 5] and seqs[2] == [6]


def test_linearise_smallest_ready_first():
    g = mk([([5], [6]), ([0], [5]), ([6], [7])])        # op1 must run before op0
    assert P.Flow(g).linearise() == [1, 0, 2]


def test_chain_edges():
    f = P.Flow(mk([([9, 0], [1]), ([1, 8], [2, 3]), ([3, 2], [4])]), const_ids={9, 8})
    assert P.chain_edges(f, [0, 1, 2]) == [0, 1, 2, 4]


@pytest.mark.parametrize("seed", range(8))
def test_dp_is_optimal_on_a_branch_free_chain(seed):
    ncand = {t: 3 for t in range(5)}
    ncand[0] = 1; ncand[4] = 1                            # pinned graph input / output
    ev = table_eval(seed)
    a, cost, seqs = P.plan_layouts(CHAIN, ncand, ev)
    assert seqs == [[0, 1, 2, 3]]
    _, best = P.brute_force_layouts(CHAIN, ncand, ev)
    assert cost == best == P.total_cost(CHAIN, a, ev)


@pytest.mark.parametrize("seed", range(8))
def test_chain_with_weights_is_still_optimal(seed):
    ops = mk([([0, 10], [1]), ([1, 11], [2]), ([2, 12], [3])])
    ncand = {0: 1, 1: 3, 2: 2, 3: 1, 10: 2, 11: 2, 12: 2}
    ev = table_eval(100 + seed)
    a, cost, _ = P.plan_layouts(ops, ncand, ev, const_ids={10, 11, 12})
    assert cost == P.brute_force_layouts(ops, ncand, ev)[1]


@pytest.mark.parametrize("seed", range(12))
def test_branched_graph_between_optimum_and_canonical(seed):
    ncand = {t: 2 for t in range(7)}
    ncand[0] = 1; ncand[6] = 1
    ev = table_eval(200 + seed)
    a, cost, _ = P.plan_layouts(DIAMOND, ncand, ev)
    _, best = P.brute_force_layouts(DIAMOND, ncand, ev)
    canon = P.total_cost(DIAMOND, {t: 0 for t in ncand}, ev)
    assert best <= cost <= canon
    assert all(0 <= a[t] < ncand[t] for t in ncand)
    assert cost == P.total_cost(DIAMOND, a, ev)


def test_majority_vote():
    assert P.majority({0: 1, 2: 3, 1: 2}) == 2
    assert P.majority({1: 2, 0: 2}) == 0          # tie -> lowest index
    assert P.majority({3: 1}) == 3


def test_conflict_is_resolved_by_vote_and_losers_reoptimise():
    # tensor 1 feeds three single-op consumers; two prefer layout 1, the producer chain prefers 0
    ops = mk([([0], [1]), ([1], [2]), ([1], [3]), ([1], [4])])
    ncand = {0: 1, 1: 2, 2: 1, 3: 1, 4: 1}

    def ev(op, lay):
        l = lay[1]
        return {0: [1.0, 2.0], 1: [1.0, 5.0], 2: [9.0, 1.0], 3: [9.0, 1.0]}[op][l]
    a, cost, seqs = P.plan_layouts(ops, ncand, ev)
    # sequences: [0,1] votes 0 twice? no: one vote per edge occurrence -> edge 1 once per chain
    assert a[1] == 1 and cost == 2.0 + 5.0 + 1.0 + 1.0
    # the guard: if voting makes things worse than canonical, canonical comes back

    def ev2(op, lay):
        l = lay[1]
        return {0: [1.0, 50.0], 1: [1.0, 50.0], 2: [2.0, 1.0], 3: [2.0, 1.0]}[op][l]
    a2, cost2, _ = P.plan_layouts(ops, ncand, ev2)
    assert a2[1] == 0 and cost2 == 6.0


def test_unsupported_combination_is_avoided():
    ops = mk([([0], [1]), ([1], [2])])
    ncand = {0: 1, 1: 2, 2: 1}

    def ev(op, lay):
        return math.inf if lay[1] == 1 else 3.0
    a, cost, _ = P.plan_layouts(ops, ncand, ev)
    assert a[1] == 0 and cost == 6.0


def test_merge_loss_on_toy_graphs_is_reported_next_to_the_papers():
    """The paper's "Cost of Conflict Resolution" experiment: on a linear toy model the schedule is optimal by
    construction; on a branched one the majority-vote merge may lose against exhaustive search. The paper prints
    156.5 vs 130.5 ms and 152.0 vs 138.9 ms for its two (unpublished) toy graphs, i.e. losses of 16.6 % and 8.6 % of
    its own schedule's time. Here: a 5-op chain (loss exactly 0) and the diamond above under 200 random cost tables;
    the mean and the worst loss are printed, and bounded by what the guard guarantees (never above canonical)."""
    ncand = {t: 2 for t in range(6)}
    losses = []
    for seed in range(50):
        ev = table_eval(500 + seed)
        _, cost, _ = P.plan_layouts(CHAIN, ncand, ev)
        assert cost == P.brute_force_layouts(CHAIN, ncand, ev)[1]
    ncand = {t: 2 for t in range(7)}
    ncand[0] = 1; ncand[6] = 1
    for seed in range(200):
        ev = table_eval(1000 + seed)
        _, cost, _ = P.plan_layouts(DIAMOND, ncand, ev)
        _, best = P.brute_force_layouts(DIAMOND, ncand, ev)
        assert best <= cost
        losses.append(1.0 - best / cost)
    mean, worst, hit = sum(losses) / len(losses), max(losses), sum(l == 0 for l in losses)
    print(f"merge loss on the branched toy graph over {len(losses)} cost tables: mean {mean:.1%}, worst {worst:.1%}, "
          f"optimal in {hit} cases (paper's two toy graphs: 16.6 % and 8.6 %); chain: 0 % in every case")
    assert mean < 0.10 and worst < 0.5
