"""CPU oracle for the layout planner: the paper's algorithms step by step. TEST INFRASTRUCTURE ONLY.

Follows Sec. "Design", "Holistic Graph-Operator Optimization": Algorithm 1
(LongestSequenceExtraction), Algorithm 2 (RecursiveExtraction), Eq. 1 / Algorithm 3
(DPOnSequence) and the majority-vote merge paragraph, in that order, plus the exhaustive search
the paper uses in Sec. "Cost of Conflict Resolution" to bound the merge loss.

Vocabulary: a *node* is an operator, an *edge* is a tensor; `eval(node, layouts)` is the paper's
external cost function (Algorithm 3): here any callable (op id, {tensor id: layout index}) ->
cost. A layout is referred to by its index in the tensor's candidate list; index 0 is canonical.

Readings taken where the text is terse or at odds with itself (each is also what the library
implements, so that both produce the same plan bit for bit):
  * Algorithm 1's prose asks for the *longest* distance while its pseudo-code enqueues a node
    once; this follows the prose: dist(v) = 1 + max dist(pred), sources 0, ties -> smaller id.
  * Algorithm 2's inner call is the recursion split(subflow) (its result is iterated as many
    sequences); sub-flows are the connected components of what remains, smallest id first.
  * Eq. 1 sums over predecessor layouts where it must minimise; the table is filled forward and
    the layouts are read back from the best final layout (the prose after Eq. 1), ties -> the
    lower candidate index.
  * Tensors of a node that are not the chain's incoming or outgoing edge (weights, skip
    connections, edges owned by another sequence) are minimised over inside eval's argument and
    reported as that sequence's proposal for them.
  * Majority vote: most proposals wins. The paper breaks ties at random; here a tie goes to the
    tied layout under which the sequences, re-optimised with it fixed, cost least in total, then
    to the lowest index (any choice is valid; tests check validity and cost, not the pick).
    After each vote all sequences are re-run with the winners fixed until no edge is proposed
    two ways.
  * Not in the paper: if the merged plan costs more than the all-canonical plan, canonical is
    returned (so a plan never loses to doing nothing).

Pins (tests/test_oracle_planner.py): on a branch-free chain the result equals the exhaustive
optimum (the paper's Fig. "dp" caption: simple connections are solved optimally); on branched
graphs optimum <= result <= canonical; hand-made vote tables; hand-made graphs for Algorithms 1-2.
Which of several equally cheap plans is returned is "parity unpinned" (tie-breaks are a reading).
"""
from __future__ import annotations

import itertools
import math


class Flow:
    """Producer/consumer relations of a graph given as ops = [{"ins": [...], "outs": [...]}]."""

    def __init__(self, ops, const_ids=()):
        self.ops = ops
        self.const_ids = set(const_ids)
        self.producer = {}
        for oid, op in enumerate(ops):
            for t in op["outs"]:
                self.producer[t] = oid
        self.pred = [sorted({self.producer[t] for t in op["ins"] if t in self.producer})
                     for op in ops]
        self.succ = [[] for _ in ops]
        for v, ps in enumerate(self.pred):
            for p in ps:
                self.succ[p].append(v)

    def linearise(self):
        """Topological order, smallest ready op id first (the graph -> linear sequence pass)."""
        indeg = [len(p) for p in self.pred]
        ready = sorted(v for v, d in enumerate(indeg) if d == 0)
        order = []
        while ready:
            v = ready.pop(0)
            order.append(v)
            for s in self.succ[v]:
                indeg[s] -= 1
                if indeg[s] == 0:
                    ready.append(s)
                    ready.sort()
        assert len(order) == len(self.ops), "graph has a cycle"
        return order


def find_longest_sequence(flow: Flow, nodes, order_pos):
    """Algorithm 1 on the sub-flow `nodes`: label longest distances from the sub-flow's sources,
    take the farthest node, walk back along the recorded predecessors."""
    inside = set(nodes)
    dist, back = {}, {}
    for v in sorted(nodes, key=lambda n: order_pos[n]):
        best_d, best_p = -1, None
        for p in flow.pred[v]:
            if p in inside and (dist[p] > best_d):
                best_d, best_p = dist[p], p
        dist[v] = best_d + 1 if best_p is not None else 0
        back[v] = best_p
    end = min(nodes, key=lambda n: (-dist[n], n))
    seq = [end]
    while back[seq[-1]] is not None:
        seq.append(back[seq[-1]])
    seq.reverse()
    return seq


def split(flow: Flow, nodes=None, order_pos=None):
    """Algorithm 2: peel the longest sequence, recurse into the connected remains."""
    if nodes is None:
        nodes = list(range(len(flow.ops)))
    if order_pos is None:
        order_pos = {v: i for i, v in enumerate(flow.linearise())}
    if not nodes:
        return []
    seq = find_longest_sequence(flow, nodes, order_pos)
    rest = set(nodes) - set(seq)
    sequences = [seq]
    seen = set()
    for start in sorted(rest):
        if start in seen:
            continue
        comp, stack = [], [start]
        seen.add(start)
        while stack:
            v = stack.pop()
            comp.append(v)
            for u in flow.pred[v] + flow.succ[v]:
                if u in rest and u not in seen:
                    seen.add(u)
                    stack.append(u)
        sequences += split(flow, sorted(comp), order_pos)
    return sequences


def chain_edges(flow: Flow, seq):
    """Edges e_0..e_n of a sequence o_1..o_n: e_i joins o_i to o_(i+1) (smallest tensor id if
    several do); e_0 is o_1's first non-constant input (None if it has none); e_n is o_n's
    first output."""
    ops = flow.ops
    e0 = next((t for t in ops[seq[0]]["ins"] if t not in flow.const_ids), None)
    edges = [e0]
    for a, b in zip(seq, seq[1:]):
        edges.append(min(set(ops[a]["outs"]) & set(ops[b]["ins"])))
    edges.append(ops[seq[-1]]["outs"][0])
    return edges


def _op_tensors(op):
    seen, out = set(), []
    for t in list(op["ins"]) + list(op["outs"]):
        if t not in seen:
            seen.add(t)
            out.append(t)
    return out


def dp_on_sequence(flow: Flow, seq, ncand, fixed, evalfn):
    """Eq. 1 / Algorithm 3 on one sequence. Returns (proposals, cost): proposals is a list of
    (tensor, layout index), one per chain edge and one per side-tensor occurrence."""
    edges = chain_edges(flow, seq)

    def allowed(t):
        if t is None:
            return [0]
        return [fixed[t]] if t in fixed else list(range(ncand[t]))

    prev = {l: 0.0 for l in allowed(edges[0])}
    backs = []
    for i, oid in enumerate(seq, start=1):
        e_in, e_out = edges[i - 1], edges[i]
        side = [t for t in _op_tensors(flow.ops[oid]) if t != e_in and t != e_out]
        side_opts = [allowed(s) for s in side]
        cur, back = {}, {}
        for l in allowed(e_out):
            best, arg = math.inf, None
            for lp in allowed(e_in):
                if math.isinf(prev[lp]):
                    continue
                for assign in itertools.product(*side_opts):
                    lay = dict(zip(side, assign))
                    if e_in is not None:
                        lay[e_in] = lp
                    lay[e_out] = l
                    c = prev[lp] + evalfn(oid, lay)
                    if c < best:
                        best, arg = c, (lp, assign)
            cur[l], back[l] = best, arg
        backs.append((side, back))
        prev = cur
    l = min(prev, key=lambda k: (prev[k], k))
    cost = prev[l]
    if math.isinf(cost):
        return None, cost
    proposals = [(edges[-1], l)]
    for i in range(len(seq), 0, -1):
        side, back = backs[i - 1]
        lp, assign = back[l]
        proposals += list(zip(side, assign))
        if edges[i - 1] is not None:
            proposals.append((edges[i - 1], lp))
        l = lp
    return proposals, cost


def majority(votes):
    """votes: {layout index: count} -> the index proposed most often, ties -> lowest index."""
    return min(votes, key=lambda k: (-votes[k], k))


def total_cost(ops, assignment, evalfn):
    return sum(evalfn(oid, {t: assignment[t] for t in _op_tensors(op)})
               for oid, op in enumerate(ops))


def plan_layouts(ops, ncand, evalfn, const_ids=()):
    """The whole layout schedule: split, DP per sequence, vote, re-optimise, guard.

    ncand: {tensor id: number of layout candidates} (1 pins a tensor to canonical).
    Returns (assignment {tensor: index}, cost, sequences).
    """
    flow = Flow(ops, const_ids)
    sequences = split(flow)
    fixed = {}
    while True:
        votes = {}
        for seq in sequences:
            proposals, _ = dp_on_sequence(flow, seq, ncand, fixed, evalfn)
            if proposals is None:
                raise ValueError("no supported layout assignment on a sequence")
            for t, l in proposals:
                votes.setdefault(t, {})
                votes[t][l] = votes[t].get(l, 0) + 1
        conflicted = sorted(t for t, v in votes.items() if len(v) > 1)
        if not conflicted:
            break
        for t in conflicted:
            top = max(votes[t].values())
            tied = sorted(l for l, c in votes[t].items() if c == top)
            if len(tied) == 1:
                fixed[t] = tied[0]
                continue
            best, best_cost = None, None
            for l in tied:
                trial = dict(fixed)
                trial[t] = l
                c = sum(dp_on_sequence(flow, seq, ncand, trial, evalfn)[1] for seq in sequences)
                if best is None or c < best_cost:
                    best, best_cost = l, c
            fixed[t] = best
    assignment = {t: next(iter(v)) for t, v in votes.items()}
    for t in ncand:
        assignment.setdefault(t, 0)
    cost = total_cost(ops, assignment, evalfn)
    canonical = {t: 0 for t in assignment}
    c0 = total_cost(ops, canonical, evalfn)
    if cost > c0:
        assignment, cost = canonical, c0
    return assignment, cost, sequences


def brute_force_layouts(ops, ncand, evalfn):
    """Exhaustive optimum over every combination of candidate layouts (tiny graphs only)."""
    tids = sorted(ncand)
    best, arg = math.inf, None
    for combo in itertools.product(*[range(ncand[t]) for t in tids]):
        a = dict(zip(tids, combo))
        c = total_cost(ops, a, evalfn)
        if c < best:
            best, arg = c, a
    return arg, best
