"""TEST INFRASTRUCTURE ONLY -- logical optimization (paper Section 4): choosing one join-agg spec per
abstract operator of a computation tree so that the communication proxy Cost is minimal.

Written from Section 4.2 (the recurrence Opt(Op, T), B(J), Algorithm 1 with its traceback) and Section
4.3 (the three sub-costs).  Two independent routes are provided so that one pins the other:
  * `optimize_tree`   the dynamic program of Algorithm 1, operators visited bottom-up;
  * `exhaustive`      every assignment of one spec per operator, costed directly (tiny trees only).

A computation is a list of operators in topological order.  Operator = dict(einsum=..., extents={letter: n},
inputs=[producer index | None, ...], fixed=set of letters that are not shardable).  `None` marks an input of
the computation (Opt = 0 for every tiling, and no repartition charge).  A tiling of a tensor is the tuple of
interval counts of its indices (Einsummable asks for near-equal intervals, so counts determine the tiling).
"""
from __future__ import annotations

import itertools

from . import blocked


def parse(einsum: str):
    lhs, out = einsum.replace(" ", "").split("->")
    ins = lhs.split(",")
    letters = []
    for term in ins:
        for c in term:
            if c not in letters:
                letters.append(c)
    return ins, out, letters


def specs(op: dict, p: int):
    """specs(Op): one join-agg spec per decomposition of the shardable indices into interval counts whose
    product is p (an index cannot have more intervals than cells).  A spec is {letter: count}; enumerated
    in lexicographic order of the count vector over the letters in order of first appearance."""
    _, _, letters = parse(op["einsum"])
    fixed = op.get("fixed", set())

    def rec(i, rest):
        if i == len(letters):
            if rest == 1:
                yield ()
            return
        l = letters[i]
        choices = [1] if l in fixed else [c for c in range(1, rest + 1) if rest % c == 0 and c <= op["extents"][l]]
        for c in choices:
            for tail in rec(i + 1, rest // c):
                yield (c,) + tail

    return [dict(zip(letters, counts)) for counts in rec(0, p)]


def tiling_of(op: dict, spec: dict, operand: int):
    """in_k(J) for operand k >= 0, out(J) for operand -1, as a tuple of interval counts."""
    ins, out, _ = parse(op["einsum"])
    term = out if operand < 0 else ins[operand]
    return tuple(spec[c] for c in term)


def card(op: dict, operand: int) -> int:
    ins, out, _ = parse(op["einsum"])
    term = out if operand < 0 else ins[operand]
    n = 1
    for c in term:
        n *= op["extents"][c]
    return n


def cost(op: dict, spec: dict, input_tilings) -> int:
    """Cost(J, T_1..T_n), Section 4.3.  input_tilings[k] is None for an input of the computation.
    (1) repartition: card of the whole input if in_k(J) != T_k; (2) join: over all function specs, the
    cells of every input block; (3) aggregation: (m - 1) cells of every distinct output type.  Sub-costs
    (2) and (3) are counted on the explicit spec (blocked.Spec), not by a closed form."""
    ins, _, letters = parse(op["einsum"])
    parts = {l: blocked.equal_splits(op["extents"][l], spec[l]) for l in letters}
    join, agg = blocked.Spec(op["einsum"], parts).cost_terms()
    total = join + agg
    for k, T in enumerate(input_tilings):
        if T is not None and tuple(T) != tiling_of(op, spec, k):
            total += card(op, k)
    return int(total)


def optimize_tree(ops, p: int):
    """Algorithm 1.  Returns (total cost, [spec per operator])."""
    cand, opt, choice = {}, {}, {}
    for idx, op in enumerate(ops):
        cand[idx] = []
        prods = op["inputs"]
        for J in specs(op, p):
            lists = [[None] if q is None else cand[q] for q in prods]
            best, best_T = None, None
            for Ts in itertools.product(*lists):
                b = sum(0 if q is None else opt[(q, T)] for q, T in zip(prods, Ts)) + cost(op, J, Ts)
                if best is None or b < best:
                    best, best_T = b, Ts
            T = tiling_of(op, J, -1)
            if T not in cand[idx] or best < opt[(idx, T)]:
                if T not in cand[idx]:
                    cand[idx].append(T)
                opt[(idx, T)] = best
                choice[(idx, T)] = (J, best_T)
    root = len(ops) - 1
    T_star = min(cand[root], key=lambda T: opt[(root, T)])
    chosen = [None] * len(ops)

    def assign(idx, T):
        J, Ts = choice[(idx, T)]
        chosen[idx] = J
        for q, Tq in zip(ops[idx]["inputs"], Ts):
            if q is not None:
                assign(q, Tq)

    assign(root, T_star)
    return opt[(root, T_star)], chosen


def greedy(ops, p: int):
    """The greedy selector of Section 6, Experiment 3: the dynamic program with the repartition sub-cost removed.  Nothing
    then couples an operator to its producers, so each takes the spec of least join + aggregation cost on its own (the
    first such spec in the order of `specs`).  Returns (full cost of that plan, repartition charges included, plan)."""
    plan = []
    for op in ops:
        free = [None] * len(op["inputs"])
        plan.append(min(specs(op, p), key=lambda J: cost(op, J, free)))      # min() keeps the first of equal keys
    return plan_cost(ops, plan), plan


def plan_cost(ops, plan) -> int:
    """Cost of a complete assignment: every operator pays Cost with its producers' output tilings."""
    total = 0
    for op, J in zip(ops, plan):
        Ts = [None if q is None else tiling_of(ops[q], plan[q], -1) for q in op["inputs"]]
        total += cost(op, J, Ts)
    return total


def exhaustive(ops, p: int):
    """Minimum of plan_cost over every assignment of one spec per operator."""
    best, best_plan = None, None
    for plan in itertools.product(*[specs(op, p) for op in ops]):
        c = plan_cost(ops, plan)
        if best is None or c < best:
            best, best_plan = c, list(plan)
    return best, best_plan


# ---------------------------------------------------------------------------------------------------
# Outputs with several consumers (Section 4.5): the graph is cut at every edge out of a multiply
# consumed tensor and the resulting trees are optimised one at a time, largest first, each subject
# to the specs already fixed.
# ---------------------------------------------------------------------------------------------------
def cut_into_trees(ops):
    """Returns [(root, sorted member nodes)], largest tree first (ties: smaller root first).  Roots are the
    operators whose output is not consumed exactly once; a tree is its root plus every producer reachable
    through singly-consumed outputs."""
    consumers = [0] * len(ops)
    for op in ops:
        for q in op["inputs"]:
            if q is not None:
                consumers[q] += 1
    trees = []
    for root in range(len(ops)):
        if consumers[root] == 1:
            continue
        members, stack = [], [root]
        while stack:
            i = stack.pop()
            members.append(i)
            stack += [q for q in ops[i]["inputs"] if q is not None and consumers[q] == 1]
        trees.append((root, sorted(members)))
    trees.sort(key=lambda t: (-len(t[1]), t[0]))
    return trees


def optimize_graph(ops, p: int):
    """Section 4.5.  An operand produced in a tree that is already optimised enters like an input whose tiling
    is fixed (Cost charges the repartition when in_k(J) differs from it); an operand produced in a tree not
    yet optimised enters like an input of the computation.  When the root of a tree feeds consumers whose
    specs are already fixed, the root's tiling is chosen with their repartition charges added (the paper only
    says 'subject to the specs already fixed'; this is the reading taken).
    Returns (plan_cost of the assembled plan, plan)."""
    plan = [None] * len(ops)
    for root, members in cut_into_trees(ops):
        inside = set(members)
        cand, opt, choice = {}, {}, {}
        for idx in members:                     # members are sorted = topological
            op = ops[idx]
            cand[idx] = []
            for J in specs(op, p):
                lists = []
                for q in op["inputs"]:
                    if q is None or (q not in inside and plan[q] is None):
                        lists.append([None])
                    elif q in inside:
                        lists.append(cand[q])
                    else:
                        lists.append([tiling_of(ops[q], plan[q], -1)])
                best, best_T = None, None
                for Ts in itertools.product(*lists):
                    b = cost(op, J, Ts) + sum(opt[(q, T)] for q, T in zip(op["inputs"], Ts) if q is not None and q in inside)
                    if best is None or b < best:
                        best, best_T = b, Ts
                T = tiling_of(op, J, -1)
                if T not in cand[idx] or best < opt[(idx, T)]:
                    if T not in cand[idx]:
                        cand[idx].append(T)
                    opt[(idx, T)] = best
                    choice[(idx, T)] = (J, best_T)

        def consumer_charge(T):
            c = 0
            for j, op in enumerate(ops):
                if plan[j] is None:
                    continue
                for k, q in enumerate(op["inputs"]):
                    if q == root and tiling_of(op, plan[j], k) != T:
                        c += card(op, k)
            return c

        T_star = min(cand[root], key=lambda T: opt[(root, T)] + consumer_charge(T))

        def assign(idx, T):
            J, Ts = choice[(idx, T)]
            plan[idx] = J
            for q, Tq in zip(ops[idx]["inputs"], Ts):
                if q is not None and q in inside:
                    assign(q, Tq)

        assign(root, T_star)
    return plan_cost(ops, plan), plan
