"""Physical optimization in miniature (Section 5.1): walking a planned graph of abstract operators in topological order
and compiling, for every operand that another operator produces, the exchange program that links the two -- preamble from
the two join-agg specs (`ja_exprog_preamble`), placement of the consumer's function specs (`ja_exprog_place`), body
(`ja_exprog_body` / `ja_exprog_synthesize`), completion time from the library's simulator.  Host bookkeeping over the
library's calls; nothing here touches a GPU.

Conventions.  A plan is one dict letter -> interval count per operator (the logical optimizer's output).  The function specs
of an operator are the cells of its count grid in row-major order over its letters (order of first appearance in the
einsum); with p GPUs every operator has p function specs and spec F of a placed operator runs on GPU placement[F].  Copy c
of output block b of a producer is the output of the function spec with output coordinates b and contracted coordinates
c (both row-major).  Inputs of the computation (weights, the block's input) are taken to be where they are needed, as the
logical cost model does (Opt = 0 for them).
"""
from __future__ import annotations

import itertools
import math

from . import exprog as X


def _terms(einsum: str):
    lhs, out = einsum.replace(" ", "").split("->")
    ins = lhs.split(",")
    letters = []
    for t in ins + [out]:
        for c in t:
            if c not in letters:
                letters.append(c)
    return ins, out, letters


def equal_splits(extent: int, n: int):
    return [s * extent // n for s in range(n + 1)]


def edge(ops, plan, consumer: int, operand: int, producer_sites, width_bytes: int = 2) -> dict:
    """Arguments of ja_exprog_preamble for operand `operand` of operator `consumer`."""
    op = ops[consumer]
    prod = op["inputs"][operand]
    pins, pout, pletters = _terms(ops[prod]["einsum"])
    cins, _, cletters = _terms(op["einsum"])
    pc, cc = plan[prod], plan[consumer]
    term = cins[operand]
    ext = [ops[prod]["extents"][c] for c in pout]
    contracted = [c for c in pletters if c not in pout]
    m = math.prod(pc[c] for c in contracted)
    n_blocks = math.prod(pc[c] for c in pout)
    copy_site = [None] * (n_blocks * m)
    for f, cell in enumerate(itertools.product(*[range(pc[c]) for c in pletters])):
        at = dict(zip(pletters, cell))
        b = 0
        for c in pout:
            b = b * pc[c] + at[c]
        k = 0
        for c in contracted:
            k = k * pc[c] + at[c]
        copy_site[b * m + k] = producer_sites[f]
    specs = []
    for cell in itertools.product(*[range(cc[c]) for c in cletters]):
        at = dict(zip(cletters, cell))
        b = 0
        for c in term:
            b = b * cc[c] + at[c]
        specs.append(b)
    return {"producer_splits": [equal_splits(e, pc[c]) for e, c in zip(ext, pout)],
            "consumer_splits": [equal_splits(e, cc[c]) for e, c in zip(ext, term)],
            "m": m, "copy_site": copy_site, "consumer_specs": specs, "width_bytes": width_bytes,
            "tensor_bytes": math.prod(ext) * width_bytes}


def compile_exchanges(ops, plan, machine, optimise: bool, depth: int = 2, beam: int = 6, width_bytes: int = 2, joint: bool = True):
    """Every producer -> consumer edge of the planned graph as an exchange program, operators in topological order.
    joint: the exchanges of all operands of one operator form ONE program (`ja_exprog_merge`), as Section 5.1 compiles one
    program per operator -- they share the placement of its function specs and run at the same time; operators whose operands
    together have more than 64 atoms, and joint = False, fall back to one program per operand, their times added.
    optimise = False: the naive programs of the paper's Experiment 4 -- function spec i on GPU i, every aggregated block
    gathered and aggregated where it is consumed.  optimise = True: every body goes through ja_exprog_synthesize, and the
    placement of a consumer's function specs is the best, by simulated time, of spec i on GPU i and of what ja_exprog_place
    chooses (for the joint program, or for each operand by itself); since a placement also moves the copies the next operator
    starts from, the whole compilation is done a second time with every operator left at spec i on GPU i and the faster of the
    two is returned.  Returns (total simulated ms, per-operator records)."""
    if not optimise:
        return _compile(ops, plan, machine, "naive", depth, beam, width_bytes, joint)
    placed = _compile(ops, plan, machine, "placed", depth, beam, width_bytes, joint)
    fixed = _compile(ops, plan, machine, "fixed", depth, beam, width_bytes, joint)
    return placed if placed[0] <= fixed[0] else fixed


def _compile(ops, plan, machine, mode, depth, beam, width_bytes, joint):
    p = None
    placement = {}
    records = []
    total = 0.0
    for j, op in enumerate(ops):
        _, _, letters = _terms(op["einsum"])
        n_specs = math.prod(plan[j][c] for c in letters)
        p = p or n_specs
        if n_specs != p:
            raise ValueError("operator %d has %d function specs, the others %d" % (j, n_specs, p))
        operands = [k for k, i in enumerate(op["inputs"]) if i is not None]
        identity = list(range(p))
        if not operands:
            placement[j] = identity
            continue
        args = {k: edge(ops, plan, j, k, placement[op["inputs"][k]], width_bytes) for k in operands}

        def operand_program(k, sites):
            a = args[k]
            h = X.ExchangeProgram(handle=X.ja_exprog_preamble(a["producer_splits"], a["consumer_splits"], a["m"], a["copy_site"],
                                                              a["consumer_specs"], a["width_bytes"]))
            if sites is not None:
                for i, s in enumerate(sites):
                    X.ja_exprog_bind_members(h, "S%d" % (i + 1), [s])
            return h

        def programs(sites):
            """The operator's exchange as a list of programs: one (all operands merged) or one per operand."""
            hs = [operand_program(k, sites) for k in operands]
            if joint and len(hs) > 1 and sum(X.ja_exprog_counts(h)["atoms"] for h in hs) <= 64:
                merged = hs[0]
                for n, h in enumerate(hs[1:], 1):
                    merged = merged.merge(h, "k0_" if n == 1 else "", "k%d_" % n)
                return [merged]
            return hs

        def sites_of(h):
            return [X.ja_exprog_membership(h, "S%d" % (i + 1)).bit_length() - 1 for i in range(p)]

        def cost_with(sites):
            hs = programs(sites)
            if mode == "naive":
                for h in hs:
                    X.ja_exprog_body(h, "naive")
                ms = [X.ja_exprog_simulate(h, machine) for h in hs]
            else:
                ms = [X.ja_exprog_synthesize(h, machine, depth, beam) for h in hs]
            return sum(ms), sum(X.ja_exprog_counts(h)["expanded"] for h in hs), len(hs)

        candidates = [identity]
        if mode == "placed":
            for h in programs(None):
                X.ja_exprog_place(h, machine, "best")
                sites = sites_of(h)
                if sites not in candidates:
                    candidates.append(sites)
        best = None
        for sites in candidates:
            ms, n_actions, n_programs = cost_with(sites)
            if best is None or ms < best[0] * (1.0 - 1e-12):
                best = (ms, sites, n_actions, n_programs)
        placement[j] = best[1]
        records.append({"consumer": j, "operands": operands, "ms": best[0], "actions": best[2], "programs": best[3],
                        "m": [args[k]["m"] for k in operands], "tensor_MB": [args[k]["tensor_bytes"] / 1e6 for k in operands]})
        total += best[0]
    return total, records
