"""Pins of the exchange-program oracle (oracle/exprog.py) to what the paper prints and to what Definition
"Closure; validity" and the cost model of Section 5.2 fix: the completion times and the membership of the three worked
examples, the generated preamble of Section 5.3, closed forms of the simulator, the two primitive transformations and the
completeness theorem, and the guards of the four rule families."""
import itertools
import json
import os
import random

import pytest

from oracle import exprog as E

G = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "exprog_examples.json")))
H100, V100 = E.machine("dgx_h100"), E.machine("dgx_v100")


def printed(ms, digits):
    return round(ms, digits)


@pytest.mark.parametrize("name", ["swap", "doubling"])
def test_completion_times_the_paper_reports_on_the_h100(name):
    g = G[name]
    p = E.parse(g["program"])
    assert E.valid(p)
    assert printed(E.simulate(p, E.machine(g["machine"])), g["printed_digits"]) == g["completion_ms"]


def test_swap_transfers_overlap_and_take_what_the_paper_says():
    ms, trace = E.simulate(E.parse(G["swap"]["program"]), H100, trace=True)
    sends = [t for (x, s, d), t in trace if d]
    assert len(sends) == 2 and all(t[0] == 0.0 for t in sends)                     # both eligible at once, concurrent
    assert all(round(t[2], 1) == G["swap"]["transfers_ms"] for t in sends)
    aggs = [t for (x, s, d), t in trace if not d]
    assert all(t[0] == sends[0][2] and t[2] == ms for t in aggs)                    # the aggregations run when they complete
    assert abs(ms - (1 / 450 + 3 / 3350) * 1e3) < 1e-9                              # 1 GB over the link, then 2 reads + 1 write


def test_v100_example_membership_time_and_body():
    g = G["v100"]
    p = E.parse(g["program"])
    ok = [m for m in E.memberships(p) if E.valid_bound(E.bind(p, m))]
    assert ok == [{k: tuple(v) for k, v in g["membership"].items()}]                # the only choice the printed body is valid for
    assert len(list(E.memberships(p))) == 70
    m, q, ms = E.place(p, V100)
    assert printed(ms, g["printed_digits"]) == g["completion_ms"]
    ms_trace, trace = E.simulate(q, V100, trace=True)
    # first round on 25 GB/s links inside a socket, second on the 50 GB/s pillars, nothing over the PCIe bridge
    for (x, s, d), t in trace:
        for dst in d:
            assert E._link(V100, s, dst)[0] == "link"
            assert E._link(V100, s, dst)[1] == (25.0 if len(x) == 1 else 50.0)
    # from the preamble alone: the synthesiser and the placement search give the printed membership and the printed body
    pre = E.parse(g["program"])
    pre.actions = []
    m2, q2, ms2 = E.place(pre, V100, body=lambda b: E.synthesize(b, V100, depth=0)[0])
    assert m2 == m and abs(ms2 - ms) < 1e-9
    assert set(E.expanded(q2)) == set(E.expanded(E.bind(p, m)))


def test_doubling_body_from_its_preamble_and_against_gathering():
    p = E.parse(G["doubling"]["program"])
    pre = p.copy()
    pre.actions = []
    q, ms = E.synthesize(pre, H100, depth=1, beam=4)
    assert set(E.expanded(q)) == set(E.expanded(p))
    naive = E.naive_body(pre)
    assert E.valid(naive)
    # gathering: every site multicasts to three (egress / 3), then one aggregation of four parts
    assert abs(E.simulate(naive, H100) - (3 / 450 + 5 / 3350) * 1e3) < 1e-9
    assert ms < E.simulate(naive, H100)


def test_generated_preamble_is_the_printed_one():
    g = G["preamble"]
    want = E.parse(g["program"])
    got = E.preamble(g["extents"], g["producer_splits"], {(b, c): s for b, c, s in g["copy_site"]}, g["consumer_splits"],
                     g["consumer_specs"], 4, name=lambda j, c: "XY"[c] + str(j + 1))
    assert got.gpus == want.gpus
    assert list(got.partitions) == list(want.partitions) and all(p == {"size": 1, "members": None} for p in got.partitions.values())
    assert list(got.atoms) == list(want.atoms)                                      # same atoms in the same order
    assert {a: s for a, (s, _) in got.atoms.items()} == {a: s for a, (s, _) in want.atoms.items()}
    assert got.out == want.out
    assert all(abs(gb - 64 * 256 * 4 / 1e9) < 1e-18 for _, gb in got.atoms.values())  # cardinality x width of the datatype
    # synthesis chooses S1..S4: with each aggregate placed where one of its copies already is, one transfer per atom
    m, q, ms = E.place(got, H100, body=E.naive_body)
    assert all(q.atoms[a][0] in [q.atoms[b][0] for b in x] for x, s in E.requirements(q) for a in x)
    assert sum(len(d) for _, _, d in E.expanded(q)) == 4


# ------------------------------------------------------------------------------------------ closed forms of the cost model
def test_multicast_divides_the_egress():
    for k in (1, 2, 3, 7):
        dst = ", ".join(str(i) for i in range(1, k + 1))
        p = E.parse("IN: A @ 0 (size: 2.5 GB)\nOUT: A @ %s\n\nA @ 0 -> %s\n" % (dst, dst))
        assert abs(E.simulate(p, H100) - k * 2.5 / 450 * 1e3) < 1e-9


def test_ingress_contention_and_hbm_sharing():
    p = E.parse("IN: A @ 1; B @ 2; C @ 3\nOUT: A @ 0; B @ 0; C @ 0\n\nA @ 1 -> 0; B @ 2 -> 0; C @ 3 -> 0\n")
    assert abs(E.simulate(p, H100) - 3 / 450 * 1e3) < 1e-9                           # three flows share the ingress of site 0
    p = E.parse("IN: A @ 0; B @ 0; C @ 0 (size: 2 GB); D @ 0 (size: 2 GB)\nOUT: A+B @ 0; C+D @ 0\n\nA+B @ 0; C+D @ 0\n")
    # two aggregations share the HBM: 3 GB and 6 GB of traffic; the first ends at 6/3350, the second at 9/3350
    ms, trace = E.simulate(p, H100, trace=True)
    ends = sorted(t[2] for _, t in trace)
    assert abs(ends[0] - 6 / 3350 * 1e3) < 1e-9 and abs(ends[1] - 9 / 3350 * 1e3) < 1e-9 and ms == ends[1]
    # an aggregate of m parts reads m and writes one
    for m in (2, 3, 5):
        names = [chr(65 + i) for i in range(m)]
        p = E.parse("IN: %s\nOUT: %s @ 0\n\n%s @ 0\n" % ("; ".join(n + " @ 0" for n in names), "+".join(names), "+".join(names)))
        assert abs(E.simulate(p, H100) - (m + 1) / 3350 * 1e3) < 1e-9


def test_cube_mesh_links_and_the_shared_bridge():
    def one(src, dst):
        return E.simulate(E.parse("GPUS: 0,1,2,3,4,5,6,7\nIN: A @ %d\nOUT: A @ %d\n\nA @ %d -> %d\n" % (src, dst, src, dst)), V100)
    assert abs(one(0, 4) - 1e3 / 50) < 1e-9 and abs(one(6, 2) - 1e3 / 50) < 1e-9    # pillars
    assert abs(one(0, 1) - 1e3 / 25) < 1e-9 and abs(one(5, 7) - 1e3 / 25) < 1e-9    # inside a socket
    assert abs(one(0, 5) - 1e3 / 15.75) < 1e-9                                        # no direct link
    two = E.parse("GPUS: 0,1,2,3,4,5,6,7\nIN: A @ 0; B @ 2\nOUT: A @ 5; B @ 7\n\nA @ 0 -> 5; B @ 2 -> 7\n")
    assert abs(E.simulate(two, V100) - 2e3 / 15.75) < 1e-9                            # the bridge's capacity is shared by all such transfers
    both = E.parse("GPUS: 0,1,2,3,4,5,6,7\nIN: A @ 0; B @ 4\nOUT: A @ 4; B @ 0\n\nA @ 0 -> 4; B @ 4 -> 0\n")
    assert abs(E.simulate(both, V100) - 1e3 / 50) < 1e-9                              # the two directions of a link do not contend


# ---------------------------------------------------------------------------------------- Definition "Closure; validity"
def test_exact_cover_against_brute_force():
    rng = random.Random(5)
    atoms = list("abcdef")
    for _ in range(200):
        x = frozenset(rng.sample(atoms, rng.randint(1, 6)))
        avail = [frozenset(rng.sample(atoms, rng.randint(1, 3))) for _ in range(rng.randint(0, 7))]
        got = E.exact_cover(x, avail)
        best = None
        uniq = list(set(avail))
        for r in range(1, len(uniq) + 1):
            for combo in itertools.combinations(uniq, r):
                if sum(len(c) for c in combo) == len(x) and frozenset().union(*combo) == x:
                    best = r
                    break
            if best:
                break
        assert (got is None) == (best is None)
        if got is not None:
            assert len(got) == best and frozenset().union(*got) == x and sum(len(y) for y in got) == len(x)


def test_not_well_formed_and_not_valid():
    never = E.parse("IN: A @ 0; B @ 1\nOUT: A+B @ 0\n\nA+B @ 0\n")                    # B never reaches site 0
    assert not E.well_formed(never) and not E.valid(never)
    with pytest.raises(ValueError):
        E.simulate(never, H100)
    short = E.parse("IN: A @ 0; B @ 1\nOUT: A+B @ 0, 1\n\nB @ 1 -> 0; A+B @ 0\n")    # well-formed, requirement at 1 unmet
    assert E.well_formed(short) and not E.valid(short)
    # parts must be disjoint: A+B and B+C at a site do not make A+B+C
    over = E.parse("IN: A @ 0; B @ 0; C @ 0\nOUT: A+B+C @ 0\n\nA+B @ 0; B+C @ 0; A+B+C @ 0\n")
    assert E.valid(over)                                                                # the atoms themselves partition it
    state = {(frozenset("AB"), 0), (frozenset("BC"), 0)}
    assert E.exact_cover(frozenset("ABC"), [y for y, _ in state]) is None
    for bad in ("IN: A @ 0\nOUT: A+Z @ 0\n", "IN: A @ 0; A @ 1\nOUT: A @ 0\n", "GPUS: 0, 1\nPARTITIONS: P {size 1}\nIN: A @ 0\nOUT: A @ P\n",
                "IN: A @ 0; B @ 1\nOUT: A @ 1\n\nA+B @ 0, 1 -> 1\n", "IN: A @ 0; B @ 0 (size: 2 GB)\nOUT: A+B @ 0\n"):
        with pytest.raises(ValueError):
            E.parse(bad)


def test_a_program_is_a_set_and_text_round_trips():
    a = E.parse(G["doubling"]["program"])
    lines = G["doubling"]["program"].split("\n\n", 1)
    items = [t for t in lines[1].replace("\n", ";").split(";") if t.strip()]
    random.Random(1).shuffle(items)
    b = E.parse(lines[0] + "\n\n" + ";".join(items + items[:3]) + "\n")                # shuffled, with repeats
    assert set(a.actions) == set(b.actions) and len(b.actions) == len(a.actions)
    assert E.simulate(a, H100) == E.simulate(b, H100)
    for name in ("swap", "doubling", "v100", "preamble"):
        p = E.parse(G[name]["program"])
        q = E.parse(E.format_program(p))
        assert (q.gpus, q.partitions, q.atoms, q.out, q.actions) == (p.gpus, p.partitions, p.atoms, p.out, p.actions)


def test_insert_delete_and_the_completeness_theorem():
    q_prog = E.normalised(E.parse(G["doubling"]["program"]))
    pre = q_prog.copy()
    pre.actions = []
    p_prog = E.normalised(E.naive_body(pre))
    assert E.valid_bound(p_prog) and E.valid_bound(q_prog)
    # insert Q \ P in a firing order of Q (the simulator's start times give one), then delete P \ Q latest-firing first
    _, trace = E.simulate(q_prog, H100, trace=True)
    firing = [a for a, t in sorted(trace, key=lambda at: at[1][0])]
    cur = p_prog
    n_ins = 0
    for x, s, d in firing:
        act = (x, ("sites", (s,)), d)
        if act in cur.actions:
            continue
        before = E.closure(cur)
        cur = E.insert(cur, act)
        assert cur is not None and E.valid_bound(cur) and before <= E.closure(cur)      # monotone: insertion only grows the closure
        n_ins += 1
    assert n_ins == len(set(q_prog.actions) - set(p_prog.actions))
    _, trace = E.simulate(cur, H100, trace=True)
    start = {(x, ("sites", (s,)), d): t[0] for (x, s, d), t in trace}
    for act in sorted(set(p_prog.actions) - set(q_prog.actions), key=lambda a: -start[a]):
        cur = E.delete(cur, cur.actions.index(act))
        assert cur is not None and E.valid_bound(cur)
    assert set(cur.actions) == set(q_prog.actions)
    # the guards: an insertion that is not enabled, a deletion that breaks validity
    assert E.insert(p_prog, (frozenset("AB"), ("sites", (2,)), (3,))) is not None       # enabled by the gathered atoms
    lonely = E.normalised(E.parse("IN: A @ 0; B @ 1\nOUT: A @ 0\n\n"))
    assert E.insert(lonely, (frozenset("AB"), ("sites", (0,)), ())) is None
    assert E.delete(q_prog, 0) is None


def test_rule_families_keep_validity_and_their_closures():
    p = E.normalised(E.naive_body(E.parse("IN: A @ 0; B @ 1; C @ 2; D @ 3\nOUT: A+B+C+D @ 0, 1, 2, 3\n")))
    base = E.closure(p)
    f = E.fission(p, 0, (1,))
    assert f is not None and E.closure(f) == base and len(f.actions) == len(p.actions) + 1      # closure unchanged both ways
    back = E.fusion(f, 0, len(f.actions) - 1)
    assert back is not None and E.closure(back) == base and set(back.actions) == set(p.actions)
    r = E.relay_introduction(f, 0, 1, 2)                                                          # A @ 0 -> 1 becomes A @ 0 -> 2, A @ 2 -> 1
    assert r is not None and base <= E.closure(r)
    # eager aggregation: B is at 0 after B @ 1 -> 0, ...; redirect B's copy for site 2 to come from 0, then push down
    g = E.fission(p, 0, (2,))                       # A @ 0 -> 1, 3 and A @ 0 -> 2
    g = E.fission(g, 1, (2,))                       # B @ 1 -> 0, 3 and B @ 1 -> 2
    i_a = g.actions.index((frozenset("A"), ("sites", (0,)), (2,)))
    i_b = g.actions.index((frozenset("B"), ("sites", (1,)), (2,)))
    g2 = E.source_substitution(g, i_b, 0)
    assert g2 is not None
    g3 = E.pushdown(g2, min(i_a, i_b), max(i_a, i_b))
    assert g3 is not None and (frozenset("AB"), ("sites", (0,)), (2,)) in g3.actions
    assert (frozenset("A"), 2) not in E.closure(g3) and (frozenset("AB"), 2) in E.closure(g3)     # pushdown deletes the separate materialisations
    up = E.pullup(g3, g3.actions.index((frozenset("AB"), ("sites", (0,)), (2,))), ("A",))
    assert up is not None and (frozenset("A"), 2) in E.closure(up) and (frozenset("AB"), 2) in E.closure(up)
    # guards: substitution from a site that never holds X; relay elimination when the relay's copy is required
    assert E.source_substitution(g, i_b, 3) is not None                                            # B does reach 3
    assert E.source_substitution(E.normalised(E.parse(G["swap"]["program"])), 0, 1) is None
    need = E.normalised(E.parse("IN: A @ 0\nOUT: A @ 1, 2\n\nA @ 0 -> 1; A @ 1 -> 2\n"))
    assert E.relay_elimination(need, 0, 1) is None                                                 # A at 1 is itself required
    free = E.normalised(E.parse("IN: A @ 0\nOUT: A @ 2\n\nA @ 0 -> 1; A @ 1 -> 2\n"))
    el = E.relay_elimination(free, 0, 1)
    assert el is not None and el.actions == [(frozenset("A"), ("sites", (0,)), (2,))]
    # random walks through the neighbourhood never leave the valid programs, and the search never returns a slower one
    rng = random.Random(3)
    cur = p
    for _ in range(12):
        nb = E.neighbours(cur)
        assert nb and all(E.valid_bound(q) for q in nb)
        cur = rng.choice(nb)
    q, ms = E.synthesize(cur, H100, depth=2, beam=6)
    assert E.valid_bound(q) and ms <= E.simulate(cur, H100) * (1 + 1e-12)


def test_executing_any_valid_program_gives_the_aggregate_of_all_copies():
    """The oracle's executor (decompose, fire the actions, recompose) against the plain definition it must reach: the
    consumer's tensor is the (+)-aggregate of the m copies, whatever the program's route (oracle/blocked.py
    aggregate_repartition, itself pinned to the preamble example and to brute force)."""
    import numpy as np

    from oracle import blocked
    rng = np.random.default_rng(4)
    mo = E.machine("dgx_h100")
    cases = [
        ([256, 256], [[0, 128, 256], [0, 256]], [[0, 64, 128, 192, 256], [0, 256]], 2, [0, 1, 2, 3], [0, 1, 2, 3]),
        ([6, 33, 10], [[0, 3, 6], [0, 10, 33], [0, 10]], [[0, 6], [0, 33], [0, 3, 10]], 3, [0, 1, 2, 2, 0, 1, 1, 2, 0, 0, 2, 1], [0, 1, 1]),
        ([128, 64], [[0, 128], [0, 64]], [[0, 128], [0, 64]], 4, [0, 1, 2, 3], [0, 0, 0, 0]),
    ]
    for ext, ps, cs, m, sites, specs in cases:
        pre = E.preamble(ext, ps, {(b, c): sites[b * m + c] for b in range(len(sites) // m) for c in range(m)}, cs, specs, 4)
        P = rng.standard_normal([m] + ext)
        for body in (E.naive_body, E.butterfly_body, lambda b: E.synthesize(b, mo, depth=2, beam=5)[0]):
            _, q, _ = E.place(pre, mo, body=body)
            for agg in ("sum", "max"):
                out = E.exchange(q, P, ps, cs, specs, agg)
                ref = blocked.aggregate_repartition(P, ps, cs, agg)
                assert np.abs(out - ref).max() <= (1e-12 if agg == "sum" else 0.0)
        # a rewritten program: the walk changes the aggregation trees, not the result
        rnd = random.Random(7)
        _, cur, _ = E.place(pre, mo, body=E.naive_body)
        cur = E.normalised(cur)
        for _ in range(6):
            cur = rnd.choice(E.neighbours(cur))
        assert np.abs(E.exchange(cur, P, ps, cs, specs, "sum") - blocked.aggregate_repartition(P, ps, cs, "sum")).max() <= 1e-12
    # the schedule fires every action once, in an order in which each is enabled
    q = E.parse(G["doubling"]["program"])
    sched = E.schedule(q)
    assert len(sched) == len(E.expanded(q))
    assert [len(c) for x, s, d, c in sched if len(x) == 4] == [2, 2, 2, 2]          # A+B and C+D, not four atoms
