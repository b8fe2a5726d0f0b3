"""Physical optimization in miniature (paper_2609_03905_b200/physical.py): the preamble arguments derived from two
planned operators against the paper's worked example, and the naive-against-optimised comparison of Section 6,
Experiment 4 on the library's simulator.  Host only."""
import json
import os

import paper_2609_03905_b200 as ja
from oracle import exprog as E
from paper_2609_03905_b200 import exprog as X, physical
from paper_2609_03905_b200.planned_block import block_graph

G = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "exprog_examples.json")))


def test_edge_of_the_papers_preamble_example():
    """Section 5.3: the four-spec matmul of Example 3.8 (i and j cut in two; F_11, F_12, F_21, F_22 on GPUs 0..3) feeding a
    row-wise softmax cut into four row intervals."""
    ops = [{"einsum": "ij,jk->ik", "extents": {"i": 256, "j": 512, "k": 256}, "inputs": [None, None]},
           {"einsum": "ik->ik", "extents": {"i": 256, "k": 256}, "inputs": [0]}]
    plan = [{"i": 2, "j": 2, "k": 1}, {"i": 4, "k": 1}]
    a = physical.edge(ops, plan, 1, 0, [0, 1, 2, 3], width_bytes=4)
    g = G["preamble"]
    assert a["producer_splits"] == g["producer_splits"] and a["consumer_splits"] == g["consumer_splits"]
    assert a["m"] == 2 and a["consumer_specs"] == g["consumer_specs"]
    assert a["copy_site"] == [s for _, _, s in sorted(map(tuple, g["copy_site"]))]
    h = X.ExchangeProgram(handle=X.ja_exprog_preamble(a["producer_splits"], a["consumer_splits"], a["m"], a["copy_site"],
                                                      a["consumer_specs"], a["width_bytes"]))
    text = str(h)
    for j in range(4):
        text = text.replace("a%d_0" % j, "X%d" % (j + 1)).replace("a%d_1" % j, "Y%d" % (j + 1))
    got, want = E.parse(text), E.parse(g["program"])
    assert list(got.atoms) == list(want.atoms) and got.out == want.out
    assert {k: v[0] for k, v in got.atoms.items()} == {k: v[0] for k, v in want.atoms.items()}


def test_naive_against_optimised_exchanges_of_a_planned_block():
    ops = block_graph(8, 256, 512, 8, 1024)
    cost, plan = ja.ja_plan_optimize_graph(ops, 8)
    out = {}
    for name in ("dgx_a100", "dgx_v100"):
        mach = X.ja_machine_preset(name)
        naive, en = physical.compile_exchanges(ops, plan, mach, False)
        opt, eo = physical.compile_exchanges(ops, plan, mach, True, depth=1, beam=4)
        assert len(en) == len(eo) == sum(1 for op in ops if any(i is not None for i in op["inputs"]))
        assert opt <= naive * (1 + 1e-12)                       # the naive program is in the search space
        # one program per operator runs its operands' exchanges at the same time: never slower than one after the other
        naive_sep, en_sep = physical.compile_exchanges(ops, plan, mach, False, joint=False)
        assert naive <= naive_sep * (1 + 1e-12)
        assert all(e["programs"] == 1 for e in en) and any(e["programs"] > 1 for e in en_sep)
        # operators whose producers and they agree on tiling and placement, with one copy and nothing replicated, move nothing
        for e in en_sep:
            j = e["consumer"]
            quiet = all(m == 1 for m in e["m"])
            for k in e["operands"]:
                i = ops[j]["inputs"][k]
                quiet = quiet and tuple(plan[i][c] for c in op_out(ops[i])) == tuple(plan[j][c] for c in op_in(ops[j], k))
                quiet = quiet and not any(c not in op_in(ops[j], k) and plan[j][c] > 1 for c in letters(ops[j]))
            assert not quiet or e["ms"] == 0.0
        out[name] = naive / opt if opt > 0 else 1.0
    assert out["dgx_a100"] < 1.02                               # nothing to exploit on a non-blocking fabric
    assert out["dgx_v100"] >= out["dgx_a100"] - 1e-12


def letters(op):
    return physical._terms(op["einsum"])[2]


def op_out(op):
    return physical._terms(op["einsum"])[1]


def op_in(op, k):
    return physical._terms(op["einsum"])[0][k]


def test_swap_descent_placement_matches_the_oracle_and_enumeration():
    # eight partitions of size one: 40320 memberships, searched by exchanges of two sites
    a = physical.edge([{"einsum": "ij,jk->ik", "extents": {"i": 512, "j": 512, "k": 512}, "inputs": [None, None]},
                       {"einsum": "ik,kl->il", "extents": {"i": 512, "k": 512, "l": 512}, "inputs": [0, None]}],
                      [{"i": 2, "j": 4, "k": 1}, {"i": 1, "k": 8, "l": 1}], 1, 0, [3, 6, 1, 4, 7, 2, 5, 0])
    for name in ("dgx_v100", "dgx_h100"):
        h = X.ExchangeProgram(handle=X.ja_exprog_preamble(a["producer_splits"], a["consumer_splits"], a["m"], a["copy_site"],
                                                          a["consumer_specs"], a["width_bytes"]))
        assert X.ja_exprog_num_memberships(h.handle) == 40320
        pre = E.parse(str(h))
        ms = X.ja_exprog_place(h.handle, X.ja_machine_preset(name), "best")
        mo = E.machine(name)
        mem, q, ms_o = E.place(pre, mo, body=lambda b: E.synthesize(b, mo, depth=0)[0])
        assert abs(ms - ms_o) <= 1e-9 * ms_o
        assert {n: X.ja_exprog_membership(h.handle, n) for n in mem} == {n: sum(1 << s for s in v) for n, v in mem.items()}
        assert X.ja_exprog_check(h.handle) == (True, True)
        # never worse than where the descent started (function spec i on GPU i)
        g = X.ExchangeProgram(str(E.format_program(pre)))
        for i in range(8):
            X.ja_exprog_bind_members(g.handle, "S%d" % (i + 1), [i])
        X.ja_exprog_body(g.handle, "naive")
        assert ms <= X.ja_exprog_simulate(g.handle, X.ja_machine_preset(name)) * (1 + 1e-12)
    # on a small case the descent's answer costs what full enumeration finds
    small = "GPUS: 0, 1, 2, 3\nPARTITIONS: S1 {size 1} S2 {size 1} S3 {size 1} S4 {size 1}\nIN: A @ 0; B @ 1; C @ 2; D @ 3\nOUT: A+B @ S3; C+D @ S1; A @ S2; D @ S4\n"
    p = E.parse(small)
    mo = E.machine("dgx_v100")
    full = E.place(p, mo, body=E.naive_body)
    desc = E.place(p, mo, body=E.naive_body, enumeration_limit=0)
    assert desc[2] >= full[2] * (1 - 1e-12)                      # enumeration is exact; descent may stop in a local minimum
    assert E.valid_bound(desc[1])


def test_the_plan_for_one_long_sequence_is_the_one_the_paper_reports():
    """Section 6, Experiment 1: for the 1 x 128K workload the optimizer "discovers" the DeepSpeed-Ulysses decomposition --
    tokens sharded everywhere outside attention, heads sharded inside it, a repartition at the boundary.  With the sequence
    index of attention not shardable inside one sequence (Example 3.10) the library's optimizer and the oracle's both return
    exactly that for eight processors, and the four boundary exchanges are all-to-alls."""
    from oracle import optimizer as O
    from paper_2609_03905_b200.planned_block import plan_repartition_charges
    ops = block_graph(1, 131072, 4096, 32, 14336)
    ops[4] = dict(ops[4], fixed={"d", "q", "k"})
    cost, plan = ja.ja_plan_optimize_graph(ops, 8)
    for j, counts in enumerate(plan):
        cut = {k: v for k, v in counts.items() if v > 1}
        assert cut == ({"h": 8} if j == 4 else {"s": 8}), (j, cut)
    assert plan_repartition_charges(ops, plan)[0] == 4                     # q, k, v into attention, its output back
    cost_o, plan_o = O.optimize_graph(ops, 8)
    assert cost_o == cost and [dict(p) for p in plan_o] == [dict(p) for p in plan]
    mach = X.ja_machine_preset("dgx_a100")
    total, recs = physical.compile_exchanges(ops, plan, mach, True, depth=0)
    moving = [r for r in recs if r["ms"] > 0]
    assert [r["consumer"] for r in moving] == [4, 5]                       # attention (q, k, v as one program) and the output projection
    # an all-to-all: every GPU sends 7/8 of its eighth of each tensor, one eighth to each other GPU, at full egress
    eighth_gb = 131072 * 4096 * 2 / 8 / 1e9
    assert abs(moving[1]["ms"] - 7 / 8 * eighth_gb / 300 * 1e3) < 1e-6
    assert abs(moving[0]["ms"] - 3 * 7 / 8 * eighth_gb / 300 * 1e3) < 1e-6  # q, k and v together share the endpoints
