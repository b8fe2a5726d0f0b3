"""The library's exchange-program host code (include/ja_exprog.h) against the oracle (oracle/exprog.py): parsed
programs, closures, validity verdicts, memberships and expanded actions are compared exactly, simulated times to 1e-9
relative.  No CUDA call is made here."""
import json
import os
import random

import pytest

from oracle import exprog as E
from paper_2609_03905_b200 import exprog as X

G = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "exprog_examples.json")))
MACHINES = ["dgx_h100", "dgx_a100", "hgx_b200", "dgx_v100"]


def masks(prog):
    order = {a: i for i, a in enumerate(prog.atoms)}
    return lambda x: sum(1 << order[a] for a in x)


def sites_mask(d):
    return sum(1 << s for s in d)


def same_program(handle, oracle_prog):
    """The library's program, read back through its text, is the oracle's."""
    q = E.parse(X.ja_exprog_format(handle))
    assert q.gpus == oracle_prog.gpus and q.partitions == oracle_prog.partitions
    assert q.atoms == oracle_prog.atoms and q.out == oracle_prog.out and q.actions == oracle_prog.actions


def close(a, b):
    return abs(a - b) <= 1e-9 * max(1.0, abs(b))


@pytest.mark.parametrize("name", ["swap", "doubling", "v100", "preamble"])
def test_parse_and_format_agree_with_the_oracle(name):
    text = G[name]["program"]
    p = E.parse(text)
    h = X.ExchangeProgram(text)
    same_program(h.handle, p)
    c = X.ja_exprog_counts(h.handle)
    assert (c["gpus"], c["partitions"], c["atoms"], c["out"], c["actions"]) == (
        len(p.gpus), len(p.partitions), len(p.atoms), len(p.out), len(p.actions))
    assert X.ja_exprog_get_atoms(h.handle) == list(p.atoms.values())
    assert X.ja_exprog_num_memberships(h.handle) == len(list(E.memberships(p)))
    assert X.ja_exprog_valid_any(h.handle) == E.valid(p)


def test_sizes_round_trip_through_text():
    text = "IN: A @ 0 (size: 0.0001 GB); B @ 1 (size: 0.0001 GB); C @ 2 (size: 2.5e-07 GB); D @ 0 (size: 12 GB)\nOUT: A+B @ 0; C @ 1; D @ 2\n"
    h = X.ExchangeProgram(text)
    same_program(h.handle, E.parse(text))
    assert [gb for _, gb in X.ja_exprog_get_atoms(h.handle)] == [0.0001, 0.0001, 2.5e-07, 12.0]


@pytest.mark.parametrize("bad,status", [
    ("IN: A @ 0\nOUT: A+Z @ 0\n", "JA_ERR_PARSE"), ("IN: A @ 0; A @ 1\nOUT: A @ 0\n", "JA_ERR_PARSE"),
    ("IN: A @ 0\n", "JA_ERR_PARSE"), ("IN: A @ 0; B @ 1\nOUT: A @ 1\n\nA+B @ 0, 1 -> 1\n", "JA_ERR_PARSE"),
    ("GPUS: 0, 1\nPARTITIONS: P {size 1}\nIN: A @ 0\nOUT: A @ P\n", "JA_ERR_INVALID_ARG"),
    ("GPUS: 0, 1\nPARTITIONS: P {0, 1} Q {1}\nIN: A @ 0\nOUT: A @ P\n", "JA_ERR_INVALID_ARG"),
    ("GPUS: 0, 1\nIN: A @ 2\nOUT: A @ 0\n", "JA_ERR_INVALID_ARG"),
    ("IN: A @ 0; B @ 0 (size: 2 GB)\nOUT: A+B @ 0\n", "JA_ERR_INVALID_ARG"),
    ("GPUS: 0, 1\nIN: A @ 0\nOUT: A @ 1\n\nA @ 0 -> 1, 70\n", "JA_ERR_INVALID_ARG"),
    ("GPUS: 0, 1\nIN: A @ 0\nOUT: A @ 2\n", "JA_ERR_INVALID_ARG"),
    ("GPUS: 0, 1\nIN: A @ 0; B @ 0 (size: 3 GB)\nOUT: A @ 1\n\nA+B @ 0 -> 1\n", "JA_ERR_INVALID_ARG"),
])
def test_malformed_programs_are_refused(bad, status):
    from paper_2609_03905_b200.binding import JaError
    with pytest.raises(JaError) as e:
        X.ja_exprog_parse(bad)
    assert e.value.status_name == status
    with pytest.raises(ValueError):
        E.parse(bad)


def test_the_interface_limits_of_the_library():
    from paper_2609_03905_b200.binding import JaError
    with pytest.raises(JaError) as e:                      # site masks are 64 bits wide
        X.ja_exprog_parse("IN: A @ 64\nOUT: A @ 64\n")
    assert e.value.status_name == "JA_ERR_INVALID_ARG"
    many = "IN: " + "; ".join("a%d @ 0" % i for i in range(65)) + "\nOUT: a0 @ 0\n"
    with pytest.raises(JaError) as e:                      # aggregate masks too
        X.ja_exprog_parse(many)
    assert e.value.status_name == "JA_ERR_INVALID_ARG"
    ok = X.ExchangeProgram("IN: " + "; ".join("a%d @ %d" % (i, i) for i in range(64)) + "\nOUT: " + "+".join("a%d" % i for i in range(64)) + " @ 63\n")
    X.ja_exprog_body(ok.handle, "naive")
    assert X.ja_exprog_check(ok.handle) == (True, True)
    assert abs(X.ja_exprog_simulate(ok.handle, X.ja_machine_preset("dgx_h100")) - (63 / 450 + 65 / 3350) * 1e3) < 1e-6


def test_membership_spaces_too_large_to_list():
    from paper_2609_03905_b200.binding import JaError
    n = 12
    text = ("GPUS: " + ", ".join(str(i) for i in range(n)) + "\nPARTITIONS: " + " ".join("S%d {size 1}" % i for i in range(n)) +
            "\nIN: " + "; ".join("a%d @ %d" % (i, i) for i in range(n)) + "\nOUT: " + "; ".join("a%d @ S%d" % (i, (i + 1) % n) for i in range(n)) + "\n")
    h = X.ExchangeProgram(text)
    import math
    assert X.ja_exprog_num_memberships(h.handle) == math.factorial(n)         # counted, not listed
    for call in (lambda: X.ja_exprog_bind(h.handle, 5), lambda: X.ja_exprog_valid_any(h.handle)):
        with pytest.raises(JaError) as e:
            call()
        assert e.value.status_name == "JA_ERR_UNSUPPORTED"
    ms = X.ja_exprog_place(h.handle, X.ja_machine_preset("dgx_h100"), "naive")   # the swap descent still places it
    assert X.ja_exprog_check(h.handle) == (True, True) and ms == 0.0             # every atom's requirement put where the atom is


def library_state(handle):
    return set(X.ja_exprog_closure(handle))


def oracle_state(prog):
    mk = masks(prog)
    return {(mk(x), s) for x, s in E.closure(prog)}


def test_memberships_closure_validity_and_actions_on_every_membership_of_the_v100_example():
    p = E.parse(G["v100"]["program"])
    base = X.ExchangeProgram(G["v100"]["program"])
    n_valid = 0
    for k, mem in enumerate(E.memberships(p)):
        h = base.clone()
        X.ja_exprog_bind(h.handle, k)
        q = E.bind(p, mem)
        for name, members in mem.items():
            assert X.ja_exprog_membership(h.handle, name) == sites_mask(members)
        same_program(h.handle, q)
        mk = masks(q)
        assert X.ja_exprog_get_actions(h.handle) == [(mk(x), s, sites_mask(d)) for x, s, d in E.expanded(q)]
        assert X.ja_exprog_get_requirements(h.handle) == [(mk(x), s) for x, s in E.requirements(q)]
        assert library_state(h.handle) == oracle_state(q)
        assert X.ja_exprog_check(h.handle) == (E.well_formed(q), E.valid_bound(q))
        n_valid += E.valid_bound(q)
    assert n_valid == 1
    from paper_2609_03905_b200.binding import JaError
    with pytest.raises(JaError):
        X.ja_exprog_check(base.handle)                  # memberships not bound yet
    with pytest.raises(JaError):
        X.ja_exprog_bind(base.handle, 70)


@pytest.mark.parametrize("machine", MACHINES)
def test_simulator_against_the_oracle_on_the_examples_and_their_naive_bodies(machine):
    m, mo = X.ja_machine_preset(machine), E.machine(machine)
    assert (m.hbm_gbs, m.link_gbs if mo["kind"] == "nvswitch" else m.pcie_gbs) == (
        mo["hbm"], mo["link"] if mo["kind"] == "nvswitch" else mo["pcie"])
    for name in ("swap", "doubling", "v100"):
        p = E.parse(G[name]["program"])
        mem = next(mm for mm in E.memberships(p) if E.valid_bound(E.bind(p, mm)))
        k = list(E.memberships(p)).index(mem)
        for body in ("own", "naive", "butterfly"):
            q = E.bind(p, mem)
            h = X.ExchangeProgram(G[name]["program"])
            X.ja_exprog_bind(h.handle, k)
            if body == "naive":
                q = E.naive_body(q)
            elif body == "butterfly":
                q = E.butterfly_body(q)
            X.ja_exprog_body(h.handle, body)
            same_program(h.handle, q)
            ms, trace = E.simulate(q, mo, trace=True)
            got, times = X.ja_exprog_simulate(h.handle, m, trace=True)
            assert close(got, ms)
            for (_, want), have in zip(trace, times):
                assert all(close(a, b) for a, b in zip(have, want))


def test_printed_times_through_the_library():
    for name in ("swap", "doubling"):
        h = X.ExchangeProgram(G[name]["program"])
        assert round(X.ja_exprog_simulate(h.handle, X.ja_machine_preset(G[name]["machine"])), 1) == G[name]["completion_ms"]
    h = X.ExchangeProgram(G["v100"]["program"])
    ms = X.ja_exprog_place(h.handle, X.ja_machine_preset("dgx_v100"), "own")
    assert round(ms) == G["v100"]["completion_ms"]
    for name, members in G["v100"]["membership"].items():
        assert X.ja_exprog_membership(h.handle, name) == sites_mask(members)
    # from the preamble alone
    pre = G["v100"]["program"].split("\n\n")[0] + "\n"
    h2 = X.ExchangeProgram(pre)
    ms2 = X.ja_exprog_place(h2.handle, X.ja_machine_preset("dgx_v100"), "best")
    assert close(ms2, ms)
    assert set(X.ja_exprog_get_actions(h2.handle)) == set(X.ja_exprog_get_actions(h.handle))
    p = E.parse(pre)
    mo = E.machine("dgx_v100")
    mem, q, ms_o = E.place(p, mo, body=lambda b: E.synthesize(b, mo, depth=0)[0])
    assert close(ms2, ms_o)
    mk = masks(q)
    assert set(X.ja_exprog_get_actions(h2.handle)) == {(mk(x), s, sites_mask(d)) for x, s, d in E.expanded(q)}


def test_random_programs_closure_check_and_simulation():
    rng = random.Random(11)
    names = list("ABCDEF")
    n_sim = 0
    for trial in range(60):
        n_sites = rng.randint(2, 5)
        atoms = names[:rng.randint(2, 6)]
        text = "GPUS: " + ", ".join(str(s) for s in range(n_sites)) + "\nIN: " + "; ".join(
            "%s @ %d" % (a, rng.randrange(n_sites)) for a in atoms)
        out = []
        for _ in range(rng.randint(1, 3)):
            x = rng.sample(atoms, rng.randint(1, len(atoms)))
            out.append("+".join(x) + " @ " + ", ".join(str(s) for s in sorted(rng.sample(range(n_sites), rng.randint(1, n_sites)))))
        text += "\nOUT: " + "; ".join(out) + "\n\n"
        acts = []
        for _ in range(rng.randint(0, 9)):
            x = rng.sample(atoms, rng.randint(1, min(3, len(atoms))))
            s = rng.randrange(n_sites)
            d = sorted(rng.sample([t for t in range(n_sites) if t != s], rng.randint(0, min(2, n_sites - 1))))
            acts.append("+".join(x) + " @ %d" % s + (" -> " + ", ".join(str(t) for t in d) if d else ""))
        text += "\n".join(acts) + "\n"
        p = E.parse(text)
        h = X.ExchangeProgram(text)
        same_program(h.handle, p)
        assert library_state(h.handle) == oracle_state(p)
        wf, v = X.ja_exprog_check(h.handle)
        assert (wf, v) == (E.well_formed(p), E.valid_bound(p))
        for machine in ("dgx_h100", "dgx_v100") if n_sites <= 5 else ("dgx_h100",):
            m, mo = X.ja_machine_preset(machine), E.machine(machine)
            if wf:
                assert close(X.ja_exprog_simulate(h.handle, m), E.simulate(p, mo))
                n_sim += 1
            else:
                from paper_2609_03905_b200.binding import JaError
                with pytest.raises(JaError):
                    X.ja_exprog_simulate(h.handle, m)
        # the naive body always satisfies OUT
        X.ja_exprog_body(h.handle, "naive")
        q = E.naive_body(p)
        same_program(h.handle, q)
        assert X.ja_exprog_check(h.handle) == (True, True) and E.valid_bound(q)
        assert close(X.ja_exprog_simulate(h.handle, X.ja_machine_preset("dgx_a100")), E.simulate(q, E.machine("dgx_a100")))
    assert n_sim > 20


def test_rules_against_the_oracle():
    text = "IN: A @ 0; B @ 1; C @ 2; D @ 3\nOUT: A+B+C+D @ 0, 1, 2, 3\n"
    p = E.normalised(E.naive_body(E.parse(text)))
    h = X.ExchangeProgram(text)
    X.ja_exprog_body(h.handle, "naive")
    X.ja_exprog_normalise(h.handle)
    same_program(h.handle, p)
    mk = masks(p)

    def step(rule, oracle_result, *args, **kw):
        nonlocal p
        applied = X.ja_exprog_rewrite(h.handle, rule, *args, **kw)
        assert applied == (oracle_result is not None)
        if applied:
            p = oracle_result
        same_program(h.handle, p)

    step("fission", E.fission(p, 0, (2,)), 0, a=1 << 2)                     # A @ 0 -> 1, 3 | A @ 0 -> 2
    step("fission", E.fission(p, 1, (2,)), 1, a=1 << 2)                     # B @ 1 -> 0, 3 | B @ 1 -> 2
    i_a = p.actions.index((frozenset("A"), ("sites", (0,)), (2,)))
    i_b = p.actions.index((frozenset("B"), ("sites", (1,)), (2,)))
    step("source", E.source_substitution(p, i_b, 0), i_b, 0)
    step("source", E.source_substitution(p, i_b, 0), i_b, 0)                  # already there: refused by both
    step("pushdown", E.pushdown(p, min(i_a, i_b), max(i_a, i_b)), min(i_a, i_b), max(i_a, i_b))
    i_ab = p.actions.index((frozenset("AB"), ("sites", (0,)), (2,)))
    step("relay_in", E.relay_introduction(p, i_ab, 2, 3), i_ab, 2, a=3)
    step("pullup", E.pullup(p, i_ab, ("A",)), i_ab, a=mk("A"), b=1)
    step("delete", E.delete(p, 0), 0)                                         # breaks validity: refused
    step("insert", E.insert(p, (frozenset("CD"), ("sites", (3,)), (0,))), 3, a=mk("CD"), b=1 << 0)
    step("insert", E.insert(p, (frozenset("AC"), ("sites", (1,)), ())), 1, a=mk("AC"), b=0)
    step("delete", E.delete(p, len(p.actions) - 1), len(p.actions) - 1)
    step("fusion", E.fusion(p, 0, 1), 0, 1)
    wf, v = X.ja_exprog_check(h.handle)
    assert wf and v and E.valid_bound(p)
    for m_name in ("dgx_h100", "dgx_v100"):
        assert close(X.ja_exprog_simulate(h.handle, X.ja_machine_preset(m_name)), E.simulate(p, E.machine(m_name)))
    # relay elimination and its guard
    for txt, want in (("IN: A @ 0\nOUT: A @ 1, 2\n\nA @ 0 -> 1; A @ 1 -> 2\n", False), ("IN: A @ 0\nOUT: A @ 2\n\nA @ 0 -> 1; A @ 1 -> 2\n", True)):
        g = X.ExchangeProgram(txt)
        X.ja_exprog_normalise(g.handle)
        assert X.ja_exprog_rewrite(g.handle, "relay_out", 0, 1) == want
        assert (E.relay_elimination(E.normalised(E.parse(txt)), 0, 1) is not None) == want


def test_synthesis_stays_valid_and_matches_the_oracle_on_the_doubling_preamble():
    pre = G["doubling"]["program"].split("\n\n")[0] + "\n"
    m, mo = X.ja_machine_preset("dgx_h100"), E.machine("dgx_h100")
    h = X.ExchangeProgram(pre)
    ms = X.ja_exprog_synthesize(h.handle, m, 1, 4)
    q, ms_o = E.synthesize(E.parse(pre), mo, depth=1, beam=4)
    assert close(ms, ms_o) and round(ms, 1) == G["doubling"]["completion_ms"]
    same_program(h.handle, q)
    # from a worse starting body: never slower than where it started, always valid
    g = X.ExchangeProgram(pre)
    X.ja_exprog_body(g.handle, "naive")
    t0 = X.ja_exprog_simulate(g.handle, m)
    t1 = X.ja_exprog_synthesize(g.handle, m, 2, 6)
    assert t1 <= t0 * (1 + 1e-12) and X.ja_exprog_check(g.handle) == (True, True)
    q0 = E.naive_body(E.parse(pre))
    q1, t1_o = E.synthesize(q0, mo, depth=2, beam=6)
    assert close(t1, t1_o)


def test_generated_preamble_against_the_oracle_and_the_paper():
    g = G["preamble"]
    m = 2
    copy_site = [s for _, _, s in sorted(map(tuple, g["copy_site"]))]
    h = X.ExchangeProgram(handle=X.ja_exprog_preamble(g["producer_splits"], g["consumer_splits"], m, copy_site, g["consumer_specs"], 4))
    want = E.preamble(g["extents"], g["producer_splits"], {(b, c): s for b, c, s in g["copy_site"]}, g["consumer_splits"],
                      g["consumer_specs"], 4)
    same_program(h.handle, want)
    # and, renamed a<j>_<c> -> X/Y<j+1>, the preamble the paper prints
    printed = E.parse(g["program"])
    text = X.ja_exprog_format(h.handle)
    for j in range(4):
        text = text.replace("a%d_0" % j, "X%d" % (j + 1)).replace("a%d_1" % j, "Y%d" % (j + 1))
    got = E.parse(text)
    assert list(got.atoms) == list(printed.atoms) and got.out == printed.out and got.partitions == printed.partitions
    assert {a: s for a, (s, _) in got.atoms.items()} == {a: s for a, (s, _) in printed.atoms.items()}
    # a second case: a 2-D overlay, three copies, seeded sites
    rng = random.Random(2)
    ps, cs = [[0, 96, 256], [0, 128, 256]], [[0, 64, 128, 256], [0, 256]]
    sites = [rng.randrange(3) for _ in range(4 * 3)]
    h2 = X.ExchangeProgram(handle=X.ja_exprog_preamble(ps, cs, 3, sites, [0, 1, 2], 2))
    want2 = E.preamble([256, 256], ps, {(b, c): sites[b * 3 + c] for b in range(4) for c in range(3)}, cs, [0, 1, 2], 2)
    same_program(h2.handle, want2)
    ms = X.ja_exprog_place(h2.handle, X.ja_machine_preset("hgx_b200"), "best")
    mo = E.machine("hgx_b200")
    _, _, ms_o = E.place(want2, mo, body=lambda b: E.synthesize(b, mo, depth=0)[0])
    assert close(ms, ms_o)


def test_firing_order_against_the_oracle():
    rng = random.Random(23)
    texts = [G[n]["program"] for n in ("swap", "doubling")]
    for _ in range(25):
        n_sites = rng.randint(2, 4)
        atoms = list("ABCDE")[:rng.randint(2, 5)]
        t = "GPUS: " + ", ".join(str(s) for s in range(n_sites)) + "\nIN: " + "; ".join("%s @ %d" % (a, rng.randrange(n_sites)) for a in atoms)
        t += "\nOUT: " + "+".join(atoms) + " @ " + ", ".join(str(s) for s in range(n_sites)) + "\n"
        texts.append(t)
    for t in texts:
        h = X.ExchangeProgram(t)
        p = E.parse(t)
        if not p.actions:
            X.ja_exprog_body(h.handle, "naive")
            X.ja_exprog_normalise(h.handle)
            p = E.normalised(E.naive_body(p))
            for _ in range(4):                                   # a few rewrites so that aggregation trees differ
                nb = E.neighbours(p)
                if nb:
                    p = rng.choice(nb)
            h = X.ExchangeProgram(E.format_program(p))
        mk = masks(p)
        acts = E.expanded(p)
        want = [(acts.index((x, s, d)), [mk(y) for y in cover]) for x, s, d, cover in E.schedule(p)]
        assert X.ja_exprog_schedule(h.handle) == want
    from paper_2609_03905_b200.binding import JaError
    never = X.ExchangeProgram("IN: A @ 0; B @ 1\nOUT: A+B @ 0\n\nA+B @ 0\n")       # kept alive: the handle dies with the object
    with pytest.raises(JaError):
        X.ja_exprog_schedule(never.handle)


def test_parser_fuzz_agrees_with_the_oracle_and_never_crashes():
    from paper_2609_03905_b200.binding import JaError
    rng = random.Random(77)
    tokens = ["IN:", "OUT:", "GPUS:", "PARTITIONS:", "A", "B", "C", "G1", "G2", "@", "->", "+", ";", ",", "\n", "\n\n", " ", "0", "1", "2", "3",
              "{", "}", "size", "(size:", "GB)", "1.5", "(", ")", ":", "x9", "70", "-1", "A+B", "A @ 0", "B @ 1", "OUT: A+B @ 0, 1", "IN: A @ 0; B @ 1"]
    accepted = 0
    for _ in range(1500):
        text = "".join(rng.choice(tokens) + rng.choice(["", " ", " "]) for _ in range(rng.randint(1, 25)))
        try:
            p = E.parse(text)
            ok_o = True
        except Exception:
            ok_o = False
        try:
            h = X.ExchangeProgram(text)
            ok_l = True
        except JaError:
            ok_l = False
        if ok_o and ok_l:
            accepted += 1
            same_program(h.handle, p)
        # the two parsers may differ on malformed text only in WHICH of them is stricter; neither may accept what the other
        # reads as a different program, which same_program above checks whenever both accept
    assert accepted > 5
    # mutations of the paper's printed programs: a token dropped, doubled or replaced
    both = 0
    for _ in range(1500):
        base = G[rng.choice(["swap", "doubling", "v100", "preamble"])]["program"]
        parts = base.replace("\n", " \n ").split(" ")
        for _ in range(rng.randint(1, 3)):
            i = rng.randrange(len(parts))
            k = rng.random()
            if k < 0.4:
                del parts[i]
            elif k < 0.7:
                parts.insert(i, parts[i])
            else:
                parts[i] = rng.choice(tokens)
        text = " ".join(parts).replace(" \n ", "\n")
        try:
            p = E.parse(text)
        except Exception:
            p = None
        try:
            h = X.ExchangeProgram(text)
        except JaError:
            h = None
        if p is not None and h is not None:
            both += 1
            same_program(h.handle, p)
            if not p.partitions or all(q["members"] is not None for q in p.partitions.values()):
                assert X.ja_exprog_check(h.handle) == (E.well_formed(p), E.valid_bound(p))
    assert both > 100


def test_candidate_bodies_are_filtered_by_validity_and_ranked_by_the_simulator():
    pre, printed_body = G["doubling"]["program"].split("\n\n", 1)
    gather = "A @ 0 -> 1, 2, 3; B @ 1 -> 0, 2, 3; C @ 2 -> 0, 1, 3; D @ 3 -> 0, 1, 2; A+B+C+D @ 0, 1, 2, 3"
    bodies = ["A+B @ 0 -> 1",                                  # not enabled: B never reaches site 0
              gather,
              "A @ 0 -> 1; B @ 1 -> 0; A+B+C+D @ 0",            # not well-formed either
              printed_body,
              "A @ 0 -> 9",                                     # names an undeclared site
              gather.replace("A+B+C+D @ 0, 1, 2, 3", "A+B+C+D @ 0, 1, 2")]   # well-formed, a requirement unmet
    best, ms, verdicts = X.best_valid_body(pre, bodies, X.ja_machine_preset("dgx_h100"))
    assert best == 3 and round(ms, 1) == G["doubling"]["completion_ms"]
    assert [v is not None for v in verdicts] == [False, True, False, True, False, False]
    assert verdicts[1] > verdicts[3]
    assert X.best_valid_body(pre, bodies[:1], X.ja_machine_preset("dgx_h100"))[0] is None


def test_beam_search_against_the_oracle_on_random_preambles():
    rng = random.Random(5)
    for trial in range(12):
        n_sites = rng.choice([3, 4])
        atoms = list("ABCDEF")[:rng.randint(2, 5)]
        text = "GPUS: " + ", ".join(map(str, range(n_sites))) + "\nIN: " + "; ".join("%s @ %d" % (a, rng.randrange(n_sites)) for a in atoms)
        outs = []
        for _ in range(rng.randint(1, 2)):
            x = rng.sample(atoms, rng.randint(1, len(atoms)))
            outs.append("+".join(sorted(x)) + " @ " + ", ".join(map(str, sorted(rng.sample(range(n_sites), rng.randint(1, n_sites))))))
        text += "\nOUT: " + "; ".join(outs) + "\n"
        for mname in ("dgx_h100", "dgx_v100"):
            h = X.ExchangeProgram(text)
            ms = X.ja_exprog_synthesize(h.handle, X.ja_machine_preset(mname), 2, 5)
            q, ms_o = E.synthesize(E.parse(text), E.machine(mname), depth=2, beam=5)
            assert close(ms, ms_o)
            mk = masks(q)
            assert set(X.ja_exprog_get_actions(h.handle)) == {(mk(x), s, sites_mask(d)) for x, s, d in E.expanded(q)}
            assert X.ja_exprog_check(h.handle) == (True, True)
            start = X.ExchangeProgram(text)
            X.ja_exprog_body(start.handle, "naive")
            assert ms <= X.ja_exprog_simulate(start.handle, X.ja_machine_preset(mname)) * (1 + 1e-12)


def test_a_machine_given_as_a_table_of_links():
    from paper_2609_03905_b200.binding import JaError
    # the cube mesh written out as a table is the preset
    table = [[0.0] * 8 for _ in range(8)]
    for a in range(8):
        for b in range(8):
            if a != b:
                table[a][b] = 50.0 if abs(a - b) == 4 else (25.0 if a // 4 == b // 4 else 0.0)
    m = X.machine_from_links(table, 900.0, 15.75)
    mo = {"kind": "links", "links": table, "pcie": 15.75, "hbm": 900.0}
    h = X.ExchangeProgram(G["v100"]["program"])
    ms = X.ja_exprog_place(h.handle, m, "own")
    assert round(ms) == G["v100"]["completion_ms"]
    g = X.ExchangeProgram(G["v100"]["program"])
    assert close(X.ja_exprog_place(g.handle, X.ja_machine_preset("dgx_v100"), "own"), ms)
    assert close(E.place(E.parse(G["v100"]["program"]), mo)[2], ms)
    # a directed ring of four sites: 0 -> 1 -> 2 -> 3 -> 0 at 10 GB/s, nothing else, no bridge needed by this program
    ring = [[0.0] * 4 for _ in range(4)]
    for a in range(4):
        ring[a][(a + 1) % 4] = 10.0
    text = "IN: A @ 0 (size: 2 GB)\nOUT: A @ 3\n\nA @ 0 -> 1; A @ 1 -> 2; A @ 2 -> 3\n"
    mr = X.machine_from_links(ring, 1000.0, 5.0)
    assert close(X.ja_exprog_simulate(X.ExchangeProgram(text), mr), 3 * 2 / 10 * 1e3)          # three hops, one after the other
    direct = "IN: A @ 0 (size: 2 GB)\nOUT: A @ 3\n\nA @ 0 -> 3\n"
    assert close(X.ja_exprog_simulate(X.ExchangeProgram(direct), mr), 2 / 5 * 1e3)            # unlinked: over the bridge
    with pytest.raises(JaError):                                                                       # unlinked pairs but no bridge
        X.ja_exprog_simulate(X.ExchangeProgram(direct), X.machine_from_links(ring, 1000.0, 0.0))
    with pytest.raises(JaError):                                                                       # a site outside the table
        X.ja_exprog_simulate(X.ExchangeProgram("IN: A @ 5\nOUT: A @ 5\n"), mr)
    # random tables and random programs against the oracle
    rng = random.Random(41)
    for _ in range(25):
        n = rng.randint(2, 5)
        links = [[0.0 if a == b or rng.random() < 0.3 else rng.choice([5.0, 12.5, 40.0]) for b in range(n)] for a in range(n)]
        ml, mlo = X.machine_from_links(links, 800.0, 3.0), {"kind": "links", "links": links, "pcie": 3.0, "hbm": 800.0}
        atoms = list("ABCD")[:rng.randint(2, 4)]
        t = "GPUS: " + ", ".join(map(str, range(n))) + "\nIN: " + "; ".join("%s @ %d" % (a, rng.randrange(n)) for a in atoms)
        t += "\nOUT: " + "+".join(atoms) + " @ " + ", ".join(map(str, sorted(rng.sample(range(n), rng.randint(1, n))))) + "\n"
        for body in ("naive", "butterfly"):
            hh = X.ExchangeProgram(t)
            X.ja_exprog_body(hh.handle, body)
            q = (E.naive_body if body == "naive" else E.butterfly_body)(E.parse(t))
            assert close(X.ja_exprog_simulate(hh.handle, ml), E.simulate(q, mlo))
        hs = X.ExchangeProgram(t)
        ms_s = X.ja_exprog_synthesize(hs.handle, ml, 1, 4)
        assert close(ms_s, E.synthesize(E.parse(t), mlo, depth=1, beam=4)[1])


def test_merged_programs_run_their_exchanges_at_the_same_time():
    from paper_2609_03905_b200.binding import JaError
    a_text = "GPUS: 0, 1, 2, 3\nIN: A @ 0; B @ 1\nOUT: A+B @ 2\n\nA @ 0 -> 2; B @ 1 -> 2; A+B @ 2\n"
    b_text = "GPUS: 0, 1, 2, 3\nIN: A @ 3; B @ 2\nOUT: A+B @ 0, 1\n\nA @ 3 -> 0, 1; B @ 2 -> 0, 1; A+B @ 0, 1\n"
    a, b = X.ExchangeProgram(a_text), X.ExchangeProgram(b_text)
    m = X.ExchangeProgram(handle=X.ja_exprog_merge(a.handle, b.handle, "x_", "w_"))
    mo = E.merge(E.parse(a_text), E.parse(b_text), "x_", "w_")
    same_program(m.handle, mo)
    assert X.ja_exprog_check(m.handle) == (True, True) and E.valid_bound(mo)
    mk = masks(mo)
    assert library_state(m.handle) == {(mk(x), s) for x, s in E.closure(mo)}
    for name in ("dgx_h100", "dgx_v100"):
        mach, macho = X.ja_machine_preset(name), E.machine(name)
        ta, tb, tm = (X.ja_exprog_simulate(h.handle, mach) for h in (a, b, m))
        assert close(tm, E.simulate(mo, macho))
        assert max(ta, tb) * (1 - 1e-12) <= tm <= (ta + tb) * (1 + 1e-12)       # concurrent, sharing endpoints and memory
    with pytest.raises(JaError):
        X.ja_exprog_merge(a.handle, b.handle, "", "")                            # names clash
    other = X.ExchangeProgram("GPUS: 0, 1\nIN: A @ 0\nOUT: A @ 1\n")          # objects are kept: a handle dies with its object
    with pytest.raises(JaError):
        X.ja_exprog_merge(a.handle, other.handle, "p", "q")
    # the merged preamble of a partitioned pair places both operands with one membership
    p1 = "GPUS: 0, 1\nPARTITIONS: S1 {size 1} S2 {size 1}\nIN: A @ 0; B @ 1\nOUT: A @ S1; B @ S2\n"
    p2 = "GPUS: 0, 1\nPARTITIONS: S1 {size 1} S2 {size 1}\nIN: C @ 1 (size: 4 GB); D @ 0 (size: 4 GB)\nOUT: C @ S1; D @ S2\n"
    h1, h2 = X.ExchangeProgram(p1), X.ExchangeProgram(p2)
    j = h1.merge(h2, "a_", "b_")
    ms = X.ja_exprog_place(j.handle, X.ja_machine_preset("dgx_h100"), "naive")
    assert X.ja_exprog_membership(j.handle, "S1") == 1 << 1 and close(ms, 1 / 450 * 1e3)      # the 4 GB operand decides: S1 where C is
