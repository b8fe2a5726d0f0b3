"""CPU tests of libja's host side: the library loads and exports every declared symbol, and its integer
bookkeeping (function-spec tuples, tilings, cost counts, key tables, overlay atoms) equals, bit for bit, the
tables the oracle builds independently from the paper's definitions. No kernel is launched here."""
import ctypes
import json
import os
import re

import numpy as np
import pytest

import paper_2609_03905_b200 as ja
from oracle import blocked

RNG = np.random.default_rng(20260905)
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    inc = os.path.join(ROOT, "include")
    names = set()
    for h in sorted(os.listdir(inc)):
        if h.endswith(".h"):
            # declarations only: a name at the start of a prototype (after its return type), not one mentioned in a comment
            text = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, h)).read(), flags=re.S)
            names |= set(re.findall(r"\b(ja_[a-z0-9_]+)\s*\(", text))
    assert {"ja_spec_create", "ja_relation_create", "ja_execute", "ja_repartition", "ja_exprog_parse", "ja_exprog_simulate"} <= names
    lib = ctypes.CDLL(ja.binding.LIB_PATH)
    for n in sorted(names):
        assert hasattr(lib, n), f"{n} is declared under include/ but not exported"
    assert "sm_100a" in ja.ja_version()


def _rand_parts(letters, lo=3, hi=40):
    parts = {}
    for c in letters:
        e = int(RNG.integers(lo, hi))
        cuts = sorted(set(RNG.integers(1, e, int(RNG.integers(0, 4))).tolist()))
        parts[c] = [0] + cuts + [e]
    return parts


@pytest.mark.parametrize("einsum,fn,agg", [
    ("ij,jk->ik", "mul", "sum"), ("ij,ij->ij", "silu_mul", "none"), ("ij->i", "square", "sum"),
    ("hij->hi", "ident", "max"), ("hij,hi->hi", "exp_sub", "sum"), ("hij,hi,hi->hij", "exp_sub_div", "none"),
    ("ij,i,j->ij", "rms_scale", "none"), ("bshd->bshd", "rope", "none"), ("ij,jk,kl->il", "mul", "sum"),
])
def test_spec_tables_match_oracle(einsum, fn, agg):
    for _ in range(4):
        letters = blocked.core.parse_einsum(einsum)[2]
        parts = _rand_parts(letters)
        ref = blocked.Spec(einsum, parts)
        s = ja.ja_spec_create(einsum, parts, fn, (1e-5,), agg)
        try:
            p, n_in = ja.ja_spec_num_tuples(s)
            assert (p, n_in) == (ref.p, len(ref.ins))
            ink, outk = ja.ja_spec_get_tuples(s)
            rink, routk = ref.tuples()
            assert ink.dtype == rink.dtype and np.array_equal(ink, rink) and np.array_equal(outk, routk)
            for operand in list(range(n_in)) + [-1]:
                nb, splits = ja.ja_spec_operand_tiling(s, operand)
                rnb, rsplits = ref.operand_tiling(operand)
                assert nb == rnb and splits == [list(x) for x in rsplits]
            assert ja.ja_spec_cost_terms(s) == ref.cost_terms()
        finally:
            ja.ja_spec_destroy(s)


def test_attention_spec_band_predicate():
    parts = {"b": [0, 1, 2], "q": blocked.equal_splits(512, 4), "h": [0, 1, 2, 3], "d": [0, 128],
             "k": blocked.equal_splits(512, 4)}
    es = "bqhd,bkhd,bkhd->bqhd"
    ref = blocked.Spec(es, parts, band=("k", "q"))
    s = ja.ja_spec_create(es, parts, "attention", (0.088, 1.0), "online_softmax")
    ink, outk = ja.ja_spec_get_tuples(s)
    rink, routk = ref.tuples()
    assert np.array_equal(ink, rink) and np.array_equal(outk, routk)
    assert ja.ja_spec_num_tuples(s)[0] == 2 * 3 * (4 * 5 // 2)          # q-blocks x k-blocks with kb <= qb
    assert np.bincount(outk).reshape(2, 4, 3)[0, :, 0].tolist() == [1, 2, 3, 4]   # multiplicity m = qb + 1
    ja.ja_spec_destroy(s)
    full = ja.ja_spec_create(es, parts, "attention", (0.088, 0.0), "online_softmax")  # not causal: whole grid
    assert ja.ja_spec_num_tuples(full)[0] == 2 * 4 * 3 * 4
    ja.ja_spec_destroy(full)


def test_attention_spec_grouped_heads_and_packed_sequences(golden_dir):
    """Example 3.10: heads_q inherits its split from heads_kv; the sequence is cut at sequence ends only."""
    g = json.load(open(os.path.join(golden_dir, "gqa_packed_example.json")))
    Hq, Hkv, grp, S, ends = g["heads_q"], g["heads_kv"], g["group"], g["sequence_extent"], g["sequence_ends"]
    es = "bqhd,bkgd,bkgd->bqhd"
    parts = {"b": [0, 1], "q": [0, S], "h": [grp * m for m in range(Hkv + 1)], "d": [0, 128], "k": [0, S],
             "g": list(range(Hkv + 1))}
    s = ja.ja_spec_create(es, parts, "attention", (0.088, 1.0), "online_softmax")
    assert ja.ja_spec_num_tuples(s)[0] == g["num_function_specs_when_heads_kv_is_cut_into_unit_intervals"]
    ink, outk = ja.ja_spec_get_tuples(s)
    rink, routk = blocked.Spec(es, parts, band=("k", "q"), induced=("h", "g", grp)).tuples()
    assert np.array_equal(ink, rink) and np.array_equal(outk, routk)
    assert ink[:, 0].tolist() == ink[:, 1].tolist() == list(range(Hkv))     # m-th spec: q-head block m with kv head m
    ja.ja_spec_destroy(s)
    with pytest.raises(ja.JaError):      # heads_q is not shardable by itself
        ja.ja_spec_create(es, dict(parts, h=[0, 16, 32]), "attention", (0.088, 1.0), "online_softmax")
    # cut at the sequence ends: 3 sequences x 8 heads, no aggregation (every output key has one tuple)
    parts2 = dict(parts, q=[0] + ends, k=[0] + ends)
    prm = (0.088, 1.0) + tuple(float(e) for e in ends)
    s = ja.ja_spec_create(es, parts2, "attention", prm, "online_softmax")
    assert ja.ja_spec_num_tuples(s)[0] == g["num_function_specs_when_sequence_is_cut_at_its_ends_and_heads_kv_into_unit_intervals"]
    ink, outk = ja.ja_spec_get_tuples(s)
    ref = blocked.Spec(es, parts2, band=("k", "q"), induced=("h", "g", grp), segments=("k", "q", ends))
    rink, routk = ref.tuples()
    assert np.array_equal(ink, rink) and np.array_equal(outk, routk)
    assert np.bincount(outk).tolist() == [1] * 24
    ja.ja_spec_destroy(s)
    # finer cuts inside sequences (every end still a split point): band and same-sequence selections together
    parts3 = dict(parts, q=blocked.equal_splits(S, 8), k=blocked.equal_splits(S, 16))
    for causal in (1.0, 0.0):
        s = ja.ja_spec_create(es, parts3, "attention", (0.088, causal) + prm[2:], "online_softmax")
        ref = blocked.Spec(es, parts3, band=("k", "q") if causal else None, induced=("h", "g", grp), segments=("k", "q", ends))
        ink, outk = ja.ja_spec_get_tuples(s)
        rink, routk = ref.tuples()
        assert np.array_equal(ink, rink) and np.array_equal(outk, routk)
        ja.ja_spec_destroy(s)
    with pytest.raises(ja.JaError):      # a cut that skips a sequence end
        ja.ja_spec_create(es, dict(parts, q=[0, 2048, S], k=[0, 2048, S]), "attention", prm, "online_softmax")
    with pytest.raises(ja.JaError):      # ends must ascend and finish at the extent
        ja.ja_spec_create(es, parts2, "attention", (0.088, 1.0, 2560.0, 1024.0, 4096.0), "online_softmax")


def test_paper_worked_examples_through_the_library(golden_dir):
    g = json.load(open(os.path.join(golden_dir, "matmul_decomposed.json")))
    s = ja.ja_spec_create(g["einsum"], g["four_spec"]["parts"])
    assert ja.ja_spec_num_tuples(s)[0] == g["four_spec"]["num_function_specs"]
    ink, outk = ja.ja_spec_get_tuples(s)
    assert np.bincount(outk).tolist() == g["four_spec"]["multiplicity"]
    nb, splits = ja.ja_spec_operand_tiling(s, -1)
    types = [{"lower": [splits[0][i], 0], "upper": [splits[0][i + 1], splits[1][1]]} for i in range(nb[0])]
    assert types == g["four_spec"]["distinct_output_types"]
    ja.ja_spec_destroy(s)
    s = ja.ja_spec_create(g["einsum"], g["two_spec"]["parts"])
    assert ja.ja_spec_num_tuples(s)[0] == 2 and np.bincount(ja.ja_spec_get_tuples(s)[1]).tolist() == [2]
    ja.ja_spec_destroy(s)
    c = json.load(open(os.path.join(golden_dir, "cost_3d_matmul.json")))
    for case in c["cases"]:
        parts = {l: blocked.equal_splits(case["N"], n) for l, n in zip("ijk", (case["a"], case["b"], case["c"]))}
        s = ja.ja_spec_create("ij,jk->ik", parts)
        assert ja.ja_spec_cost_terms(s) == (case["join"], case["agg"])
        ja.ja_spec_destroy(s)


FAKE_PTR = 1 << 20  # never dereferenced on the CPU: relation creation makes no CUDA call


def _rel(extents, splits, dtype=ja.JA_BF16, ptr=FAKE_PTR):
    return ja.ja_relation_create(extents, splits, dtype, ptr, ja.ja_relation_bytes(extents, splits, dtype))


def test_relation_key_table_matches_oracle():
    for _ in range(10):
        rank = int(RNG.integers(1, 5))
        parts = _rand_parts("abcd"[:rank], 2, 20)
        splits = [parts[c] for c in "abcd"[:rank]]
        ext = [s[-1] for s in splits]
        for dt, es in ((ja.JA_BF16, 2), (ja.JA_F32, 4)):
            r = _rel(ext, splits, dt)
            coords, lower, upper, offs = ja.ja_relation_get_keys(r)
            rc, rl, ru, ro, total = blocked.relation_keys(ext, splits, es)
            assert np.array_equal(coords, rc) and np.array_equal(lower, rl) and np.array_equal(upper, ru)
            assert np.array_equal(offs, ro) and ja.ja_relation_bytes(ext, splits, dt) == total
            ja.ja_relation_destroy(r)


def test_overlay_atoms_match_oracle_and_paper(golden_dir):
    g = json.load(open(os.path.join(golden_dir, "overlay_example.json")))
    src = _rel(g["extents"], g["producer_splits"])
    dst = _rel(g["extents"], g["consumer_splits"], ptr=FAKE_PTR * 2)
    lower, upper, sb, db = ja.ja_overlay_atoms(src, dst)
    assert len(sb) == g["num_atoms"] and sb.tolist() == g["atom_to_producer_block"] and db.tolist() == g["atom_to_consumer_block"]
    assert sorted(set(lower[:, 0].tolist() + upper[:, 0].tolist())) == g["overlay_row_split_points"]
    ja.ja_relation_destroy(src); ja.ja_relation_destroy(dst)
    for _ in range(10):
        rank = int(RNG.integers(1, 5))
        ext = [int(RNG.integers(3, 14)) for _ in range(rank)]
        mk = lambda: [[0] + sorted(set(RNG.integers(1, e, int(RNG.integers(0, 3))).tolist())) + [e] for e in ext]
        s_sp, d_sp = mk(), mk()
        src, dst = _rel(ext, s_sp), _rel(ext, d_sp, ptr=FAKE_PTR * 2)
        lower, upper, sb, db = ja.ja_overlay_atoms(src, dst)
        _, atoms = blocked.overlay_atoms(s_sp, d_sp)
        assert lower.tolist() == [a[0] for a in atoms] and upper.tolist() == [a[1] for a in atoms]
        assert sb.tolist() == [a[2] for a in atoms] and db.tolist() == [a[3] for a in atoms]
        ja.ja_relation_destroy(src); ja.ja_relation_destroy(dst)


def _status(fn, *a, **k):
    with pytest.raises(ja.JaError) as e:
        fn(*a, **k)
    return e.value.status_name


def test_error_codes():
    ok = {"i": [0, 4], "j": [0, 2, 4], "k": [0, 4]}
    assert _status(ja.ja_spec_create, "ij,jk>ik", ok) == "JA_ERR_PARSE"
    assert _status(ja.ja_spec_create, "iJ,jk->ik", ok) == "JA_ERR_PARSE"
    assert _status(ja.ja_spec_create, "ij,jk->iz", ok) == "JA_ERR_PARSE"
    assert _status(ja.ja_spec_create, "ij,jk->ik", {"i": [0, 4], "j": [0, 4]}) == "JA_ERR_SHAPE"
    assert _status(ja.ja_spec_create, "ij,jk->ik", dict(ok, j=[0, 3, 3, 4])) == "JA_ERR_TILING"   # empty interval
    assert _status(ja.ja_spec_create, "ij,jk->ik", dict(ok, j=[1, 2, 4])) == "JA_ERR_TILING"      # gap at 0
    assert _status(ja.ja_spec_create, "ij,jk->ik", dict(ok, j=[0, 3, 2, 4])) == "JA_ERR_TILING"   # overlap
    assert _status(ja.ja_spec_create, "ij,jk->ik", ok, "mul", (), "none") == "JA_ERR_TILING"      # shared output type, no (+)
    assert _status(ja.ja_relation_create, [4, 4], [[0, 4], [0, 5]], ja.JA_BF16, FAKE_PTR, 1 << 20) == "JA_ERR_TILING"
    assert _status(ja.ja_relation_create, [4, 4], [[0, 4], [0, 4]], ja.JA_BF16, FAKE_PTR + 2, 1 << 20) == "JA_ERR_ALIGNMENT"
    assert _status(ja.ja_relation_create, [4, 4], [[0, 4], [0, 4]], ja.JA_BF16, FAKE_PTR, 8) == "JA_ERR_INVALID_ARG"
    assert _status(ja.ja_relation_create, [4, 4], [[0, 4], [0, 4]], 7, FAKE_PTR, 1 << 20) == "JA_ERR_DTYPE"
    # tiling mismatch between a relation and in_k(J) is refused before anything is enqueued
    s = ja.ja_spec_create("ij,jk->ik", ok)
    A = _rel([4, 4], [[0, 4], [0, 4]], ja.JA_F32)                    # j not split: differs from the spec
    Bm = _rel([4, 4], [[0, 2, 4], [0, 4]], ja.JA_F32, FAKE_PTR * 2)
    C = _rel([4, 4], [[0, 4], [0, 4]], ja.JA_F32, FAKE_PTR * 3)
    assert _status(ja.ja_execute, s, [A, Bm], [C]) == "JA_ERR_PARTITION_MISMATCH"
    assert _status(ja.ja_execute, s, [A], [C]) == "JA_ERR_INVALID_ARG"
    A2 = _rel([4, 5], [[0, 4], [0, 2, 5]], ja.JA_F32)
    assert _status(ja.ja_execute, s, [A2, Bm], [C]) == "JA_ERR_SHAPE"
    for h in (A, A2, Bm, C):
        ja.ja_relation_destroy(h)
    ja.ja_spec_destroy(s)


def test_partial_relation_argument_checks():
    """Join-only execution and the aggregating relayout refuse malformed partial relations before any CUDA call."""
    parts = {"i": [0, 4], "j": [0, 2, 4], "k": [0, 4]}
    s = ja.ja_spec_create("ij,jk->ik", parts)
    A = _rel([4, 4], [[0, 4], [0, 2, 4]], ja.JA_F32)
    Bm = _rel([4, 4], [[0, 2, 4], [0, 4]], ja.JA_F32, FAKE_PTR * 2)
    C = _rel([4, 4], [[0, 4], [0, 4]], ja.JA_F32, FAKE_PTR * 3)
    P_rank = _rel([4, 4], [[0, 4], [0, 4]], ja.JA_F32, FAKE_PTR * 4)                                 # no copy index
    P_m3 = _rel([3, 4, 4], [[0, 1, 2, 3], [0, 4], [0, 4]], ja.JA_F32, FAKE_PTR * 5)                  # multiplicity is 2
    P_coarse = _rel([2, 4, 4], [[0, 2], [0, 4], [0, 4]], ja.JA_F32, FAKE_PTR * 6)                    # copies share a block
    P_tiled = _rel([2, 4, 4], [[0, 1, 2], [0, 2, 4], [0, 4]], ja.JA_F32, FAKE_PTR * 7)               # not out(J)
    P_shape = _rel([2, 4, 6], [[0, 1, 2], [0, 4], [0, 6]], ja.JA_F32, FAKE_PTR * 8)
    P_ok = _rel([2, 4, 4], [[0, 1, 2], [0, 4], [0, 4]], ja.JA_F32, FAKE_PTR * 9)
    assert _status(ja.ja_execute_join, s, [A, Bm], P_rank) == "JA_ERR_SHAPE"
    assert _status(ja.ja_execute_join, s, [A, Bm], P_m3) == "JA_ERR_SHAPE"
    assert _status(ja.ja_execute_join, s, [A, Bm], P_coarse) == "JA_ERR_TILING"
    assert _status(ja.ja_execute_join, s, [A, Bm], P_tiled) == "JA_ERR_PARTITION_MISMATCH"
    assert _status(ja.ja_execute_join, s, [A, Bm], P_shape) == "JA_ERR_SHAPE"
    assert _status(ja.ja_execute_join, s, [A], P_ok) == "JA_ERR_INVALID_ARG"
    assert _status(ja.ja_repartition_agg, P_rank, "sum", C) == "JA_ERR_SHAPE"
    assert _status(ja.ja_repartition_agg, P_coarse, "sum", C) == "JA_ERR_TILING"
    assert _status(ja.ja_repartition_agg, P_shape, "sum", C) == "JA_ERR_SHAPE"
    assert _status(ja.ja_repartition_agg, P_ok, "none", C) == "JA_ERR_INVALID_ARG"      # two copies, no (+)
    assert _status(ja.ja_repartition_agg, P_ok, "online_softmax", C) == "JA_ERR_INVALID_ARG"
    for h in (A, Bm, C, P_rank, P_m3, P_coarse, P_tiled, P_shape, P_ok):
        ja.ja_relation_destroy(h)
    ja.ja_spec_destroy(s)


def _mlp_tree(T, d, f):
    return [{"einsum": "ij,jk->ik", "extents": {"i": T, "j": d, "k": f}, "inputs": [None, None]},
            {"einsum": "ij,jk->ik", "extents": {"i": T, "j": d, "k": f}, "inputs": [None, None]},
            {"einsum": "ik,ik->ik", "extents": {"i": T, "k": f}, "inputs": [0, 1]},
            {"einsum": "ik,kl->il", "extents": {"i": T, "k": f, "l": d}, "inputs": [2, None]}]


def test_logical_optimizer_matches_oracle(golden_dir):
    """ja_plan_optimize / ja_plan_cost (closed-form sub-costs) against the oracle's Algorithm 1 and its explicit
    per-function-spec cost count: total costs are integers and must be equal; the returned plan must cost what it claims."""
    from oracle import optimizer
    g = json.load(open(os.path.join(golden_dir, "optimizer_example.json")))
    for c in g["three_d"]:
        N, p, q = c["N"], c["p"], c["q"]
        op = {"einsum": "ij,jk->ik", "extents": {"i": N, "j": N, "k": N}, "inputs": [None, None]}
        total, plan = ja.ja_plan_optimize([op], p)
        assert total == (3 * q - 1) * N * N and plan == [{"i": q, "j": q, "k": q}]
    ch = g["chain"]
    for pc in ch["plan_costs"]:
        assert ja.ja_plan_cost(ch["ops"], pc["plan"]) == pc["cost"]
    assert ja.ja_plan_optimize(ch["ops"], ch["p"])[0] == ch["optimum"]
    rng = np.random.default_rng(5)
    trees = [(_mlp_tree(8, 6, 12), 4), (_mlp_tree(2048, 4096, 11008), 8), (_mlp_tree(100, 36, 50), 12),
             ([{"einsum": "bqhd,bkhd->bhqk", "extents": {"b": 2, "q": 8, "h": 4, "d": 4, "k": 8}, "inputs": [None, None], "fixed": {"d"}},
               {"einsum": "bhqk,bkhd->bqhd", "extents": {"b": 2, "h": 4, "q": 8, "k": 8, "d": 4}, "inputs": [0, None], "fixed": {"d"}}], 4)]
    for ops, p in trees:
        want, want_plan = optimizer.optimize_tree(ops, p)
        got, plan = ja.ja_plan_optimize(ops, p)
        assert got == want
        assert ja.ja_plan_cost(ops, plan) == got == optimizer.plan_cost(ops, plan)
        for _ in range(5):   # random assignments cost the same on both sides and never less than the optimum
            rp = [optimizer.specs(op, p)[int(rng.integers(len(optimizer.specs(op, p))))] for op in ops]
            c = ja.ja_plan_cost(ops, rp)
            assert c == optimizer.plan_cost(ops, rp) and c >= got
    with pytest.raises(ja.JaError):   # a node consumed twice is not a tree
        ja.ja_plan_optimize([ch["ops"][0], {"einsum": "ik,ik->ik", "extents": {"i": 4, "k": 4}, "inputs": [0, 0]}], 2)
    with pytest.raises(ja.JaError):   # producer / operand shapes must agree
        ja.ja_plan_optimize([ch["ops"][0], {"einsum": "ik->i", "extents": {"i": 4, "k": 5}, "inputs": [0]}], 2)


def test_logical_optimizer_on_graphs_with_shared_tensors():
    """Section 4.5 through the library against the oracle: same trees, same order, same assembled cost."""
    from oracle import optimizer
    from test_oracle_pins import _block_graph
    for dims, p in (((16, 8, 12), 2), ((16, 8, 12), 4), ((64, 32, 48), 8)):
        ops = _block_graph(*dims)
        want, want_plan = optimizer.optimize_graph(ops, p)
        got, plan = ja.ja_plan_optimize_graph(ops, p)
        assert got == want == optimizer.plan_cost(ops, plan) == ja.ja_plan_cost(ops, plan)
    tree = _mlp_tree(100, 36, 50)
    assert ja.ja_plan_optimize_graph(tree, 12)[0] == ja.ja_plan_optimize(tree, 12)[0]


def test_greedy_selector_against_the_oracle_and_the_optimizer():
    """The greedy selector of the plan-selection experiment (Section 6, Experiment 3): per operator the spec of least join +
    aggregation cost, the repartition sub-cost ignored. The library's choice equals the oracle's, its cost is the full
    cost of that plan, and on trees it is never below the optimizer's (equal where no relayout can be saved)."""
    from oracle import optimizer
    from test_oracle_pins import _block_graph
    worse = 0
    for tree, p in ((_mlp_tree(64, 32, 48), 4), (_mlp_tree(100, 36, 50), 12), (_mlp_tree(16, 16, 16), 8)):
        want_cost, want_plan = optimizer.greedy(tree, p)
        got_cost, got_plan = ja.ja_plan_select_greedy(tree, p)
        assert got_plan == want_plan and got_cost == want_cost == optimizer.plan_cost(tree, got_plan) == ja.ja_plan_cost(tree, got_plan)
        best = ja.ja_plan_optimize(tree, p)[0]
        assert got_cost >= best
        worse += got_cost > best
    assert worse > 0       # the cases are not all degenerate: somewhere ignoring the relayouts costs something
    for dims, p in (((16, 8, 12), 4), ((64, 32, 48), 8)):       # graphs with multiply consumed tensors
        ops = _block_graph(*dims)
        want_cost, want_plan = optimizer.greedy(ops, p)
        got_cost, got_plan = ja.ja_plan_select_greedy(ops, p)
        assert got_plan == want_plan and got_cost == want_cost == ja.ja_plan_cost(ops, got_plan)
    # every operator's choice really is its own minimum: brute force over its specs with no producer tilings
    ops = _block_graph(16, 8, 12)
    _, plan = ja.ja_plan_select_greedy(ops, 4)
    for op, J in zip(ops, plan):
        free = [None] * len(op["inputs"])
        assert optimizer.cost(op, J, free) == min(optimizer.cost(op, K, free) for K in optimizer.specs(op, 4))
