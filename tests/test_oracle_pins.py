"""Pins for the CPU oracle: it is checked against things other than itself -- the paper's printed
worked examples (tests/golden), closed forms, invariants, brute force on tiny inputs and
torch-CPU fp64 library routines -- before anything on the GPU is trusted against it."""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import blocked, core, operators, relational

RNG = np.random.default_rng(3905)


def _golden(golden_dir, name):
    with open(os.path.join(golden_dir, name)) as f:
        return json.load(f)


# ---------------------------------------------------------------------------------------------
# rounding
# ---------------------------------------------------------------------------------------------
def test_round_bf16_matches_torch_and_ties_to_even():
    x = np.concatenate([RNG.standard_normal(20000) * 10.0 ** RNG.integers(-30, 30, 20000),
                        [0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38, 1e-40, -1e-45, 65504.0]])
    x32 = x.astype(np.float32).astype(np.float64)  # torch rounds from fp32; feed fp32-representable values
    want = torch.from_numpy(x32.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    got = core.round_to(x32, "bf16")
    assert np.array_equal(got, want)
    # exact ties: 1 + 2^-8 lies midway between 1 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert core.round_to([1.0 + 2.0 ** -8], "bf16")[0] == 1.0
    assert core.round_to([1.0 + 3 * 2.0 ** -8], "bf16")[0] == 1.0 + 2.0 ** -6
    # one rounding from fp64, not two: just above the tie must round up
    assert core.round_to([1.0 + 2.0 ** -8 + 2.0 ** -40], "bf16")[0] == 1.0 + 2.0 ** -7
    assert np.array_equal(core.round_to(x, "f32"), x.astype(np.float32).astype(np.float64))


def test_round_f16_matches_numpy_and_torch_ties_range_and_subnormals():
    """IEEE binary16, the storage type of the paper's experiments (Section 6): one rounding from fp64, ties to even,
    overflow to infinity from 65520 on, subnormals in steps of 2^-24. numpy converts fp64 to float16 with one correct
    rounding; torch is fed fp32-representable values (it rounds from fp32)."""
    x = np.concatenate([RNG.standard_normal(20000) * 10.0 ** RNG.integers(-9, 5, 20000),
                        [0.0, 1.0, 65504.0, 65519.9, 65520.0, -65520.0, 70000.0, 2.0 ** -14, 2.0 ** -24, 2.0 ** -25,
                         1.5 * 2.0 ** -24, 2.5 * 2.0 ** -24, 2.0 ** -25 * (1 + 2.0 ** -30), 1e-9]])
    with np.errstate(over="ignore"):
        assert np.array_equal(core.round_to(x, "f16"), x.astype(np.float16).astype(np.float64))
    x32 = x.astype(np.float32).astype(np.float64)
    want = torch.from_numpy(x32.astype(np.float32)).to(torch.float16).to(torch.float64).numpy()
    assert np.array_equal(core.round_to(x32, "f16"), want)
    # exact ties: 1 + 2^-11 lies midway between 1 and 1 + 2^-10 -> 1.0 (even); 1 + 3 * 2^-11 -> 1 + 2^-9
    assert core.round_to([1.0 + 2.0 ** -11], "f16")[0] == 1.0
    assert core.round_to([1.0 + 3 * 2.0 ** -11], "f16")[0] == 1.0 + 2.0 ** -9
    # one rounding from fp64, not two: just above the tie rounds up (fp64 -> fp32 -> f16 would land on the tie and round down)
    assert core.round_to([1.0 + 2.0 ** -11 + 2.0 ** -40], "f16")[0] == 1.0 + 2.0 ** -10
    # range and subnormals
    r = core.round_to([65519.9, 65520.0, 2.0 ** -25, 1.5 * 2.0 ** -24, 2.5 * 2.0 ** -24], "f16")
    assert r[0] == 65504.0 and np.isinf(r[1]) and r[2] == 0.0 and r[3] == 2.0 ** -23 and r[4] == 2.0 ** -23
    # f16 keeps three more bits than bf16 on the same values
    v = RNG.standard_normal(4096)
    assert np.abs(core.round_to(v, "f16") - v).max() < np.abs(core.round_to(v, "bf16") - v).max() / 4


# ---------------------------------------------------------------------------------------------
# the three engines against brute force (tiny inputs, every extent <= 6)
# ---------------------------------------------------------------------------------------------
CASES = [
    ("ij,jk->ik", "mul", "sum", ()),
    ("ij,kj->ik", "mul", "sum", ()),
    ("bqhd,bkhd->bhqk", "mul", "sum", ()),
    ("ij->i", "square", "sum", ()),
    ("hij->hi", "ident", "max", ()),
    ("hij,hi->hi", "exp_sub", "sum", ()),
    ("hij,hi,hi->hij", "exp_sub_div", "none", ()),
    ("ij,ij->ij", "silu_mul", "none", ()),
    ("ij,ij->ij", "add", "none", ()),
    ("ij,i,j->ij", "rms_scale", "none", (1e-5, 5.0)),
    ("ij,jk,kl->il", "mul", "sum", ()),
    ("i,j->ij", "mul", "none", ()),
]


@pytest.mark.parametrize("einsum,fn,agg,params", CASES)
def test_engines_agree_with_brute_force(einsum, fn, agg, params):
    ins, out, letters = core.parse_einsum(einsum)
    ext = {c: int(RNG.integers(2, 6)) for c in letters}
    if fn == "rms_scale":
        ext["j"] = 5
    inputs = [RNG.standard_normal([ext[c] for c in t]) for t in ins]
    if fn in ("rms_scale",):
        inputs[1] = np.abs(inputs[1]) + 0.1
    if fn == "exp_sub_div":
        inputs[2] = np.abs(inputs[2]) + 0.5
    want = relational.brute_einsum(einsum, inputs, fn, agg, params)
    t1 = core.join_agg(einsum, inputs, fn, agg, params)
    t0 = relational.t0_join_agg(einsum, inputs, fn, agg, params)
    np.testing.assert_allclose(t1, want, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(t0, want, rtol=1e-13, atol=1e-13)
    # ascending fold order is the same in T0 and T1 => identical bits (numpy's exp may differ from libm's)
    if fn in ("mul", "ident", "square", "add"):
        assert np.array_equal(t0, t1)


def test_selection_predicate_against_brute_force():
    S = RNG.standard_normal((2, 5, 5))
    for eng in (core.join_agg, relational.t0_join_agg):
        got = eng("hqk->hq", [S], fn="ident", agg="max", pred=("k", "q"))
        want = relational.brute_einsum("hqk->hq", [S], "ident", "max", (), pred=("k", "q"))
        assert np.array_equal(got, want)
        assert np.array_equal(got, np.array([[S[h, q, : q + 1].max() for q in range(5)] for h in range(2)]))


def test_t0_equals_t1_on_config1_shape():
    """Config 1 through the literal tuple engine: 256^3 = 16.8 M joined tuples."""
    A = RNG.standard_normal((256, 256)).astype(np.float32).astype(np.float64)
    B = RNG.standard_normal((256, 256)).astype(np.float32).astype(np.float64)
    t1 = core.matmul(A, B)
    t0 = relational.t0_join_agg("ij,jk->ik", [A[:64], B])
    assert np.array_equal(t0, t1[:64])
    assert np.array_equal(core.join_agg("ij,jk->ik", [A, B]), t1)


# ---------------------------------------------------------------------------------------------
# paper pins: spec enumeration, multiplicities, cost counts, overlay
# ---------------------------------------------------------------------------------------------
def _distinct_out_types(spec):
    seen = {}
    for cell in spec.cells:
        c = spec.block_coords(cell, -1)
        lo, hi = spec.bounds(c, -1)
        seen[spec.flat_key(c, -1)] = {"lower": lo, "upper": hi}
    return [seen[k] for k in sorted(seen)]


def test_matmul_decomposed_example(golden_dir):
    g = _golden(golden_dir, "matmul_decomposed.json")
    two = blocked.Spec(g["einsum"], g["two_spec"]["parts"])
    assert two.p == g["two_spec"]["num_function_specs"]
    assert _distinct_out_types(two) == g["two_spec"]["distinct_output_types"]
    assert two.multiplicity().tolist() == g["two_spec"]["multiplicity"]
    cols = [two.bounds(two.block_coords(c, 0), 0) for c in two.cells]
    assert [[lo[1], hi[1]] for lo, hi in cols] == g["two_spec"]["A_columns"]
    four = blocked.Spec(g["einsum"], g["four_spec"]["parts"])
    assert [four.nb[c] for c in "ijk"] == [g["four_spec"]["intervals"][c] for c in "ijk"]
    assert four.p == g["four_spec"]["num_function_specs"] == 2 * 2 * 1
    assert _distinct_out_types(four) == g["four_spec"]["distinct_output_types"]
    assert four.multiplicity().tolist() == g["four_spec"]["multiplicity"]
    # F_{m,n}: rows in the m-th half of i, columns in the n-th half of j, times rows in the n-th half of j
    ink, outk = four.tuples()
    assert ink.tolist() == [[0, 0], [1, 1], [2, 0], [3, 1]] and outk.tolist() == [0, 0, 1, 1]


def test_cost_closed_form(golden_dir):
    g = _golden(golden_dir, "cost_3d_matmul.json")
    for c in g["cases"]:
        N = c["N"]
        spec = blocked.Spec("ij,jk->ik", {"i": blocked.equal_splits(N, c["a"]), "j": blocked.equal_splits(N, c["b"]),
                                          "k": blocked.equal_splits(N, c["c"])})
        assert spec.p == c["a"] * c["b"] * c["c"]
        assert spec.cost_terms() == (c["join"], c["agg"]) == ((c["a"] + c["c"]) * N * N, (c["b"] - 1) * N * N)


def test_overlay_example(golden_dir):
    g = _golden(golden_dir, "overlay_example.json")
    over, atoms = blocked.overlay_atoms(g["producer_splits"], g["consumer_splits"])
    assert over[0] == g["overlay_row_split_points"] and over[1] == [0, 256]
    assert len(atoms) == g["num_atoms"]
    assert [a[2] for a in atoms] == g["atom_to_producer_block"]
    assert [a[3] for a in atoms] == g["atom_to_consumer_block"]
    assert all(g["atom_to_producer_block"].count(b) == g["atoms_per_producer_block"] for b in (0, 1))


def test_overlay_invariants_random():
    for _ in range(20):
        rank = int(RNG.integers(1, 4))
        ext = [int(RNG.integers(3, 12)) for _ in range(rank)]

        def rand_splits(e):
            cuts = sorted(set(RNG.integers(1, e, int(RNG.integers(0, 4))).tolist()))
            return [0] + cuts + [e]

        src = [rand_splits(e) for e in ext]
        dst = [rand_splits(e) for e in ext]
        _, atoms = blocked.overlay_atoms(src, dst)
        cover = np.zeros(ext, dtype=np.int32)
        _, slo, sup, _, _ = blocked.relation_keys(ext, src, 2)
        _, dlo, dup, _, _ = blocked.relation_keys(ext, dst, 2)
        for lo, hi, sb, db in atoms:
            cover[tuple(slice(l, h) for l, h in zip(lo, hi))] += 1
            for blo, bup in ((slo[sb], sup[sb]), (dlo[db], dup[db])):  # atom inside exactly one block of each family
                assert all(bl <= l and h <= bu for l, h, bl, bu in zip(lo, hi, blo, bup))
        assert (cover == 1).all()  # atoms tile the tensor


def test_tiling_validation():
    blocked.check_splits(8, [0, 3, 8])
    for bad in ([0, 3], [1, 8], [0, 5, 5, 8], [0, 6, 4, 8], [0]):
        with pytest.raises(ValueError):
            blocked.check_splits(8, bad)
    # brute-force cover + disjointness of the block types of a key table (Definition 3.2)
    ext, splits = [7, 5, 4], [[0, 2, 7], [0, 5], [0, 1, 3, 4]]
    _, lo, up, off, total = blocked.relation_keys(ext, splits, 2)
    cover = np.zeros(ext, dtype=int)
    for l, u in zip(lo, up):
        cover[tuple(slice(a, b) for a, b in zip(l, u))] += 1
    assert (cover == 1).all() and (off % 128 == 0).all() and total % 128 == 0
    assert blocked.equal_splits(10, 4) == [0, 2, 5, 7, 10]


# ---------------------------------------------------------------------------------------------
# decomposition invariance (Definition 3.7: every spec recovers the same output)
# ---------------------------------------------------------------------------------------------
def test_decomposition_invariance_config1():
    A = RNG.standard_normal((256, 256)).astype(np.float32).astype(np.float64)
    B = RNG.standard_normal((256, 256)).astype(np.float32).astype(np.float64)
    ref = core.matmul(A, B)
    for grid in ((4, 4, 4), (2, 8, 4), (1, 1, 1), (4, 8, 4)):
        parts = {c: blocked.equal_splits(256, n) for c, n in zip("ijk", grid)}
        got = blocked.t2_join_agg("ij,jk->ik", parts, [A, B])
        assert np.abs(got - ref).max() <= 1e-12 * np.abs(ref).max()
    np.testing.assert_allclose(ref, torch.from_numpy(A).matmul(torch.from_numpy(B)).numpy(), rtol=0, atol=1e-11)


@pytest.mark.parametrize("einsum,fn,agg", [("ij->i", "square", "sum"), ("hij->hi", "ident", "max"),
                                           ("ij,ij->ij", "silu_mul", "none"), ("ij,kj->ik", "mul", "sum")])
def test_decomposition_invariance_uneven(einsum, fn, agg):
    ins, out, letters = core.parse_einsum(einsum)
    ext = {c: int(RNG.integers(5, 11)) for c in letters}
    inputs = [RNG.standard_normal([ext[c] for c in t]) for t in ins]
    ref = core.join_agg(einsum, inputs, fn, agg)
    for _ in range(3):
        parts = {c: blocked.equal_splits(ext[c], int(RNG.integers(1, 4))) for c in letters}
        got = blocked.t2_join_agg(einsum, parts, inputs, fn, agg)
        np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)
        if agg == "max":
            assert np.array_equal(got, ref)


# ---------------------------------------------------------------------------------------------
# relation layout and repartition
# ---------------------------------------------------------------------------------------------
def test_pack_unpack_repartition():
    ext = [12, 10, 6]
    dense = RNG.integers(0, 60000, ext).astype(np.uint16)
    one = [[0, e] for e in ext]
    t1 = [[0, 5, 12], [0, 10], [0, 2, 6]]
    t2 = [[0, 4, 8, 12], [0, 3, 10], [0, 6]]
    p1 = blocked.pack(dense, t1)
    assert np.array_equal(blocked.unpack(p1, ext, t1), dense)
    # repartition to the one-block tiling = the dense row-major tensor
    assert np.array_equal(blocked.repartition(p1, ext, t1, one)[: dense.size], dense.reshape(-1))
    p2 = blocked.repartition(p1, ext, t1, t2)
    assert np.array_equal(p2, blocked.pack(dense, t2))                       # direct
    assert np.array_equal(blocked.repartition(p2, ext, t2, t1), p1)          # round trip
    via = blocked.repartition(blocked.repartition(p1, ext, t1, one), ext, one, t2)
    assert np.array_equal(via, p2)                                           # via an intermediate tiling


# ---------------------------------------------------------------------------------------------
# operators against closed forms and library routines
# ---------------------------------------------------------------------------------------------
def test_matmul_special_cases():
    A = RNG.standard_normal((9, 9))
    assert np.array_equal(core.matmul(A, np.eye(9)), A)
    perm = np.eye(9)[RNG.permutation(9)]
    assert np.array_equal(core.matmul(perm, A), perm @ A)
    # transposed operands would give A^T: the join must pair A's SECOND index with B's FIRST
    B = RNG.standard_normal((9, 4))
    assert np.abs(core.matmul(A, B) - A @ B).max() < 1e-13 and np.abs(core.matmul(A, B) - A.T @ B).max() > 1e-3


def test_silu_mul():
    t = RNG.standard_normal((7, 9)) * 4
    one = np.ones_like(t)
    s = core.join_agg("ij,ij->ij", [t, one], "silu_mul", "none")
    s_neg = core.join_agg("ij,ij->ij", [-t, one], "silu_mul", "none")
    np.testing.assert_allclose(s - s_neg, t, rtol=1e-13, atol=1e-13)          # silu(t) - silu(-t) = t
    assert core.join_agg("ij,ij->ij", [np.zeros((1, 1)), np.ones((1, 1))], "silu_mul", "none")[0, 0] == 0.0
    b = RNG.standard_normal((7, 9))
    want = (torch.nn.functional.silu(torch.from_numpy(t)) * torch.from_numpy(b)).numpy()
    np.testing.assert_allclose(core.join_agg("ij,ij->ij", [t, b], "silu_mul", "none"), want, rtol=1e-13, atol=1e-14)


def test_rmsnorm():
    X = RNG.standard_normal((6, 32)) * 2
    g = 1 + 0.1 * RNG.standard_normal(32)
    eps = 1e-5
    out = operators.rmsnorm(X, g, eps, out_dtype=None)
    want = torch.nn.functional.rms_norm(torch.from_numpy(X), (32,), torch.from_numpy(g), eps).numpy()
    np.testing.assert_allclose(out["y"], want, rtol=1e-6, atol=1e-7)  # ss is stored in fp32
    y1 = operators.rmsnorm(X, np.ones(32), eps, out_dtype=None)["y"]
    ms = (X * X).mean(axis=1)
    np.testing.assert_allclose((y1 * y1).mean(axis=1), ms / (ms + eps), rtol=1e-6)  # closed form with gamma = 1
    y_scaled = operators.rmsnorm(1000 * X, g, eps, out_dtype=None)["y"]
    np.testing.assert_allclose(y_scaled, out["y"], rtol=1e-4)                        # scale invariance (eps small)


def test_softmax():
    S = RNG.standard_normal((3, 5, 16)) * 2
    out = operators.softmax_rows(S, out_dtype=None)
    np.testing.assert_allclose(out["p"].sum(axis=-1), 1.0, rtol=1e-6)
    np.testing.assert_allclose(out["p"], torch.softmax(torch.from_numpy(S), -1).numpy(), rtol=1e-6, atol=1e-9)
    shifted = operators.softmax_rows(S + 3.0, out_dtype=None)["p"]
    np.testing.assert_allclose(shifted, out["p"], rtol=1e-6)
    assert np.array_equal(out["m"], S.max(axis=-1).astype(np.float32).astype(np.float64))


def test_attention_closed_forms_and_library():
    B, S, H, D = 2, 12, 3, 8
    Q, K, V = (RNG.standard_normal((B, S, H, D)) for _ in range(3))
    O = operators.attention(Q, K, V, out_dtype=None)
    t = lambda a: torch.from_numpy(a).permute(0, 2, 1, 3)
    want = torch.nn.functional.scaled_dot_product_attention(t(Q), t(K), t(V), is_causal=True).permute(0, 2, 1, 3).numpy()
    np.testing.assert_allclose(O, want, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(O[:, 0], V[:, 0], rtol=1e-14)                               # row 0 sees only key 0
    prefix_mean = np.cumsum(V, axis=1) / np.arange(1, S + 1)[None, :, None, None]
    np.testing.assert_allclose(operators.attention(0 * Q, K, V, out_dtype=None), prefix_mean, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(operators.attention(Q, K, np.ones_like(V), out_dtype=None), 1.0, rtol=1e-13)
    want_nc = torch.nn.functional.scaled_dot_product_attention(t(Q), t(K), t(V)).permute(0, 2, 1, 3).numpy()
    np.testing.assert_allclose(operators.attention(Q, K, V, causal=False, out_dtype=None), want_nc, rtol=1e-12, atol=1e-13)
    # S = 1: O = V
    np.testing.assert_allclose(operators.attention(Q[:, :1], K[:, :1], V[:, :1], out_dtype=None), V[:, :1], rtol=1e-14)
    # a subset of query rows, given their positions
    rows = np.array([0, 5, 11])
    np.testing.assert_array_equal(operators.attention(Q[:, rows], K, V, out_dtype=None, qpos=rows), O[:, rows])
    # the operator as an explicit chain of scalar-keyed join-aggs
    np.testing.assert_allclose(operators.attention_as_join_aggs(Q, K, V), O, rtol=1e-12, atol=1e-13)
    # Definition 3.7 with the KV index split inside the sequence and the triple aggregation
    for qs, ks in (([0, 4, 8, 12], [0, 4, 8, 12]), ([0, 12], [0, 3, 12]), ([0, 5, 12], [0, 2, 7, 12])):
        np.testing.assert_allclose(operators.attention_blocked(Q, K, V, qs, ks), O, rtol=1e-12, atol=1e-13)


def test_online_softmax_aggregation_is_a_valid_aggregation():
    def rand_triple():
        return RNG.standard_normal((4, 3)), RNG.standard_normal(4) * 3, np.abs(RNG.standard_normal(4)) + 0.1

    a, b, c = rand_triple(), rand_triple(), rand_triple()
    comb = operators.softmax_triple_combine
    for x, y in zip(comb(a, b), comb(b, a)):
        np.testing.assert_allclose(x, y, rtol=1e-14)                       # commutative
    for x, y in zip(comb(comb(a, b), c), comb(a, comb(b, c))):
        np.testing.assert_allclose(x, y, rtol=1e-12)                       # associative
    ident = (np.zeros((4, 3)), np.full(4, -np.inf), np.zeros(4))
    for x, y in zip(comb(a, ident), a):
        np.testing.assert_array_equal(x, y)                                # identity (0, -inf, 0)
    for x, y in zip(comb(ident, ident), ident):
        np.testing.assert_array_equal(x, y)


def test_rope_properties():
    B, S, H, D = 1, 9, 2, 8
    x, y = RNG.standard_normal((B, S, H, D)), RNG.standard_normal((B, S, H, D))
    rx = operators.rope(x, 1e4, out_dtype=None)
    np.testing.assert_allclose(rx[:, 0], x[:, 0], rtol=1e-15)                               # t = 0 is the identity
    pair_norm = lambda a: a.reshape(B, S, H, D // 2, 2) ** 2
    np.testing.assert_allclose(pair_norm(rx).sum(-1), pair_norm(x).sum(-1), rtol=1e-12)     # rotation
    # <RoPE(q, t1), RoPE(k, t2)> depends on t1 - t2 only
    q, k = x[0, 0, 0], y[0, 0, 0]

    def at(vec, t):
        return operators.rope(vec.reshape(1, 1, 1, D), 1e4, out_dtype=None, pos=[t])[0, 0, 0]

    assert abs(at(q, 7) @ at(k, 3) - at(q, 5) @ at(k, 1)) < 1e-12
    assert abs(at(q, 7) @ at(k, 3) - at(q, 4) @ at(k, 1)) > 1e-6
    # pair p = 0 rotates by exactly t radians; pair p by t * theta^(-2p/d); (1, 0) -> (cos, sin)
    e = np.zeros((1, 1, 1, 4)); e[..., 0] = 1.0; e[..., 2] = 1.0
    r = operators.rope(e, 100.0, out_dtype=None, pos=[3])[0, 0, 0]
    np.testing.assert_allclose(r, [math.cos(3), math.sin(3), math.cos(3 / 10.0), math.sin(3 / 10.0)], rtol=1e-14)


def _torch_block(x, w, n_heads, theta, eps):
    """An independent composition from torch-CPU fp64 library routines (no rounding anywhere)."""
    T = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    x = T(x)
    S, hidden = x.shape
    d = hidden // n_heads
    n1 = torch.nn.functional.rms_norm(x, (hidden,), T(w["g1"]), eps)
    q, k, v = (n1 @ T(w[n]) for n in ("wq", "wk", "wv"))

    def rot(t):
        t = t.reshape(S, n_heads, d // 2, 2)
        ang = torch.arange(S, dtype=torch.float64)[:, None] * theta ** (-torch.arange(0, d, 2, dtype=torch.float64) / d)
        z = torch.view_as_complex(t.contiguous()) * torch.polar(torch.ones_like(ang), ang)[:, None, :]
        return torch.view_as_real(z).reshape(S, n_heads, d)

    q, k, v = rot(q), rot(k), v.reshape(S, n_heads, d)
    att = torch.nn.functional.scaled_dot_product_attention(q.transpose(0, 1), k.transpose(0, 1), v.transpose(0, 1),
                                                           is_causal=True).transpose(0, 1).reshape(S, hidden)
    h = x + att @ T(w["wo"])
    n2 = torch.nn.functional.rms_norm(h, (hidden,), T(w["g2"]), eps)
    y = (torch.nn.functional.silu(n2 @ T(w["w1"])) * (n2 @ T(w["w3"]))) @ T(w["w2"])
    return (h + y).numpy()


def test_llama_block_composition():
    S, hidden, ffn, H = 10, 16, 24, 2
    x = RNG.standard_normal((S, hidden))
    w = {n: RNG.standard_normal(s) * 0.3 for n, s in (("wq", (hidden, hidden)), ("wk", (hidden, hidden)),
         ("wv", (hidden, hidden)), ("wo", (hidden, hidden)), ("w1", (hidden, ffn)), ("w3", (hidden, ffn)),
         ("w2", (ffn, hidden)))}
    w["g1"], w["g2"] = 1 + 0.1 * RNG.standard_normal(hidden), 1 + 0.1 * RNG.standard_normal(hidden)
    full = operators.llama_block(x, w, H, 1e4, 1e-5, dtype=None)
    np.testing.assert_allclose(full["out"], _torch_block(x, w, H, 1e4, 1e-5), rtol=1e-5, atol=1e-6)
    rows = np.array([0, 3, 9])
    sub = operators.llama_block(x, w, H, 1e4, 1e-5, rows=rows, dtype=None)
    np.testing.assert_array_equal(sub["out"], full["out"][rows])
    # with storage rounding the result stays within bf16 distance of the unrounded one
    b16 = operators.llama_block(x, w, H, 1e4, 1e-5, dtype="bf16")["out"]
    assert np.linalg.norm(b16 - full["out"]) / np.linalg.norm(full["out"]) < 2e-2


# ---------------------------------------------------------------------------------------------------
# grouped-query attention and packed sequences (Example 3.10)
# ---------------------------------------------------------------------------------------------------
def test_gqa_packed_spec_example(golden_dir):
    g = _golden(golden_dir, "gqa_packed_example.json")
    Hq, Hkv, grp, S = g["heads_q"], g["heads_kv"], g["group"], g["sequence_extent"]
    es = "bqhd,bkgd,bkgd->bqhd"
    parts = {"b": [0, 1], "q": [0, S], "h": [grp * m for m in range(Hkv + 1)], "d": [0, 128], "k": [0, S],
             "g": list(range(Hkv + 1))}
    spec = blocked.Spec(es, parts, induced=("h", "g", grp))
    assert spec.p == g["num_function_specs_when_heads_kv_is_cut_into_unit_intervals"]
    for cell in spec.cells:   # the m-th specification: key/value head m, query heads [4m, 4(m+1))
        m = cell[spec.letters.index("g")]
        lo, hi = spec.bounds(spec.block_coords(cell, 0), 0)
        assert [lo[2], hi[2]] == [grp * m, grp * (m + 1)]
        if str(m) in g["query_head_interval_of_kv_head"]:
            assert [lo[2], hi[2]] == g["query_head_interval_of_kv_head"][str(m)]
    with pytest.raises(ValueError):   # heads_q is not shardable on its own
        blocked.Spec(es, dict(parts, h=[0, 16, 32]), induced=("h", "g", grp))
    ends = g["sequence_ends"]
    parts2 = dict(parts, q=[0] + ends, k=[0] + ends)
    spec2 = blocked.Spec(es, parts2, induced=("h", "g", grp), segments=("k", "q", ends), band=("k", "q"))
    assert spec2.p == g["num_function_specs_when_sequence_is_cut_at_its_ends_and_heads_kv_into_unit_intervals"]
    assert (spec2.multiplicity() == 1).all()     # pure join + recompose: no aggregation (as the paper notes)
    with pytest.raises(ValueError):   # a cut that is not at a sequence end and removes an end is refused
        blocked.Spec(es, dict(parts, q=[0, 2048, S], k=[0, 2048, S]), induced=("h", "g", grp), segments=("k", "q", ends))


def test_gqa_packed_attention_against_library():
    B, S, Hq, Hkv, D = 1, 24, 4, 2, 8
    ends = [5, 16, 24]
    Q = RNG.standard_normal((B, S, Hq, D))
    K, V = RNG.standard_normal((B, S, Hkv, D)), RNG.standard_normal((B, S, Hkv, D))
    got = operators.attention_gqa_packed(Q, K, V, group=2, ends=ends, causal=True, out_dtype=None)
    # torch: repeat the kv heads, block-diagonal causal mask
    t = lambda a: torch.from_numpy(a).permute(0, 2, 1, 3)
    seq = np.searchsorted(np.array(ends), np.arange(S), side="right")
    mask = torch.from_numpy((seq[:, None] == seq[None, :]) & (np.arange(S)[None, :] <= np.arange(S)[:, None]))
    want = torch.nn.functional.scaled_dot_product_attention(t(Q), t(K).repeat_interleave(2, dim=1), t(V).repeat_interleave(2, dim=1),
                                                            attn_mask=mask).permute(0, 2, 1, 3).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)
    # one sequence, group 1 reduces to plain attention
    np.testing.assert_array_equal(operators.attention_gqa_packed(Q, Q, Q, 1, None, True, None), operators.attention(Q, Q, Q, True, None))
    # the first row of every sequence sees only itself
    for s0 in [0] + ends[:-1]:
        np.testing.assert_allclose(got[:, s0], V[:, s0].repeat(2, axis=1), rtol=1e-14)


# ---------------------------------------------------------------------------------------------------
# producers compiled through their join + the aggregating relayout (Sections 5.1, 5.3)
# ---------------------------------------------------------------------------------------------------
def test_preamble_example_atoms_and_aggregates(golden_dir):
    g = _golden(golden_dir, "preamble_example.json")
    ext, src, dst = g["extents"], g["producer_splits"], g["consumer_splits"]
    # label every cell of copy X of atom j with j and of copy Y with 10 j: OUT must hold 11 j in consumer block j-1
    P = np.zeros([g["copies_per_block"]] + ext)
    for name, info in g["in"].items():
        for j in info["atoms"]:
            r0, r1 = g["atom_rows"][str(j)]
            P[info["copy"], r0:r1] = j * (1 if name == "X" else 10)
    out = blocked.aggregate_repartition(P, src, dst, "sum")
    payload = blocked.pack(out, dst)
    _, lower, upper, offsets, _ = blocked.relation_keys(ext, dst, 8)
    for req in g["out"]:
        j = int(req["sum_of"][0][1:])
        assert req["sum_of"] == [f"X{j}", f"Y{j}"]
        b = req["consumer_block"]
        n = int(np.prod(upper[b] - lower[b]))
        blk = payload[offsets[b] // 8: offsets[b] // 8 + n]
        assert (blk == 11 * j).all() and [int(lower[b][0]), int(upper[b][0])] == g["atom_rows"][str(j)]


def test_join_partials_sum_to_the_aggregated_output():
    A, B = RNG.standard_normal((24, 30)), RNG.standard_normal((30, 20))
    parts = {"i": [0, 8, 24], "j": [0, 10, 20, 30], "k": [0, 5, 20]}
    P = blocked.join_partials("ij,jk->ik", parts, [A, B])
    assert P.shape == (3, 24, 20)
    np.testing.assert_allclose(P.sum(axis=0), A @ B, rtol=1e-12, atol=1e-12)       # plain definition
    for c, (j0, j1) in enumerate(zip(parts["j"], parts["j"][1:])):                 # copy c = contracted block c
        np.testing.assert_allclose(P[c], A[:, j0:j1] @ B[j0:j1], rtol=1e-12, atol=1e-12)
    src = [parts["i"], parts["k"]]
    for dst in (src, [[0, 24], [0, 20]], [[0, 3, 12, 24], [0, 7, 11, 20]]):
        out = blocked.aggregate_repartition(P, src, dst, "sum")
        # same (+) order as Definition 3.7's aggregate step: bit-equal to the one-shot implementation
        np.testing.assert_array_equal(out, blocked.t2_join_agg("ij,jk->ik", parts, [A, B]))
    with pytest.raises(ValueError):    # several copies of an atom and no aggregation operator
        blocked.aggregate_repartition(P, src, src, "none")


def test_aggregate_repartition_against_dense_reduction_and_plain_repartition():
    ext = [20, 12]
    src, dst = [[0, 7, 20], [0, 4, 12]], [[0, 5, 10, 20], [0, 12]]
    P = RNG.standard_normal([4] + ext)
    # brute force through an independent route: pack copies, unpack to dense, reduce with numpy
    payload = blocked.pack(P, blocked.partial_splits(4, src))
    dense = blocked.unpack(payload, [4] + ext, blocked.partial_splits(4, src))
    np.testing.assert_array_equal(dense, P)
    np.testing.assert_array_equal(blocked.aggregate_repartition(P, src, dst, "max"), dense.max(axis=0))
    np.testing.assert_allclose(blocked.aggregate_repartition(P, src, dst, "sum"), dense.sum(axis=0), rtol=1e-13, atol=1e-13)
    # ascending copy order, one rounding at the store
    s = ((P[0] + P[1]) + P[2]) + P[3]
    np.testing.assert_array_equal(blocked.aggregate_repartition(P, src, dst, "sum", "bf16"), core.round_to(s, "bf16"))
    # one copy: the aggregating relayout is the plain relayout, bit for bit
    one = blocked.pack(P[:1], blocked.partial_splits(1, src))
    got = blocked.pack(blocked.aggregate_repartition(P[:1], src, dst, "none"), dst)
    np.testing.assert_array_equal(got, blocked.repartition(one, ext, src, dst))


# ---------------------------------------------------------------------------------------------------
# logical optimization (Section 4): Algorithm 1 against the paper's 3D matmul, a hand-costed chain and exhaustive search
# ---------------------------------------------------------------------------------------------------
def _mlp_tree(T, d, f):
    return [{"einsum": "ij,jk->ik", "extents": {"i": T, "j": d, "k": f}, "inputs": [None, None]},
            {"einsum": "ij,jk->ik", "extents": {"i": T, "j": d, "k": f}, "inputs": [None, None]},
            {"einsum": "ik,ik->ik", "extents": {"i": T, "k": f}, "inputs": [0, 1]},
            {"einsum": "ik,kl->il", "extents": {"i": T, "k": f, "l": d}, "inputs": [2, None]}]


def test_optimizer_recovers_3d_matmul_and_hand_costed_chain(golden_dir):
    from oracle import optimizer
    g = _golden(golden_dir, "optimizer_example.json")
    for c in g["three_d"]:
        N, p, q = c["N"], c["p"], c["q"]
        op = {"einsum": "ij,jk->ik", "extents": {"i": N, "j": N, "k": N}, "inputs": [None, None]}
        for J in optimizer.specs(op, p):
            assert optimizer.cost(op, J, [None, None]) == (J["i"] + J["j"] + J["k"] - 1) * N * N
        total, plan = optimizer.optimize_tree([op], p)
        assert total == (3 * q - 1) * N * N and plan == [{"i": q, "j": q, "k": q}]
    ch = g["chain"]
    for pc in ch["plan_costs"]:
        assert optimizer.plan_cost(ch["ops"], pc["plan"]) == pc["cost"]
    total, plan = optimizer.optimize_tree(ch["ops"], ch["p"])
    assert total == ch["optimum"] and plan == ch["plan_costs"][0]["plan"]


def test_optimizer_dynamic_program_equals_exhaustive_search():
    from oracle import optimizer
    trees = [(_mlp_tree(8, 6, 12), 4),
             ([{"einsum": "ij,jk->ik", "extents": {"i": 6, "j": 9, "k": 4}, "inputs": [None, None]},
               {"einsum": "ik,kl->il", "extents": {"i": 6, "k": 4, "l": 10}, "inputs": [0, None]},
               {"einsum": "il->i", "extents": {"i": 6, "l": 10}, "inputs": [1]}], 6),
             ([{"einsum": "bqhd,bkhd->bhqk", "extents": {"b": 2, "q": 8, "h": 4, "d": 4, "k": 8}, "inputs": [None, None], "fixed": {"d"}},
               {"einsum": "bhqk,bkhd->bqhd", "extents": {"b": 2, "h": 4, "q": 8, "k": 8, "d": 4}, "inputs": [0, None], "fixed": {"d"}}], 4)]
    for ops, p in trees:
        dp_cost, dp_plan = optimizer.optimize_tree(ops, p)
        ex_cost, _ = optimizer.exhaustive(ops, p)
        assert dp_cost == ex_cost == optimizer.plan_cost(ops, dp_plan)
        for op, J in zip(ops, dp_plan):
            assert int(np.prod(list(J.values()))) == p and all(J[c] == 1 for c in op.get("fixed", ()))


def test_attention_lse_combines_partial_results():
    """The second attention output pins itself against the first: attention over two disjoint key ranges, combined with
    weights exp(lse_i - lse), must equal attention over all keys (the O side comes from the C engine, lse from numpy)."""
    B, S, H, D = 2, 24, 3, 8
    Q, K, V = (RNG.standard_normal((B, S, H, D)) for _ in range(3))
    lse = operators.attention_lse(Q, K, causal=False).astype(np.float64)
    want = operators.attention(Q, K, V, causal=False, out_dtype=None)
    parts = []
    for k0, k1 in ((0, 10), (10, 24)):
        parts.append((operators.attention(Q, K[:, k0:k1], V[:, k0:k1], causal=False, out_dtype=None),
                      operators.attention_lse(Q, K[:, k0:k1], causal=False).astype(np.float64)))
    tot = np.log(sum(np.exp(l) for _, l in parts))
    np.testing.assert_allclose(tot, lse, rtol=1e-6, atol=1e-6)                      # f32-rounded statistics
    got = sum(o * np.exp(l - tot)[..., None] for o, l in parts)
    np.testing.assert_allclose(got, want, rtol=1e-5, atol=1e-6)
    # causal: the first row joins one key, so lse is that single score; closed form
    lc = operators.attention_lse(Q, K, causal=True).astype(np.float64)
    np.testing.assert_allclose(lc[:, 0], np.einsum("bhd,bhd->bh", Q[:, 0], K[:, 0]) / np.sqrt(D), rtol=1e-6, atol=1e-6)
    # all keys equal: lse = score + log(number of keys)
    K1 = np.repeat(K[:, :1], S, axis=1)
    np.testing.assert_allclose(operators.attention_lse(Q, K1, causal=False), np.einsum("bqhd,bhd->bqh", Q, K[:, 0]) / np.sqrt(D) + np.log(S), rtol=1e-6, atol=1e-6)


def test_attention_combine_equals_attention_over_all_keys():
    """operators.attention_combine against the plain definition: attention over three disjoint key ranges, combined,
    equals attention over all keys -- also causal, where a whole key range lies after some query rows (their partial is
    empty: lse = -inf, and must drop out), and the order of the partials does not matter."""
    B, S, H, D = 2, 24, 3, 8
    Q, K, V = (RNG.standard_normal((B, S, H, D)) for _ in range(3))
    ranges = ((0, 7), (7, 16), (16, 24))
    for causal in (False, True):
        want = operators.attention(Q, K, V, causal=causal, out_dtype=None)
        want_l = operators.attention_lse(Q, K, causal=causal)
        o_parts, l_parts = [], []
        for k0, k1 in ranges:
            if causal:   # key i of the range sits at position k0 + i: query q sees it iff i <= q - k0; rows before k0 see none of it
                o = np.zeros_like(Q)                             # what an empty partial holds is never looked at
                o[:, k0:] = operators.attention(Q[:, k0:], K[:, k0:k1], V[:, k0:k1], causal=True, out_dtype=None,
                                                qpos=np.minimum(np.arange(k0, S) - k0, k1 - k0 - 1))
                o_parts.append(o)
                l_parts.append(operators.attention_lse(Q, K[:, k0:k1], causal=True, qpos=np.arange(S) - k0))
            else:
                o_parts.append(operators.attention(Q, K[:, k0:k1], V[:, k0:k1], causal=False, out_dtype=None))
                l_parts.append(operators.attention_lse(Q, K[:, k0:k1], causal=False))
        if causal:
            assert np.isneginf(l_parts[2][:, :16]).all() and np.isfinite(l_parts[2][:, 16:]).all()     # the case does hold empty partials
        got, got_l = operators.attention_combine(o_parts, l_parts, out_dtype=None)
        np.testing.assert_allclose(got, want, rtol=1e-5, atol=1e-6)
        np.testing.assert_allclose(got_l, want_l, rtol=1e-6, atol=1e-6)
        rev, rev_l = operators.attention_combine(o_parts[::-1], l_parts[::-1], out_dtype=None)
        np.testing.assert_allclose(rev, got, rtol=1e-12, atol=1e-12)
        # one partial alone is returned as it is; a row without any key gives O = 0 and lse = -inf
        one, one_l = operators.attention_combine(o_parts[:1], l_parts[:1], out_dtype=None)
        np.testing.assert_allclose(one, o_parts[0], rtol=1e-12, atol=0)
    z, zl = operators.attention_combine([np.ones((1, 2, 1, 4))], [np.full((1, 2, 1), -np.inf)], out_dtype=None)
    assert np.array_equal(z, np.zeros((1, 2, 1, 4))) and np.isneginf(zl).all()


def _block_graph(T=16, d=8, f=12, S=4):
    """The operators of a transformer block as a DAG with multiply consumed tensors (x, n1, h): small extents."""
    E = lambda **k: k
    return [
        {"einsum": "ij,j->ij", "extents": E(i=T, j=d), "inputs": [None, None]},                       # 0 n1 = norm(x)
        {"einsum": "ij,jk->ik", "extents": E(i=T, j=d, k=d), "inputs": [0, None]},                    # 1 q
        {"einsum": "ij,jk->ik", "extents": E(i=T, j=d, k=d), "inputs": [0, None]},                    # 2 k
        {"einsum": "ij,jk->ik", "extents": E(i=T, j=d, k=d), "inputs": [0, None]},                    # 3 v
        {"einsum": "ik,ik,ik->ik", "extents": E(i=T, k=d), "inputs": [1, 2, 3]},                      # 4 att (row-local stand-in)
        {"einsum": "ik,kl,il->il", "extents": E(i=T, k=d, l=d), "inputs": [4, None, None]},           # 5 h = x + att Wo
        {"einsum": "ij,j->ij", "extents": E(i=T, j=d), "inputs": [5, None]},                          # 6 n2
        {"einsum": "ij,jk->ik", "extents": E(i=T, j=d, k=f), "inputs": [6, None]},                    # 7 a
        {"einsum": "ij,jk->ik", "extents": E(i=T, j=d, k=f), "inputs": [6, None]},                    # 8 b
        {"einsum": "ik,ik->ik", "extents": E(i=T, k=f), "inputs": [7, 8]},                            # 9 silu(a) b
        {"einsum": "ik,kl,il->il", "extents": E(i=T, k=f, l=d), "inputs": [9, None, 5]},              # 10 out = h + . W2
    ]


def test_optimizer_graph_cut_into_trees():
    from oracle import optimizer
    ops = _block_graph()
    trees = optimizer.cut_into_trees(ops)
    # multiply consumed: n1 (0), h (5), n2 (6); final: 10
    assert sorted(r for r, _ in trees) == [0, 5, 6, 10]
    assert dict(trees)[5] == [1, 2, 3, 4, 5] and dict(trees)[10] == [7, 8, 9, 10] and dict(trees)[0] == [0] and dict(trees)[6] == [6]
    assert [r for r, _ in trees] == [5, 10, 0, 6]                        # largest first, ties by root
    for p in (2, 4):
        total, plan = optimizer.optimize_graph(ops, p)
        assert total == optimizer.plan_cost(ops, plan)
        # the tree optimised last cannot be improved with everything else fixed (its root's consumers included)
        last_root, members = trees[-1]
        for alt in itertools.product(*[optimizer.specs(ops[i], p) for i in members]):
            trial = list(plan)
            for i, J in zip(members, alt):
                trial[i] = J
            assert optimizer.plan_cost(ops, trial) >= total
    # on a tree the graph procedure is Algorithm 1
    tree = _mlp_tree(8, 6, 12)
    assert optimizer.optimize_graph(tree, 4)[0] == optimizer.optimize_tree(tree, 4)[0]
