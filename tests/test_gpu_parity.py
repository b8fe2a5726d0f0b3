"""GPU parity: every kernel of libja, called through the C ABI, against the CPU oracle on the same seeded
inputs, element by element. Sizes here are small enough for the oracle to finish in seconds and still span
several tiles, several blocks and ragged tails. Tolerances: relative Frobenius error 1e-5 for f32 relations,
2e-2 for bf16 and 2.5e-3 for f16 relations (f32 accumulation); bit-exact for MAX aggregation and for every relayout.
The f16 cases of the contractions, attention, the fused chains and the block are in test_gpu_f16.py."""
import numpy as np
import pytest
import torch

import paper_2609_03905_b200 as ja
import synth_inputs as si
from oracle import blocked, core, operators

from gpu_util import TOL, check_status, download, download_bits, empty_like_tiling, np_bits, relfro, upload

pytestmark = pytest.mark.gpu
ES = blocked.equal_splits
BF, F32, F16 = torch.bfloat16, torch.float32, torch.float16
ORC_DT = {BF: "bf16", F32: "f32", F16: "f16"}

# every attention kernel form, forced through the library's switches (conftest.py puts them back after each test)
ATTN_FORMS = ["tcgen05_two_tiles", "tcgen05_two_tiles_persistent", "tcgen05_two_tiles_poly_exp", "tcgen05_two_tiles_exp_first", "tcgen05_one_tile", "mma_sync"]


def force_attention_form(form):
    ja.ja_debug_set("attn_mma_sync", 1 if form == "mma_sync" else 0)
    ja.ja_debug_set("attn_one_tile", 1 if form == "tcgen05_one_tile" else 0)
    ja.ja_debug_set("attn_persistent", 0 if form == "tcgen05_two_tiles" else 1)
    ja.ja_debug_set("attn_variant", 3 if form.endswith("poly_exp") else 4 if form.endswith("exp_first") else 0 if form == "tcgen05_two_tiles" else -1)


def _matmul_case(M, J, N, si_, sj, sk, dtype, cfg=1, std_b=1.0):
    A = si.normal((M, J), 0.0, 1.0, dtype, cfg, 1)
    Bm = si.normal((J, N), 0.0, std_b, dtype, cfg, 2)
    parts = {"i": si_, "j": sj, "k": sk}
    spec = ja.Spec("ij,jk->ik", parts, "mul", (), "sum")
    rA, rB = upload(A, [si_, sj]), upload(Bm, [sj, sk])
    rC = empty_like_tiling([M, N], [si_, sk], dtype, fill=float("nan"))
    spec.execute([rA, rB], rC)
    got = download(rC)
    check_status()
    ref = operators.matmul(si.to_f64(A), si.to_f64(Bm), ORC_DT[dtype])
    return got, ref


# ---------------------------------------------------------------------------------------------------
# config 1: matmul as a join-agg, f32, 256^3; decomposition invariance
# ---------------------------------------------------------------------------------------------------
def test_config1_matmul_f32_decompositions():
    outs = {}
    for grid in ((4, 4, 4), (2, 8, 4), (1, 1, 1), (4, 8, 4)):
        got, ref = _matmul_case(256, 256, 256, ES(256, grid[0]), ES(256, grid[1]), ES(256, grid[2]), F32)
        assert relfro(got, ref) <= TOL[F32], grid
        outs[grid] = got
    base = outs[(1, 1, 1)]
    for grid, got in outs.items():  # every block decomposition of the same operator yields the same result
        assert relfro(got, base) <= TOL[F32], grid


def test_matmul_plain_alu_uneven_tilings():
    got, ref = _matmul_case(100, 77, 90, [0, 33, 100], [0, 10, 50, 77], [0, 64, 65, 90], F32)
    assert relfro(got, ref) <= TOL[F32]
    got, ref = _matmul_case(70, 50, 45, [0, 70], [0, 17, 50], [0, 20, 45], BF)     # bf16 on irregular blocks
    assert relfro(got, ref) <= TOL[BF]


def test_degenerate_tilings_scalar_keys_and_single_block():
    """The two ends of the decomposition space: every sub-tensor one scalar (the classical relational form: key = cell,
    p = 12 * 10 * 9 function specs, m = 10 tuples per output key) and one block per relation (p = 1, no aggregation)."""
    unit = lambda n: list(range(n + 1))
    for dt in (F32, BF):
        got, ref = _matmul_case(12, 10, 9, unit(12), unit(10), unit(9), dt)
        assert relfro(got, ref) <= TOL[dt]
        got1, ref1 = _matmul_case(12, 10, 9, [0, 12], [0, 10], [0, 9], dt)
        assert relfro(got1, ref1) <= TOL[dt] and relfro(got, got1) <= TOL[dt]
    # relayout between the two ends, bit-exact both ways
    x = si.normal((12, 9), 0.0, 1.0, F32, 1, 7)
    one, cells = [[0, 12], [0, 9]], [unit(12), unit(9)]
    r1 = upload(x, one)
    rc = empty_like_tiling([12, 9], cells, F32)
    ja.repartition(r1, rc)
    assert np.array_equal(download_bits(rc), blocked.pack(np_bits(x), cells))
    back = empty_like_tiling([12, 9], one, F32)
    ja.repartition(rc, back)
    assert np.array_equal(download_bits(back), download_bits(r1))
    # a row-structured join-agg over scalar blocks (sum of squares: m = 9 tuples per row key)
    ss = ja.Relation([12], [unit(12)], F32)
    ja.Spec("ij->i", {"i": unit(12), "j": unit(9)}, "square", (), "sum").execute([rc], ss)
    assert relfro(download(ss), operators.sumsq_rows(si.to_f64(x))) <= TOL[F32]
    check_status()


# ---------------------------------------------------------------------------------------------------
# tensor-core matmul join-agg (bf16 relations, uniform blocks)
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("M,J,N,gi,gj,gk", [
    (256, 256, 512, 2, 2, 2),      # 128x128 / 128x256 blocks: one full tile per output key
    (256, 512, 256, 1, 4, 1),      # m = 4 tuples per output key, 256-row block = two row tiles
    (384, 192, 640, 3, 3, 1),      # 64-deep contraction blocks, 640-wide block = 256+256+128 tiles
    (256, 704, 352, 2, 2, 2),      # ragged: 352-deep blocks (5.5 k-steps), 176-wide blocks (N = 176)
    (256, 128, 512, 4, 1, 8),      # 64-row and 64-column blocks: tiles span several output keys
    (512, 256, 384, 2, 2, 3),      # 128-wide blocks: a 256-column tile covers two output keys (+ tail)
    (200, 160, 136, 1, 1, 1),      # one ragged block: 200 rows (128+72), 136 columns
])
@pytest.mark.parametrize("cta_group", ["2", "1"])   # two-SM tiles where the shape allows them / one-SM tiles everywhere
def test_matmul_tensor_core(M, J, N, gi, gj, gk, cta_group):
    ja.ja_debug_set("gemm_cta_group", int(cta_group))
    got, ref = _matmul_case(M, J, N, ES(M, gi), ES(J, gj), ES(N, gk), BF, cfg=2, std_b=0.05)
    assert relfro(got, ref) <= TOL[BF]
    # the error must look like bf16 rounding of the output, not like a dropped k-step or a misplaced tile
    assert np.abs(got - ref).max() <= 2.0 ** -7 * np.abs(ref).max() + 1e-6


# the same contraction with operands staged by plain loads: the tensor-core form for tilings TMA cannot address
@pytest.mark.parametrize("M,J,N,si_,sj,sk", [
    (256, 256, 512, ES(256, 2), ES(256, 2), ES(512, 2)),                   # TMA-friendly blocks, loader forced
    (384, 704, 640, ES(384, 3), ES(704, 2), ES(640, 1)),                   # 352-deep blocks (5.5 stages), three column tiles
    (512, 1376, 344, ES(512, 2), ES(1376, 8), ES(344, 2)),                 # 172-cell block rows: 8-byte aligned only
    (300, 330, 270, [0, 100, 300], [0, 130, 330], [0, 135, 270]),          # odd widths: 2-byte aligned rows, ragged everything
    (260, 200, 522, [0, 129, 260], [0, 67, 200], [0, 261, 522]),           # irregular blocks a cell past a tile / stage boundary
    (1024, 96, 256, ES(1024, 1), ES(96, 1), ES(256, 1)),                   # one block, 96-deep: a stage and a half
])
def test_matmul_tensor_core_plain_load_form(M, J, N, si_, sj, sk):
    ja.ja_debug_set("gemm_loader", 1)
    before = ja.ja_launch_count()
    got, ref = _matmul_case(M, J, N, si_, sj, sk, BF, cfg=2, std_b=0.05)
    assert ja.ja_launch_count() == before + 1
    assert relfro(got, ref) <= TOL[BF]
    assert np.abs(got - ref).max() <= 2.0 ** -7 * np.abs(ref).max() + 1e-6
    # the plain-ALU kernel on the same tiling gives the same result up to its different summation order
    ja.ja_debug_set("gemm_loader", 0)
    ja.ja_debug_set("gemm_cta_group", 1)
    if any(len(set(np.diff(sp))) > 1 or np.diff(sp)[0] % 8 for sp in (sj, sk)) or len(set(np.diff(si_))) > 1:
        alu, _ = _matmul_case(M, J, N, si_, sj, sk, BF, cfg=2, std_b=0.05)      # this tiling has no TMA form: plain ALUs
        assert relfro(got, alu) <= 1e-2


def test_matmul_tensor_core_identity_is_exact():
    M = 256
    A = si.normal((M, M), 0.0, 1.0, BF, 2, 3)
    eye = torch.eye(M, dtype=BF)
    sp = ES(M, 2)
    spec = ja.Spec("ij,jk->ik", {"i": sp, "j": sp, "k": sp})
    rC = empty_like_tiling([M, M], [sp, sp], BF, fill=float("nan"))
    spec.execute([upload(A, [sp, sp]), upload(eye, [sp, sp])], rC)
    assert np.array_equal(download(rC), si.to_f64(A))
    rC2 = empty_like_tiling([M, M], [sp, sp], BF, fill=float("nan"))
    spec.execute([upload(eye, [sp, sp]), upload(A, [sp, sp])], rC2)
    assert np.array_equal(download(rC2), si.to_f64(A))
    check_status()


# ---------------------------------------------------------------------------------------------------
# repartition: bit-exact block relayout
# ---------------------------------------------------------------------------------------------------
def test_repartition_bit_exact():
    rng = np.random.default_rng(5)
    cases = [([256, 256], [ES(256, 2), [0, 256]], [ES(256, 4), [0, 256]], BF),       # the paper's overlay example
             ([512, 1024], [ES(512, 4), ES(1024, 2)], [ES(512, 4), ES(1024, 8)], BF),
             ([96, 200], [[0, 31, 96], [0, 7, 200]], [[0, 50, 96], [0, 100, 101, 200]], BF),  # odd offsets: 2-byte path
             ([2, 64, 4, 128], [[0, 1, 2], ES(64, 2), [0, 4], [0, 128]], [[0, 2], ES(64, 4), ES(4, 4), [0, 128]], BF),
             ([33, 17, 9], [[0, 33], [0, 5, 17], [0, 9]], [[0, 10, 33], [0, 17], [0, 4, 9]], F32),
             ([1000], [[0, 1000]], [ES(1000, 7)], F32)]
    for ext, s_sp, d_sp, dt in cases:
        if dt == BF:
            dense = torch.from_numpy(rng.integers(0, 1 << 16, ext, dtype=np.uint16).view(np.int16)).view(BF)
        else:
            dense = torch.from_numpy(rng.standard_normal(ext).astype(np.float32))
        src = upload(dense, s_sp)
        dst = empty_like_tiling(ext, d_sp, dt)
        ja.repartition(src, dst)
        want = blocked.repartition(np_bits(src.payload.cpu()), ext, s_sp, d_sp)
        assert np.array_equal(download_bits(dst), want)
        back = empty_like_tiling(ext, s_sp, dt)
        ja.repartition(dst, back)                                                    # round trip
        assert np.array_equal(download_bits(back), download_bits(src))
        one = empty_like_tiling(ext, [[0, e] for e in ext], dt)
        ja.repartition(src, one)                                                     # one block = the dense tensor
        assert np.array_equal(download_bits(one)[: dense.numel()], np_bits(dense).reshape(-1))
        via = empty_like_tiling(ext, d_sp, dt)
        ja.repartition(one, via)                                                     # via an intermediate = direct
        assert np.array_equal(download_bits(via), want)
        # the library's own packing helper agrees with the oracle's packing
        assert np.array_equal(download_bits(ja.from_dense(dense.cuda(), d_sp)), want)
        assert np.array_equal(np_bits(ja.to_dense(dst)), np_bits(dense))
    check_status()


# ---------------------------------------------------------------------------------------------------
# memory-bound join-aggs
# ---------------------------------------------------------------------------------------------------
TILINGS_2D = [((256, 1024), ES(256, 2), ES(1024, 8)),           # 128-bit path, m = 8 column blocks per row key
              ((64, 4096), ES(64, 1), ES(4096, 8)),              # LLaMA row length
              ((40, 8192), ES(40, 2), ES(8192, 8)),              # 65B row length: two warps per row
              ((37, 300), [0, 5, 37], [0, 7, 150, 300]),         # irregular splits: scalar path
              ((9, 20000), [0, 9], ES(20000, 2))]                # long row: streaming path


@pytest.mark.parametrize("dtype", [BF, F32, F16])
@pytest.mark.parametrize("shape,si_,sj", TILINGS_2D)
def test_rmsnorm_join_aggs(shape, si_, sj, dtype):
    X = si.normal(shape, 0.0, 2.0, dtype, 3, 1)
    G = si.normal((shape[1],), 1.0, 0.1, dtype, 3, 2)
    ref = operators.rmsnorm(si.to_f64(X), si.to_f64(G), 1e-5, ORC_DT[dtype])
    rX, rG = upload(X, [si_, sj]), upload(G, [sj])
    parts = {"i": si_, "j": sj}
    # SUM-of-squares aggregation, then the key-aligned scale join
    rSS = empty_like_tiling([shape[0]], [si_], F32, fill=float("nan"))
    ja.Spec("ij->i", parts, "square", (), "sum").execute([rX], rSS)
    assert relfro(download(rSS), ref["ss"]) <= 1e-5
    rY = empty_like_tiling(list(shape), [si_, sj], dtype, fill=float("nan"))
    ja.Spec("ij,i,j->ij", parts, "rms_scale", (1e-5,), "none").execute([rX, rSS, rG], rY)
    assert relfro(download(rY), ref["y"]) <= TOL[dtype]
    # the fused chain
    rY2 = empty_like_tiling(list(shape), [si_, sj], dtype, fill=float("nan"))
    ja.Spec("ij,j->ij", parts, "rmsnorm", (1e-5,), "none").execute([rX, rG], rY2)
    assert relfro(download(rY2), ref["y"]) <= TOL[dtype]
    check_status()


@pytest.mark.parametrize("dtype", [BF, F32, F16])
@pytest.mark.parametrize("shape,sh,si_,sj", [((4, 64, 2048), ES(4, 4), ES(64, 2), ES(2048, 8)),
                                             ((2, 17, 300), [0, 2], [0, 5, 17], [0, 7, 150, 300]),
                                             ((1, 8, 20000), [0, 1], [0, 8], ES(20000, 2))])
def test_softmax_join_aggs(shape, sh, si_, sj, dtype):
    S = si.normal(shape, 0.0, 2.0, dtype, 3, 3)
    ref = operators.softmax_rows(si.to_f64(S), ORC_DT[dtype])
    rS = upload(S, [sh, si_, sj])
    parts = {"h": sh, "i": si_, "j": sj}
    stat = lambda: empty_like_tiling(list(shape[:2]), [sh, si_], F32, fill=float("nan"))
    rM, rL = stat(), stat()
    ja.Spec("hij->hi", parts, "ident", (), "max").execute([rS], rM)
    assert np.array_equal(download(rM), ref["m"])                                   # MAX aggregation is exact
    ja.Spec("hij,hi->hi", parts, "exp_sub", (), "sum").execute([rS, rM], rL)
    assert relfro(download(rL), ref["l"]) <= 1e-5
    rP = empty_like_tiling(list(shape), [sh, si_, sj], dtype, fill=float("nan"))
    ja.Spec("hij,hi,hi->hij", parts, "exp_sub_div", (), "none").execute([rS, rM, rL], rP)
    assert relfro(download(rP), ref["p"]) <= TOL[dtype]
    rP2 = empty_like_tiling(list(shape), [sh, si_, sj], dtype, fill=float("nan"))
    ja.Spec("hij->hij", parts, "softmax", (), "none").execute([rS], rP2)
    assert relfro(download(rP2), ref["p"]) <= TOL[dtype]
    check_status()


@pytest.mark.parametrize("dtype", [BF, F32, F16])
@pytest.mark.parametrize("form", [1, 0])     # the plain read-stream kernel for all three statistics / never
def test_row_statistics_both_forms(dtype, form):
    """Sum of squares, row maximum and sum of exponentials as statistics-only join-aggs through both kernels that take
    them on uniform tilings (by default the choice depends on the form and the size), incl. rows that are not a whole
    number of 32-vector steps, three leading indices and more rows than resident warps."""
    ja.ja_debug_set("row_reduce", form)
    for shape, splits in (((6000, 1024), [ES(6000, 3), ES(1024, 8)]),
                          ((3, 40, 2000), [ES(3, 3), ES(40, 2), ES(2000, 5)]),
                          ((2, 3, 16, 264), [ES(2, 1), ES(3, 3), ES(16, 4), ES(264, 1)])):
        X = si.normal(shape, 0.0, 2.0, dtype, 3, 7)
        x64 = si.to_f64(X).reshape(-1, shape[-1])
        rX = upload(X, splits)
        letters = "abcd"[: len(shape) - 1]
        parts = dict(zip(letters + "j", splits))
        stat = lambda: empty_like_tiling(list(shape[:-1]), splits[:-1], F32, fill=float("nan"))
        rSS, rM, rL = stat(), stat(), stat()
        before = ja.ja_launch_count()
        ja.Spec(f"{letters}j->{letters}", parts, "square", (), "sum").execute([rX], rSS)
        ja.Spec(f"{letters}j->{letters}", parts, "ident", (), "max").execute([rX], rM)
        ja.Spec(f"{letters}j,{letters}->{letters}", parts, "exp_sub", (), "sum").execute([rX, rM], rL)
        assert ja.ja_launch_count() == before + 3
        m = x64.max(axis=1)
        assert relfro(download(rSS).reshape(-1), (x64 * x64).sum(axis=1)) <= 1e-5
        assert np.array_equal(download(rM).reshape(-1), m)
        assert relfro(download(rL).reshape(-1), np.exp(x64 - m[:, None]).sum(axis=1)) <= 1e-5
    check_status()


@pytest.mark.parametrize("dtype", [BF, F32, F16])
def test_key_aligned_maps(dtype):
    for shape, sp in (((256, 1376), [ES(256, 2), ES(1376, 1)]), ((50, 70), [[0, 13, 50], [0, 33, 70]])):
        a = si.normal(shape, 0.0, 1.5, dtype, 2, 4)
        b = si.normal(shape, 0.0, 1.0, dtype, 2, 5)
        parts = {"i": sp[0], "j": sp[1]}
        rA, rB = upload(a, sp), upload(b, sp)
        rO = empty_like_tiling(list(shape), sp, dtype, fill=float("nan"))
        ja.Spec("ij,ij->ij", parts, "silu_mul", (), "none").execute([rA, rB], rO)
        assert relfro(download(rO), operators.silu_mul(si.to_f64(a), si.to_f64(b), ORC_DT[dtype])) <= TOL[dtype]
        rO2 = empty_like_tiling(list(shape), sp, dtype, fill=float("nan"))
        ja.Spec("ij,ij->ij", parts, "add", (), "none").execute([rA, rB], rO2)
        want = operators.add(si.to_f64(a), si.to_f64(b), ORC_DT[dtype])
        if dtype == F16:    # the f32 sum of two f16 cells is not always exact (27 bits): rounded twice in rare cells
            assert relfro(download(rO2), want) <= 1e-4
        else:
            assert np.array_equal(download(rO2), want)                          # one exact rounding
    check_status()


@pytest.mark.parametrize("splits", [[[0, 1, 2], ES(256, 2), ES(4, 4), [0, 128]],
                                    [[0, 2], ES(256, 4), [0, 4], [0, 128]],
                                    [[0, 2], [0, 100, 256], [0, 1, 4], [0, 64, 128]]])
def test_rope(splits):
    x = si.normal((2, 256, 4, 128), 0.0, 1.0, BF, 5, 11)
    rX = upload(x, splits)
    rY = empty_like_tiling(list(x.shape), splits, BF, fill=float("nan"))
    ja.Spec("bshd->bshd", dict(zip("bshd", splits)), "rope", (1e4,), "none").execute([rX], rY)
    assert relfro(download(rY), operators.rope(si.to_f64(x), 1e4, "bf16")) <= 4e-3
    check_status()


# ---------------------------------------------------------------------------------------------------
# attention join-agg
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("B,S,H,qb,kb,hb,causal", [(1, 256, 2, 128, 128, 1, True), (2, 512, 2, 128, 128, 2, True),
                                                   (1, 256, 1, 64, 64, 1, True), (1, 384, 2, 128, 64, 1, False),
                                                   (1, 512, 1, 256, 128, 1, True), (2, 1024, 3, 128, 256, 3, True),
                                                   (1, 640, 2, 128, 128, 1, False)])
@pytest.mark.parametrize("form", ATTN_FORMS)
def test_attention(B, S, H, qb, kb, hb, causal, form):
    force_attention_form(form)
    D = 128
    Q, K, V = (si.normal((B, S, H, D), 0.0, 1.0, BF, 4, o) for o in (1, 2, 3))
    spl = lambda blk: [ES(B, B), ES(S, S // blk), ES(H, H // hb), [0, D]]
    rQ, rK, rV = upload(Q, spl(qb)), upload(K, spl(kb)), upload(V, spl(kb))
    rO = empty_like_tiling([B, S, H, D], spl(qb), BF, fill=float("nan"))
    parts = {"b": ES(B, B), "q": ES(S, S // qb), "h": ES(H, H // hb), "d": [0, D], "k": ES(S, S // kb)}
    spec = ja.Spec("bqhd,bkhd,bkhd->bqhd", parts, "attention", (1.0 / np.sqrt(D), 1.0 if causal else 0.0), "online_softmax")
    spec.execute([rQ, rK, rV], rO)
    got = download(rO)
    check_status()
    ref = operators.attention(si.to_f64(Q), si.to_f64(K), si.to_f64(V), causal, "bf16")
    assert relfro(got, ref) <= TOL[BF]
    assert np.abs(got - ref).max() <= 0.05
    if causal:
        assert np.array_equal(got[:, 0], si.to_f64(V)[:, 0])   # row 0 joins with key 0 only: O = V[0] exactly


@pytest.mark.parametrize("form", ATTN_FORMS)
@pytest.mark.parametrize("causal", [False, True])
def test_attention_scores_that_grow_along_the_keys(causal, form):
    """Keys whose magnitude grows from one 128-row key tile to the next: the running row maximum then outgrows the exponent
    offset in use by more than the 2^8 head-room at almost every key tile, so the kernels take their offset-raising path
    (rescale of the accumulated output, and in the two-tile form the redo of a tile that was exponentiated against the
    old offset) instead of the common one that N(0,1) inputs exercise."""
    force_attention_form(form)
    B, S, H, D = 1, 1024, 2, 128
    Q, K, V = (si.normal((B, S, H, D), 0.0, 1.0, BF, 4, o) for o in (31, 32, 33))
    growth = 1.0 + 3.0 * (np.arange(S) // 128)              # score spread x1, x4, x7, ... per key tile
    K = (si.to_f64(K) * growth[None, :, None, None]).astype(np.float32)
    K = torch.from_numpy(K).to(torch.bfloat16)
    sp = [ES(B, B), ES(S, S // 128), ES(H, H), [0, D]]
    rQ, rK, rV = upload(Q, sp), upload(K, sp), upload(V, sp)
    rO = empty_like_tiling([B, S, H, D], sp, BF, fill=float("nan"))
    rL = empty_like_tiling([B, S, H], sp[:3], F32, fill=float("nan"))
    parts = {"b": sp[0], "q": sp[1], "h": sp[2], "d": sp[3], "k": sp[1]}
    spec = ja.Spec("bqhd,bkhd,bkhd->bqhd", parts, "attention", (1.0 / np.sqrt(D), 1.0 if causal else 0.0), "online_softmax")
    spec.execute([rQ, rK, rV], [rO, rL])
    got, got_l = download(rO), download(rL)
    check_status()
    ref = operators.attention(si.to_f64(Q), si.to_f64(K), si.to_f64(V), causal, "bf16")
    assert relfro(got, ref) <= TOL[BF]
    ref_l = operators.attention_lse(si.to_f64(Q), si.to_f64(K), causal)
    assert np.abs(got_l - ref_l).max() <= 2e-3 * max(1.0, np.abs(ref_l).max())
    # the case does what it is for: the row maximum of the last key tile exceeds that of the first by far more than 8 / log2(e)
    s = np.einsum("qd,kd->qk", si.to_f64(Q)[0, :, 0], si.to_f64(K)[0, :, 0]) / np.sqrt(D)
    assert np.median(s[:, -128:].max(1) - s[:, :128].max(1)) > 20.0


@pytest.mark.parametrize("form", ATTN_FORMS)
@pytest.mark.parametrize("causal,S,hb", [(True, 512, 1), (False, 384, 2), (True, 256, 2)])
def test_attention_second_output_lse(causal, S, hb, form):
    """n_outputs = 2: the log of the softmax denominator beside O, and the combine it exists for."""
    force_attention_form(form)
    B, H, D = 2, 4, 128
    Q, K, V = (si.normal((B, S, H, D), 0.0, 1.0, BF, 4, o) for o in (21, 22, 23))
    sp = [ES(B, B), ES(S, S // 128), ES(H, H // hb), [0, D]]
    rQ, rK, rV = upload(Q, sp), upload(K, sp), upload(V, sp)
    rO = empty_like_tiling([B, S, H, D], sp, BF, fill=float("nan"))
    rL = empty_like_tiling([B, S, H], sp[:3], F32, fill=float("nan"))
    parts = {"b": sp[0], "q": sp[1], "h": sp[2], "d": sp[3], "k": sp[1]}
    spec = ja.Spec("bqhd,bkhd,bkhd->bqhd", parts, "attention", (1.0 / np.sqrt(D), 1.0 if causal else 0.0), "online_softmax")
    spec.execute([rQ, rK, rV], [rO, rL])
    got_o, got_l = download(rO), download(rL)
    check_status()
    assert relfro(got_o, operators.attention(si.to_f64(Q), si.to_f64(K), si.to_f64(V), causal, "bf16")) <= TOL[BF]
    ref_l = operators.attention_lse(si.to_f64(Q), si.to_f64(K), causal)
    assert np.abs(got_l - ref_l).max() <= 2e-3        # absolute: lse is a logarithm; 2e-3 = a relative 2e-3 on the denominator
    with pytest.raises(ja.JaError):                   # the second output must be tiled like the first
        spec.execute([rQ, rK, rV], [rO, empty_like_tiling([B, S, H], [sp[0], ES(S, 1), sp[2]], F32)])


# grouped-query attention over packed sequences (Example 3.10): query head h joins key/value head h // group and
# no tuple crosses a sequence end. `cut` says where the sequence index is split: "ends" = at the sequence ends only
# (irregular blocks), an integer = uniform blocks of that many rows (every end is then a split point).
@pytest.mark.parametrize("B,S,Hq,Hkv,gblk,ends,cut,causal", [
    (1, 512, 4, 2, 1, [128, 384, 512], 128, True),          # ends at odd multiples of 128: one-tile kernel
    (2, 1024, 8, 2, 1, [256, 768, 1024], "ends", True),     # the paper's cut: blocks of 256, 512, 256 rows
    (1, 1024, 4, 4, 2, [512, 1024], "ends", False),         # group 1, two heads per block, not causal
    (1, 512, 2, 1, 1, [64, 320, 512], 64, True),            # 64-row granularity: mma.sync form
    (2, 768, 6, 2, 2, [768], 256, True),                    # one sequence, grouped heads only
    (1, 1280, 4, 1, 1, [256, 384, 1280], "ends", True),     # blocks of 256, 128, 896 rows
])
@pytest.mark.parametrize("form", ATTN_FORMS)
def test_attention_grouped_heads_packed_sequences(B, S, Hq, Hkv, gblk, ends, cut, causal, form):
    force_attention_form(form)
    D, grp = 128, Hq // Hkv
    Q = si.normal((B, S, Hq, D), 0.0, 1.0, BF, 4, 11)
    K, V = (si.normal((B, S, Hkv, D), 0.0, 1.0, BF, 4, o) for o in (12, 13))
    s_split = [0] + ends if cut == "ends" else ES(S, S // cut)
    g_split = ES(Hkv, Hkv // gblk)
    h_split = [grp * x for x in g_split]
    q_sp = [ES(B, B), s_split, h_split, [0, D]]
    k_sp = [ES(B, B), s_split, g_split, [0, D]]
    rQ, rK, rV = upload(Q, q_sp), upload(K, k_sp), upload(V, k_sp)
    rO = empty_like_tiling([B, S, Hq, D], q_sp, BF, fill=float("nan"))
    parts = {"b": q_sp[0], "q": s_split, "h": h_split, "d": [0, D], "k": s_split, "g": g_split}
    prm = (1.0 / np.sqrt(D), 1.0 if causal else 0.0) + tuple(float(e) for e in ends)
    spec = ja.Spec("bqhd,bkgd,bkgd->bqhd" if grp > 1 else "bqhd,bkhd,bkhd->bqhd",
                   parts if grp > 1 else {k: v for k, v in parts.items() if k != "g"}, "attention", prm, "online_softmax")
    spec.execute([rQ, rK, rV], rO)
    got = download(rO)
    check_status()
    ref = operators.attention_gqa_packed(si.to_f64(Q), si.to_f64(K), si.to_f64(V), grp, ends, causal, "bf16")
    assert relfro(got, ref) <= TOL[BF]
    assert np.abs(got - ref).max() <= 0.05
    if causal:   # the first row of every sequence joins with its own key only: O = V exactly
        for s0 in [0] + ends[:-1]:
            assert np.array_equal(got[:, s0], np.repeat(si.to_f64(V)[:, s0], grp, axis=1))


# ---------------------------------------------------------------------------------------------------
# the online-softmax aggregation as a step of its own: partial attention results over disjoint key ranges, combined
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [BF, F16, F32])
@pytest.mark.parametrize("m,same_tiling", [(1, False), (3, False), (3, True)])
def test_attention_combine_of_partial_results(m, same_tiling, dtype):
    """Function specs of one output key executed apart: m attention calls (n_outputs = 2), each over its own 256 keys, then
    ja_attention_combine -- against attention over all m * 256 keys at once (oracle), with the partial and the output
    relations each in a tiling of its own. f32 partials come from the oracle (attention itself takes 16-bit relations)."""
    B, S, H, D = 2, 256, 4, 128
    adt = BF if dtype == F32 else dtype
    Q = si.normal((B, S, H, D), 0.0, 1.0, adt, 4, 61)
    K, V = (si.normal((B, m * S, H, D), 0.0, 1.0, adt, 4, o) for o in (62, 63))
    tilings = [[ES(B, B), ES(S, 2), ES(H, H), [0, D]], [ES(B, 1), ES(S, 4), ES(H, 2), [0, D]], [ES(B, B), [0, 100, 256], [0, 1, 4], [0, D]]]
    if same_tiling:      # one tiling for every relation: rows addressed by arithmetic instead of through the key tables
        tilings = [tilings[0]] * 3
    o_parts, l_parts, ref_o, ref_l = [], [], [], []
    for c in range(m):
        sp = tilings[c % 3]
        Kc, Vc = K[:, c * S:(c + 1) * S].contiguous(), V[:, c * S:(c + 1) * S].contiguous()
        ref_o.append(operators.attention(si.to_f64(Q), si.to_f64(Kc), si.to_f64(Vc), False, ORC_DT[dtype]))
        ref_l.append(operators.attention_lse(si.to_f64(Q), si.to_f64(Kc), False))
        if dtype == F32 or (c % 3 == 2 and not same_tiling):      # oracle partials (f32, or the irregular tiling attention is not run on here)
            o_parts.append(upload(torch.from_numpy(ref_o[-1]).to(dtype), sp))
            l_parts.append(upload(torch.from_numpy(ref_l[-1]).to(F32), sp[:3]))
            continue
        rQ, rK, rV = upload(Q, sp), upload(Kc, sp), upload(Vc, sp)
        rO = empty_like_tiling([B, S, H, D], sp, dtype, fill=float("nan"))
        rL = empty_like_tiling([B, S, H], sp[:3], F32, fill=float("nan"))
        parts = {"b": sp[0], "q": sp[1], "h": sp[2], "d": sp[3], "k": sp[1]}
        ja.Spec("bqhd,bkhd,bkhd->bqhd", parts, "attention", (1.0 / np.sqrt(D), 0.0), "online_softmax").execute([rQ, rK, rV], [rO, rL])
        o_parts.append(rO)
        l_parts.append(rL)
    out_sp = tilings[0] if same_tiling else [ES(B, B), ES(S, 1), ES(H, 4), [0, D]]
    rO = empty_like_tiling([B, S, H, D], out_sp, dtype, fill=float("nan"))
    rL = empty_like_tiling([B, S, H], out_sp[:3], F32, fill=float("nan"))
    before = ja.ja_launch_count()
    ja.attention_combine(o_parts, l_parts, rO, rL)
    assert ja.ja_launch_count() == before + 1
    got, got_l = download(rO), download(rL)
    check_status()
    want = operators.attention(si.to_f64(Q), si.to_f64(K), si.to_f64(V), False, ORC_DT[dtype])           # all keys at once
    want_l = operators.attention_lse(si.to_f64(Q), si.to_f64(K), False)
    assert relfro(got, want) <= (2e-3 if dtype == F32 else TOL[dtype])        # f32: the partials were rounded to f32, the exponentials are fast ones
    assert np.abs(got_l - want_l).max() <= 2e-3
    # the combine itself, on exactly the partials the GPU saw, is the oracle's combine up to rounding
    exact_o, exact_l = operators.attention_combine([download(r) for r in o_parts], [download(r) for r in l_parts], ORC_DT[dtype])
    assert relfro(got, exact_o) <= (1e-5 if dtype == F32 else 3e-3 if dtype == BF else 4e-4)
    assert np.abs(got_l - exact_l).max() <= 1e-5
    # a partial that holds nothing for some rows (lse = -inf, O unspecified -- here NaN) drops out of those rows
    if m == 3:
        l_parts[1].payload.fill_(float("-inf"))
        o_parts[1].payload.fill_(float("nan"))
        ja.attention_combine(o_parts, l_parts, rO, None)
        exact2, _ = operators.attention_combine([download(o_parts[0]), download(o_parts[2])], [download(l_parts[0]), download(l_parts[2])], ORC_DT[dtype])
        assert relfro(download(rO), exact2) <= (1e-5 if dtype == F32 else 3e-3 if dtype == BF else 4e-4)
        check_status()
    with pytest.raises(ja.JaError):      # an output may not alias a partial
        ja.attention_combine(o_parts, l_parts, o_parts[0], None)


# ---------------------------------------------------------------------------------------------------
# any other einsum: the definition executed cell by cell (no specialised kernel matches these signatures)
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("einsum,shapes,splits,fn,agg,dtype", [
    ("bij,bjk->bik", [(3, 20, 17), (3, 17, 12)], {"b": [0, 1, 3], "i": [0, 7, 20], "j": [0, 5, 17], "k": [0, 12]}, "mul", "sum", F32),   # batched matmul
    ("bij,bjk->bik", [(2, 16, 24), (2, 24, 8)], {"b": [0, 2], "i": ES(16, 2), "j": ES(24, 3), "k": ES(8, 1)}, "mul", "sum", BF),
    ("ij,kj->ik", [(18, 30), (11, 30)], {"i": [0, 4, 18], "j": [0, 9, 30], "k": [0, 11]}, "mul", "sum", F16),                          # second operand transposed
    ("ij,j->i", [(25, 40), (40,)], {"i": [0, 10, 25], "j": ES(40, 4)}, "mul", "sum", F32),                                             # matrix x vector
    ("i,j->ij", [(9,), (14,)], {"i": [0, 2, 9], "j": [0, 14]}, "mul", "none", F32),                                                    # outer product: nothing aggregated
    ("ij,jk,kl->il", [(6, 7), (7, 5), (5, 8)], {"i": [0, 6], "j": [0, 3, 7], "k": [0, 5], "l": [0, 1, 8]}, "mul", "sum", F32),         # three operands, two summed indices
    ("ijk->ik", [(5, 33, 6)], {"i": [0, 5], "j": [0, 20, 33], "k": ES(6, 2)}, "ident", "max", BF),                                     # MAX over a middle index
    ("ijk->i", [(7, 9, 10)], {"i": [0, 3, 7], "j": ES(9, 3), "k": [0, 10]}, "square", "sum", F32),                                     # two summed indices, one operand
    ("ij,ji->ij", [(12, 15), (15, 12)], {"i": ES(12, 3), "j": [0, 4, 15]}, "add", "none", F32),                                        # x + y^T: a join that is not key-aligned in storage
])
def test_general_einsum_runs_as_the_definition(einsum, shapes, splits, fn, agg, dtype):
    ins, out_letters = einsum.split("->")
    terms = ins.split(",")
    xs = [si.normal(sh, 0.0, 1.0, dtype, 1, 50 + k) for k, sh in enumerate(shapes)]
    rels = [upload(x, [splits[c] for c in t]) for x, t in zip(xs, terms)]
    ext = {c: splits[c][-1] for c in splits}
    rO = empty_like_tiling([ext[c] for c in out_letters], [splits[c] for c in out_letters], dtype, fill=float("nan"))
    before = ja.ja_launch_count()
    ja.Spec(einsum, splits, fn, (), agg).execute(rels, rO)
    assert ja.ja_launch_count() == before + 1
    got = download(rO)
    check_status()
    ref = core.join_agg(einsum, [si.to_f64(x) for x in xs], fn, agg)        # the scalar-keyed join + aggregation of the oracle
    if agg == "max":
        assert np.array_equal(got, ref)                                     # no arithmetic: exact in any dtype
    else:
        assert relfro(got, core.round_to(ref, ORC_DT[dtype])) <= TOL[dtype]


# Ragged attention: lengths, split points and sequence ends that are NOT multiples of 64 rows. Output key tiles then
# straddle blocks and packed sequences and run past the end of the index; the same-sequence / causal selection is applied
# per score and every row is located on its own.
@pytest.mark.parametrize("dtype", [BF, F16])
@pytest.mark.parametrize("B,S,Hq,Hkv,s_split,ends,causal", [
    (2, 100, 2, 2, [0, 100], [], True),                         # one short sequence in one block: a tile of 64 rows and one of 36
    (1, 200, 2, 2, [0, 37, 101, 200], [], False),               # odd split points, not causal
    (1, 333, 4, 2, [0, 50, 64, 131, 200, 333], [50, 131, 333], True),   # packed sequences that end inside tiles (every end is a split point, as the spec requires), grouped heads
    (2, 77, 2, 1, list(range(0, 77, 11)) + [77], [77], True),   # 11-row blocks
    (1, 64, 1, 1, [0, 1, 64], [1, 64], True),                   # a sequence of one row
])
def test_attention_ragged(B, S, Hq, Hkv, s_split, ends, causal, dtype):
    D, grp = 128, Hq // Hkv
    Q = si.normal((B, S, Hq, D), 0.0, 1.0, dtype, 4, 41)
    K, V = (si.normal((B, S, Hkv, D), 0.0, 1.0, dtype, 4, o) for o in (42, 43))
    g_split, h_split = ES(Hkv, Hkv), [grp * x for x in ES(Hkv, Hkv)]
    q_sp, k_sp = [ES(B, B), s_split, h_split, [0, D]], [ES(B, B), s_split, g_split, [0, D]]
    rQ, rK, rV = upload(Q, q_sp), upload(K, k_sp), upload(V, k_sp)
    rO = empty_like_tiling([B, S, Hq, D], q_sp, dtype, fill=float("nan"))
    rL = empty_like_tiling([B, S, Hq], q_sp[:3], F32, fill=float("nan"))
    parts = {"b": q_sp[0], "q": s_split, "h": h_split, "d": [0, D], "k": s_split, "g": g_split}
    prm = (1.0 / np.sqrt(D), 1.0 if causal else 0.0) + tuple(float(e) for e in ends)
    spec = ja.Spec("bqhd,bkgd,bkgd->bqhd" if grp > 1 else "bqhd,bkhd,bkhd->bqhd",
                   parts if grp > 1 else {k: v for k, v in parts.items() if k != "g"}, "attention", prm, "online_softmax")
    before = ja.ja_launch_count()
    spec.execute([rQ, rK, rV], [rO, rL])
    assert ja.ja_launch_count() == before + 1
    got, lse = download(rO), download(rL)          # download() checks the guard zones around both payloads
    check_status()
    ref = operators.attention_gqa_packed(si.to_f64(Q), si.to_f64(K), si.to_f64(V), grp, ends or None, causal, ORC_DT[dtype])
    assert relfro(got, ref) <= TOL[dtype]
    assert np.isfinite(lse).all()
    if causal:   # the first row of every sequence joins with its own key only: O = V exactly, lse = its one score
        for s0 in [0] + list(ends[:-1]):
            assert np.array_equal(got[:, s0], np.repeat(si.to_f64(V)[:, s0], grp, axis=1))
            q64, k64 = si.to_f64(Q)[:, s0], np.repeat(si.to_f64(K)[:, s0], grp, axis=1)
            assert np.abs(lse[:, s0] - (q64 * k64).sum(-1) / np.sqrt(D)).max() <= 2e-3


# ---------------------------------------------------------------------------------------------------
# fused chains on the tensor-core matmul: the accumulator goes through the next join-agg before its one store
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("cta_group", ["2", "1"])
@pytest.mark.parametrize("M,J,N,gi,gj,gk", [(512, 256, 512, 4, 2, 2), (256, 384, 1024, 2, 3, 8), (512, 512, 256, 2, 1, 2)])
def test_matmul_fused_chains(M, J, N, gi, gj, gk, cta_group):
    ja.ja_debug_set("gemm_cta_group", int(cta_group))
    A = si.normal((M, J), 0.0, 1.0, BF, 2, 6)
    W1 = si.normal((J, N), 0.0, 0.06, BF, 2, 7)
    W3 = si.normal((J, N), 0.0, 0.06, BF, 2, 8)
    R = si.normal((M, N), 0.0, 1.0, BF, 2, 9)
    ti, tj, tk = ES(M, gi), ES(J, gj), ES(N, gk)
    parts = {"i": ti, "j": tj, "k": tk}
    rA, rW1, rW3, rR = upload(A, [ti, tj]), upload(W1, [tj, tk]), upload(W3, [tj, tk]), upload(R, [ti, tk])
    a64 = core.matmul(si.to_f64(A), si.to_f64(W1))          # unrounded products: the fused forms store nothing in between
    b64 = core.matmul(si.to_f64(A), si.to_f64(W3))
    out = lambda: empty_like_tiling([M, N], [ti, tk], BF, fill=float("nan"))
    # MUL/SUM -> ADD
    rC = out()
    ja.Spec("ij,jk,ik->ik", parts, "matmul_add", (), "sum").execute([rA, rW1, rR], rC)
    assert relfro(download(rC), core.round_to(a64 + si.to_f64(R), "bf16")) <= 2e-3
    # two MUL/SUM -> SILU_MUL
    rC = out()
    ja.Spec("ij,jk,jk->ik", parts, "swiglu_up", (), "sum").execute([rA, rW1, rW3], rC)
    assert relfro(download(rC), operators.silu_mul(a64, b64, "bf16")) <= 3e-3
    # MUL/SUM -> ROPE: rows are 128-token sequences, columns 128-wide heads
    rC = out()
    ja.Spec("ij,jk->ik", parts, "matmul_rope", (1e4, 128, 128), "sum").execute([rA, rW1], rC)
    ref = operators.rope(a64.reshape(M // 128, 128, N // 128, 128), 1e4, "bf16").reshape(M, N)
    assert relfro(download(rC), ref) <= 3e-3
    check_status()


def test_fused_chain_refused_when_the_tiling_cannot_run_it():
    # 64-wide column blocks cannot hold the paired 128-column products of the fused SwiGLU chain: nothing is enqueued
    M, J, N = 256, 128, 256
    ti, tj, tk = ES(M, 2), ES(J, 1), ES(N, 4)
    rA = empty_like_tiling([M, J], [ti, tj], BF, fill=1.0)
    rW = empty_like_tiling([J, N], [tj, tk], BF, fill=1.0)
    rW3 = empty_like_tiling([J, N], [tj, tk], BF, fill=1.0)
    rC = empty_like_tiling([M, N], [ti, tk], BF, fill=0.0)
    with pytest.raises(ja.JaError) as e:
        ja.Spec("ij,jk,jk->ik", {"i": ti, "j": tj, "k": tk}, "swiglu_up", (), "sum").execute([rA, rW, rW3], rC)
    assert e.value.status_name == "JA_ERR_UNSUPPORTED"
    torch.cuda.synchronize()
    assert float(rC.payload.abs().max()) == 0.0


# ---------------------------------------------------------------------------------------------------
# a producer executed through its join + the aggregating relayout that consumes it (Sections 5.1, 5.3)
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("M,J,N,gi,gj,gk,dtype,pdtype", [
    (256, 512, 256, 2, 2, 1, BF, BF),          # the four-specification matmul of Example 3.8
    (512, 1024, 768, 2, 4, 3, BF, F32),        # tensor cores, accumulators kept in f32
    (256, 768, 512, 1, 3, 2, BF, BF),
    (96, 80, 72, 2, 5, 3, F32, F32),           # plain ALUs, ragged blocks
    (100, 90, 56, 3, 2, 2, BF, BF),            # bf16 on a tiling the tensor-core path cannot address
])
def test_join_only_matmul_partials(M, J, N, gi, gj, gk, dtype, pdtype):
    A = si.normal((M, J), 0.0, 1.0, dtype, 2, 21)
    Bm = si.normal((J, N), 0.0, 1.0, dtype, 2, 22)
    parts = {"i": ES(M, gi), "j": ES(J, gj), "k": ES(N, gk)}
    spec = ja.Spec("ij,jk->ik", parts)
    rA, rB = upload(A, [parts["i"], parts["j"]]), upload(Bm, [parts["j"], parts["k"]])
    rP = ja.partial_relation(gj, [M, N], [parts["i"], parts["k"]], pdtype)
    rP.payload.fill_(float("nan"))
    spec.execute_join([rA, rB], rP)
    got = download(rP)
    check_status()
    ref = blocked.join_partials("ij,jk->ik", parts, [si.to_f64(A), si.to_f64(Bm)], dtype=ORC_DT[pdtype])
    assert got.shape == (gj, M, N)
    for c in range(gj):
        assert relfro(got[c], ref[c]) <= TOL[pdtype], c
    # and the consumer's side: aggregate the copies into a different tiling
    dst_sp = [ES(M, 4), ES(N, 2)]
    rC = empty_like_tiling([M, N], dst_sp, dtype, fill=float("nan"))
    ja.repartition_agg(rP, "sum", rC)
    out = download(rC)
    check_status()
    want = blocked.aggregate_repartition(got, [parts["i"], parts["k"]], dst_sp, "sum", ORC_DT[dtype])
    if dtype == F32:
        assert relfro(out, want) <= 1e-6     # f32 additions in the oracle's order; the oracle adds in fp64 and rounds once
    else:
        assert np.mean(out != want) < 2e-3 and relfro(out, want) <= 1e-3   # double rounding f64->f32->bf16 flips rare ties
    assert relfro(out, operators.matmul(si.to_f64(A), si.to_f64(Bm), ORC_DT[dtype])) <= TOL[dtype]


@pytest.mark.parametrize("sdt,ddt", [(BF, BF), (F32, F32), (F32, BF), (BF, F32)])
@pytest.mark.parametrize("agg", ["sum", "max"])
@pytest.mark.parametrize("m,ext,src,dst", [
    (2, [256, 256], [[0, 128, 256], [0, 256]], [[0, 64, 128, 192, 256], [0, 256]]),       # the preamble example
    (5, [300, 200], [ES(300, 3), ES(200, 2)], [ES(300, 2), ES(200, 5)]),
    (3, [64, 40, 24], [ES(64, 2), ES(40, 1), ES(24, 3)], [ES(64, 4), ES(40, 5), ES(24, 1)]),
    (7, [33, 17], [[0, 10, 33], [0, 17]], [[0, 33], [0, 5, 17]]),                          # odd sizes: scalar accesses
    (1, [128, 96], [ES(128, 2), ES(96, 3)], [ES(128, 4), ES(96, 1)]),                      # one copy: a plain relayout
])
def test_aggregating_relayout(m, ext, src, dst, agg, sdt, ddt):
    P = si.normal([m] + ext, 0.0, 1.0, sdt, 3, 31)
    rP = upload(P, blocked.partial_splits(m, src))
    rD = empty_like_tiling(ext, dst, ddt, fill=float("nan"))
    before = download_bits(rP).copy()
    ja.repartition_agg(rP, agg if m > 1 else "none", rD)
    got = download(rD)
    check_status()
    assert np.array_equal(download_bits(rP), before)                      # partials are borrowed, unchanged
    P64 = si.to_f64(P)
    if agg == "max" or m == 1:
        want = blocked.aggregate_repartition(P64, src, dst, agg, ORC_DT[ddt])
        assert np.array_equal(got, want)                                  # MAX and plain relayout: bit-exact
    else:
        # the kernel adds in f32 in ascending copy order; restate that order in f32, then one rounding
        acc = P64[0].astype(np.float32)
        for c in range(1, m):
            acc = acc + P64[c].astype(np.float32)
        assert np.array_equal(got, core.round_to(acc.astype(np.float64), ORC_DT[ddt]))
        assert relfro(got, blocked.aggregate_repartition(P64, src, dst, "sum", ORC_DT[ddt])) <= TOL[ddt]
