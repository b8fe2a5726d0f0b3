"""GPU parity in IEEE half precision (JA_F16), the precision of the paper's experiments (Section 6): the same kernels as
the bf16 relations go through -- tensor-core contractions with f32 accumulation, attention with P and O in f16, the fused
chains, partial relations and their aggregating relayout, RoPE, relayouts -- against the fp64 oracle rounding once to
f16 at every store. Tolerance: 2.5e-3 relative Frobenius error (ten half-ulps of f16). The row-structured join-aggs and
the key-aligned maps take f16 as a third cell type in test_gpu_parity.py."""
import numpy as np
import pytest
import torch

import paper_2609_03905_b200 as ja
import synth_inputs as si
from oracle import blocked, core, operators

from gpu_util import TOL, check_status, download, download_bits, empty_like_tiling, np_bits, relfro, upload
from test_gpu_parity import _matmul_case, force_attention_form

pytestmark = pytest.mark.gpu
ES = blocked.equal_splits
F16, F32 = torch.float16, torch.float32


@pytest.mark.parametrize("M,J,N,gi,gj,gk", [
    (256, 256, 512, 2, 2, 2),      # one full tile per output key
    (256, 512, 256, 1, 4, 1),      # four tuples per output key
    (256, 704, 352, 2, 2, 2),      # ragged: 352-deep blocks, 176-wide blocks
    (200, 160, 136, 1, 1, 1),      # one ragged block
])
@pytest.mark.parametrize("cta_group", [2, 1])
def test_matmul_tensor_core_f16(M, J, N, gi, gj, gk, cta_group):
    ja.ja_debug_set("gemm_cta_group", cta_group)
    got, ref = _matmul_case(M, J, N, ES(M, gi), ES(J, gj), ES(N, gk), F16, cfg=2, std_b=0.05)
    assert relfro(got, ref) <= TOL[F16]
    assert np.abs(got - ref).max() <= 2.0 ** -10 * np.abs(ref).max() + 1e-6     # f16 rounding of the output, nothing larger


def test_f16_keeps_three_more_bits_than_bf16():
    """The same real-valued product stored in both 16-bit types: the f16 result must be the closer one by about 2^3 --
    a kernel that silently ran the bf16 path on f16 bits, or rounded to bf16 on the way, would fail this."""
    M, J, N = 256, 256, 256
    sp = [ES(M, 2), ES(J, 2), ES(N, 2)]
    errs = {}
    for dt in (F16, torch.bfloat16):
        got, _ = _matmul_case(M, J, N, *sp, dt, cfg=2, std_b=0.05)
        A, Bm = si.normal((M, J), 0.0, 1.0, dt, 2, 1), si.normal((J, N), 0.0, 0.05, dt, 2, 2)     # the inputs of that case
        errs[dt] = relfro(got, core.matmul(si.to_f64(A), si.to_f64(Bm)))                           # against the UNROUNDED product
    assert errs[F16] < errs[torch.bfloat16] / 5 and errs[torch.bfloat16] > 1e-3


@pytest.mark.parametrize("M,J,N,si_,sj,sk", [
    (512, 1376, 344, ES(512, 2), ES(1376, 8), ES(344, 2)),                 # 172-cell block rows: 8-byte aligned only
    (300, 330, 270, [0, 100, 300], [0, 130, 330], [0, 135, 270]),          # odd widths, ragged everything
])
def test_matmul_plain_load_and_plain_alu_forms_f16(M, J, N, si_, sj, sk):
    ja.ja_debug_set("gemm_loader", 1)                 # tensor cores fed by plain loads
    before = ja.ja_launch_count()
    got, ref = _matmul_case(M, J, N, si_, sj, sk, F16, cfg=2, std_b=0.05)
    assert ja.ja_launch_count() == before + 1
    assert relfro(got, ref) <= TOL[F16]
    ja.ja_debug_set("gemm_loader", 0)                 # plain ALUs
    alu, _ = _matmul_case(M, J, N, si_, sj, sk, F16, cfg=2, std_b=0.05)
    assert relfro(alu, ref) <= TOL[F16]
    small, ref_s = _matmul_case(70, 50, 45, [0, 70], [0, 17, 50], [0, 20, 45], F16)   # blocks under 64 cells: plain ALUs
    assert relfro(small, ref_s) <= TOL[F16]


@pytest.mark.parametrize("cta_group", [2, 1])
def test_matmul_fused_chains_f16(cta_group):
    ja.ja_debug_set("gemm_cta_group", cta_group)
    M, J, N, gi, gj, gk = 256, 384, 1024, 2, 3, 8
    A = si.normal((M, J), 0.0, 1.0, F16, 2, 6)
    W1 = si.normal((J, N), 0.0, 0.06, F16, 2, 7)
    W3 = si.normal((J, N), 0.0, 0.06, F16, 2, 8)
    R = si.normal((M, N), 0.0, 1.0, F16, 2, 9)
    ti, tj, tk = ES(M, gi), ES(J, gj), ES(N, gk)
    parts = {"i": ti, "j": tj, "k": tk}
    rA, rW1, rW3, rR = upload(A, [ti, tj]), upload(W1, [tj, tk]), upload(W3, [tj, tk]), upload(R, [ti, tk])
    a64 = core.matmul(si.to_f64(A), si.to_f64(W1))
    b64 = core.matmul(si.to_f64(A), si.to_f64(W3))
    out = lambda: empty_like_tiling([M, N], [ti, tk], F16, fill=float("nan"))
    rC = out()
    ja.Spec("ij,jk,ik->ik", parts, "matmul_add", (), "sum").execute([rA, rW1, rR], rC)
    assert relfro(download(rC), core.round_to(a64 + si.to_f64(R), "f16")) <= 3e-4
    rC = out()
    ja.Spec("ij,jk,jk->ik", parts, "swiglu_up", (), "sum").execute([rA, rW1, rW3], rC)
    assert relfro(download(rC), operators.silu_mul(a64, b64, "f16")) <= 5e-4
    rC = out()
    ja.Spec("ij,jk->ik", parts, "matmul_rope", (1e4, 128, 128), "sum").execute([rA, rW1], rC)
    ref = operators.rope(a64.reshape(M // 128, 128, N // 128, 128), 1e4, "f16").reshape(M, N)
    assert relfro(download(rC), ref) <= 5e-4
    # a chain whose relations mix the two 16-bit types is refused before anything runs
    rB = upload(R.to(torch.bfloat16), [ti, tk])
    with pytest.raises(ja.JaError) as e:
        ja.Spec("ij,jk,ik->ik", parts, "matmul_add", (), "sum").execute([rA, rW1, rB], out())
    assert e.value.status_name in ("JA_ERR_UNSUPPORTED", "JA_ERR_DTYPE")
    check_status()


@pytest.mark.parametrize("M,J,N,gi,gj,gk,pdtype", [(256, 512, 256, 2, 2, 1, F16), (512, 1024, 768, 2, 4, 3, F32),
                                                   (100, 90, 56, 3, 2, 2, F16)])
def test_join_only_partials_and_aggregating_relayout_f16(M, J, N, gi, gj, gk, pdtype):
    A = si.normal((M, J), 0.0, 1.0, F16, 2, 21)
    Bm = si.normal((J, N), 0.0, 0.25, F16, 2, 22)
    parts = {"i": ES(M, gi), "j": ES(J, gj), "k": ES(N, gk)}
    spec = ja.Spec("ij,jk->ik", parts)
    rA, rB = upload(A, [parts["i"], parts["j"]]), upload(Bm, [parts["j"], parts["k"]])
    rP = ja.partial_relation(gj, [M, N], [parts["i"], parts["k"]], pdtype)
    rP.payload.fill_(float("nan"))
    spec.execute_join([rA, rB], rP)
    got = download(rP)
    check_status()
    ref = blocked.join_partials("ij,jk->ik", parts, [si.to_f64(A), si.to_f64(Bm)], dtype={F16: "f16", F32: "f32"}[pdtype])
    for c in range(gj):
        assert relfro(got[c], ref[c]) <= TOL[pdtype], c
    dst_sp = [ES(M, 4), ES(N, 2)]
    rC = empty_like_tiling([M, N], dst_sp, F16, fill=float("nan"))
    ja.repartition_agg(rP, "sum", rC)
    out = download(rC)
    check_status()
    want = blocked.aggregate_repartition(got, [parts["i"], parts["k"]], dst_sp, "sum", "f16")
    assert np.mean(out != want) < 2e-3 and relfro(out, want) <= 2e-4       # f64 -> f32 -> f16 flips rare ties
    assert relfro(out, operators.matmul(si.to_f64(A), si.to_f64(Bm), "f16")) <= TOL[F16]
    # MAX aggregation of f16 partials is exact
    if pdtype == F16:
        rM = empty_like_tiling([M, N], dst_sp, F16, fill=float("nan"))
        ja.repartition_agg(rP, "max", rM)
        assert np.array_equal(download(rM), blocked.aggregate_repartition(got, [parts["i"], parts["k"]], dst_sp, "max", "f16"))


def test_relayout_and_rope_f16():
    rng = np.random.default_rng(11)
    for ext, s_sp, d_sp in (([512, 1024], [ES(512, 4), ES(1024, 2)], [ES(512, 4), ES(1024, 8)]),
                            ([96, 200], [[0, 31, 96], [0, 7, 200]], [[0, 50, 96], [0, 100, 101, 200]])):
        dense = torch.from_numpy(rng.integers(0, 1 << 16, ext, dtype=np.uint16).view(np.int16)).view(F16)   # any bit pattern
        src = upload(dense, s_sp)
        dst = empty_like_tiling(ext, d_sp, F16)
        ja.repartition(src, dst)
        assert np.array_equal(download_bits(dst), blocked.repartition(np_bits(src.payload.cpu()), ext, s_sp, d_sp))
        assert np.array_equal(np_bits(ja.to_dense(dst)), np_bits(dense))
    for splits in ([[0, 1, 2], ES(256, 2), ES(4, 4), [0, 128]], [[0, 2], [0, 100, 256], [0, 1, 4], [0, 64, 128]]):
        x = si.normal((2, 256, 4, 128), 0.0, 1.0, F16, 5, 11)
        rX = upload(x, splits)
        rY = empty_like_tiling(list(x.shape), splits, F16, fill=float("nan"))
        ja.Spec("bshd->bshd", dict(zip("bshd", splits)), "rope", (1e4,), "none").execute([rX], rY)
        assert relfro(download(rY), operators.rope(si.to_f64(x), 1e4, "f16")) <= 5e-4
    check_status()


@pytest.mark.parametrize("B,S,H,qb,kb,hb,causal", [(2, 512, 2, 128, 128, 2, True), (1, 384, 2, 128, 64, 1, False),
                                                   (1, 512, 1, 256, 128, 1, True), (1, 256, 1, 64, 64, 1, True)])
@pytest.mark.parametrize("form", ["tcgen05_two_tiles", "tcgen05_two_tiles_persistent", "tcgen05_one_tile", "mma_sync"])
def test_attention_f16(B, S, H, qb, kb, hb, causal, form):
    force_attention_form(form)
    D = 128
    Q, K, V = (si.normal((B, S, H, D), 0.0, 1.0, F16, 4, o) for o in (1, 2, 3))
    spl = lambda blk: [ES(B, B), ES(S, S // blk), ES(H, H // hb), [0, D]]
    rQ, rK, rV = upload(Q, spl(qb)), upload(K, spl(kb)), upload(V, spl(kb))
    rO = empty_like_tiling([B, S, H, D], spl(qb), F16, fill=float("nan"))
    rL = empty_like_tiling([B, S, H], spl(qb)[:3], F32, fill=float("nan"))
    parts = {"b": ES(B, B), "q": ES(S, S // qb), "h": ES(H, H // hb), "d": [0, D], "k": ES(S, S // kb)}
    spec = ja.Spec("bqhd,bkhd,bkhd->bqhd", parts, "attention", (1.0 / np.sqrt(D), 1.0 if causal else 0.0), "online_softmax")
    spec.execute([rQ, rK, rV], [rO, rL])
    got, lse = download(rO), download(rL)
    check_status()
    ref = operators.attention(si.to_f64(Q), si.to_f64(K), si.to_f64(V), causal, "f16")
    assert relfro(got, ref) <= TOL[F16]
    assert np.abs(got - ref).max() <= 0.01
    assert np.abs(lse - operators.attention_lse(si.to_f64(Q), si.to_f64(K), causal)).max() <= 2e-3


def test_attention_offset_raising_path_f16():
    """Keys that grow from one key tile to the next: the rescale of the accumulated output and the redo paths in f16."""
    B, S, H, D = 1, 1024, 2, 128
    Q, K, V = (si.normal((B, S, H, D), 0.0, 1.0, F16, 4, o) for o in (31, 32, 33))
    growth = 1.0 + 3.0 * (np.arange(S) // 128)
    K = torch.from_numpy((si.to_f64(K) * growth[None, :, None, None]).astype(np.float32)).to(F16)
    sp = [ES(B, B), ES(S, S // 128), ES(H, H), [0, D]]
    for form in ("tcgen05_two_tiles_persistent", "tcgen05_one_tile"):
        force_attention_form(form)
        rQ, rK, rV = upload(Q, sp), upload(K, sp), upload(V, sp)
        rO = empty_like_tiling([B, S, H, D], sp, F16, fill=float("nan"))
        parts = {"b": sp[0], "q": sp[1], "h": sp[2], "d": sp[3], "k": sp[1]}
        ja.Spec("bqhd,bkhd,bkhd->bqhd", parts, "attention", (1.0 / np.sqrt(D), 1.0), "online_softmax").execute([rQ, rK, rV], rO)
        got = download(rO)
        check_status()
        assert relfro(got, operators.attention(si.to_f64(Q), si.to_f64(K), si.to_f64(V), True, "f16")) <= TOL[F16]


@pytest.mark.parametrize("plan", ["seq", "head"])
def test_llama_block_f16(plan):
    from paper_2609_03905_b200.llama_block import LlamaBlock
    Bt, S, hidden, heads, ffn = 2, 256, 512, 4, 1408
    w = si.llama_weights(hidden, ffn, config=5, dtype=F16, first_ordinal=21)
    x = si.normal((Bt * S, hidden), 0.0, 1.0, F16, 5, 20)
    w64 = {k: si.to_f64(v) for k, v in w.items()}
    ref = np.concatenate([operators.llama_block(si.to_f64(x[b * S:(b + 1) * S]), w64, heads, dtype="f16")["out"] for b in range(Bt)])
    blk = LlamaBlock(Bt, S, hidden, heads, ffn, w, plan=plan, col_blocks=4, dtype=F16)
    ja.repartition(ja.from_dense(x.cuda(), [blk.t_sp, blk.io_c]), blk.x)
    got = download(blk.forward())
    check_status()
    assert relfro(got.reshape(Bt * S, hidden), ref) <= TOL[F16]


def test_optimizer_plan_on_small_block_f16():
    """The logical optimizer's p = 8 plan executed with every relation in f16: relayouts wherever the plan charges one."""
    from paper_2609_03905_b200.planned_block import PlannedBlock, block_graph, plan_repartition_charges
    Bt, S, hidden, heads, ffn = 2, 512, 512, 4, 1408
    ops = block_graph(Bt, S, hidden, heads, ffn)
    _, plan = ja.ja_plan_optimize_graph(ops, 8)
    w = si.llama_weights(hidden, ffn, config=5, dtype=F16, first_ordinal=21)
    x = si.normal((Bt * S, hidden), 0.0, 1.0, F16, 5, 20)
    blk = PlannedBlock(Bt, S, hidden, heads, ffn, w, plan, dtype=F16)
    assert blk.n_relayouts == plan_repartition_charges(ops, plan)[0] > 0
    blk.load_input(x.cuda())
    got = download(blk.forward()).reshape(Bt * S, hidden)
    check_status()
    w64 = {k: si.to_f64(v) for k, v in w.items()}
    ref = np.concatenate([operators.llama_block(si.to_f64(x[b * S:(b + 1) * S]), w64, heads, dtype="f16")["out"] for b in range(Bt)])
    assert relfro(got, ref) <= TOL[F16]
