// Attention join-agg "bqhd,bkhd,bkhd->bqhd" (f = ATTENTION, (+) = online softmax) on the 5th-generation
// tensor cores: both contractions of every joined tuple run as tcgen05.mma with accumulators in tensor memory.
//
// Two kernels. attention_tc2_kernel (further down) gives a CTA two output key tiles of one (batch, head) and is the one
// that runs whenever sequences are whole pairs of 128-row tiles; attention_tc_kernel, described here, takes the rest:
// one CTA owns one output key tile (128 query rows of one (batch, head)) and walks the function specs that
// share that output key -- the 128-row key/value tiles that survive the causal band predicate -- ascending.
//
//   warp 0      TMA producer: Q once, then K_j and V_j (two stages each), straight from the "bshd" block-key
//               layout through rank-3 tensor maps (d, head in block, row): with uniform blocks along b and h every
//               block is a run of rows of hblk x 128 cells, and the rows of consecutive blocks follow one another,
//               so one map serves any split of the sequence index (uniform or at packed-sequence ends).
//   warp 1      tcgen05.mma issuer (one lane):  S_j = Q K_j^T  (A, B from shared memory, both K-major)
//                                               O'_j = P_j V_j  (A = P_j from TENSOR MEMORY, B = V_j MN-major)
//   warps 2..5  one thread per query row: read S_j from TMEM, running max / sum in the base-2 domain, write
//               P_j (bf16) back into the SAME TMEM columns, then fold the finished partial O'_{j-1} into the
//               running triple held in registers:  O~ <- O~ * 2^(m_old - m_new) + O'_{j-1}.
//
// TMEM map (512 columns): S/P buffers at 0 and 128, partial-O buffers at 256 and 384. QK^T of step j+1 is issued
// before the softmax of step j finishes, so the tensor pipe works while the row threads exponentiate.
// Grouped-query attention: query head h joins key/value head h / group. Packed sequences (Example 3.10): an output
// key tile joins only the key/value tiles of its own sequence [s0, s1), so the walk starts at s0.
// Every mbarrier wait is bounded; on expiry the CTA records JA_ERR_TIMEOUT and leaves through the normal exit.
#include <stdlib.h>

#include <atomic>

#include <algorithm>
#include <utility>
#include <vector>

#include "ja_device.cuh"
#include "ja_ptx.cuh"

namespace {

using namespace ja_ptx;

constexpr int D = 128, QT = 128, KT = 128;
constexpr int TILE_BYTES = 128 * D * 2;      // 32 KiB: one 128 x 128 bf16 tile, stored as two 64-column halves
constexpr int HALF_BYTES = TILE_BYTES / 2;
constexpr int NUM_THREADS = 192;
constexpr int SMEM_BYTES = 5 * TILE_BYTES + 1024 + 256;   // Q, K x2, V x2

constexpr int MAX_SB = 64;   // sequence blocks of an irregular split held in the kernel parameters
constexpr int MAX_ORDER = 512;   // query tiles (pairs) whose launch order is held in the kernel parameters

// Tiling of one "bshd" relation: uniform blocks along b and h, any split of s, d unsplit.
struct SeqGeom {
    int32_t bblk, hblk, nhb;     // batch rows per block, heads per block, blocks along h
    int32_t sblk;                // uniform rows per s block, or 0: split[] holds the nsb + 1 split points
    int32_t nsb;
    int32_t split[MAX_SB + 1];
};

struct AttnTcParams {
    char* o_base;
    float* lse_base;             // optional second output (nullptr if absent), addressed like o without the last index
    int32_t* status;             // status word of the launching stream
    uint32_t wait_cap_us;        // limit of every bounded wait
    int32_t B, S, H;
    int32_t group;               // query heads per key/value head
    int32_t causal;
    int32_t n_ends;              // packed sequences; 0 = one sequence [0, S)
    float scale_log2e;
    int32_t ends[JA_MAX_SEQ];
    SeqGeom q, k;                // o is tiled like q, v like k
    int32_t sect;                // (batch, head) pairs per launch-order section (ja_attn_decode_cta)
    int32_t* queue;              // persistent form: {next item, CTAs finished} of this launch, both zero before and after it
    int32_t n_order;             // > 0: order[slot] = the query tile (pair) in heaviest-first slot `slot`
    uint16_t order[MAX_ORDER];
};

// Row coordinate of cell (b, s, h, :) in the rank-3 view (d, head in block, row). Block (bb, sb, hb) starts
// 128 * hblk * [ (bb*bblk*S + bblk*start(sb)) * nhb + hb*bblk*rows(sb) ] elements into the payload (blocks are stored
// in key order, each dense), and inside it the row is (b in block) * rows(sb) + (s - start(sb)).
__device__ __forceinline__ int seq_row(const SeqGeom& g, int S, int b, int s, int h) {
    int start, rows;
    if (g.sblk) {
        start = (s / g.sblk) * g.sblk;
        rows = g.sblk;
    } else {
        int sb = 0;
        while (sb + 1 < g.nsb && g.split[sb + 1] <= s) ++sb;
        start = g.split[sb];
        rows = g.split[sb + 1] - start;
    }
    const int bb = b / g.bblk, hb = h / g.hblk;
    return ((bb * g.bblk * S + g.bblk * start) * g.nhb + hb * g.bblk * rows) + (b - bb * g.bblk) * rows + (s - start);
}

// the packed sequence [s0, s1) that holds position q0
__device__ __forceinline__ void sequence_of(const AttnTcParams& p, int q0, int& s0, int& s1) {
    s0 = 0;
    s1 = p.S;
    for (int i = 0; i < p.n_ends; ++i) {
        if (p.ends[i] <= q0) s0 = p.ends[i];
        else { s1 = p.ends[i]; break; }
    }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// TMA store of one box from shared memory (bulk-group completion)
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* tm, uint32_t src, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(tm), "r"(src), "r"(c0), "r"(c1), "r"(c2)
                 : "memory");
}

// tcgen05.mma and tcgen05.commit as executed by a whole converged warp with one lane (pred != 0) issuing: every operand is then
// warp-uniform, which lets the compiler keep descriptors and addresses in uniform registers instead of moving them there before
// every instruction.
// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void umma_ss_w(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate, uint32_t pred) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(pred)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void umma_ts_w(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate, uint32_t pred) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(pred)
        : "memory");
}
__device__ __forceinline__ void commit1_w(uint32_t bar, uint32_t pred) {
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar), "r"(pred) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t* r) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <bool F16>   // cell type of Q, K, V, O and of P: bf16 or f16
__global__ void __launch_bounds__(NUM_THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ AttnTcParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t sQ = base, sK = base + TILE_BYTES, sV = base + 3 * TILE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 5 * TILE_BYTES);
    const uint32_t bar0 = smem_u32(bars);
    // barrier indices
    enum { Q_FULL = 0, K_FULL = 1, K_EMPTY = 3, V_FULL = 5, V_EMPTY = 7, S_FULL = 9, P_FULL = 11, O_FULL = 13, O_EMPTY = 15, NBAR = 17 };
    auto bar = [&](int i) { return bar0 + 8u * i; };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NBAR);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0), lane = threadIdx.x % 32;   // warp-uniform by construction
    const int n_qt = p.S / QT;
    int slot, bh;
    ja_attn_decode_cta((int)blockIdx.x, n_qt, p.H * p.B, p.sect, &slot, &bh);
    const int qt = p.n_order ? (int)p.order[slot] : n_qt - 1 - slot;   // output keys with the most surviving tuples first
    const int h = bh % p.H, b = bh / p.H;
    const int q0 = qt * QT;
    int s0, s1;
    sequence_of(p, q0, s0, s1);
    const int n_steps = p.causal ? (q0 + QT - s0) / KT : (s1 - s0) / KT;   // key tiles [s0 + j*KT, ...) joined with this tile

    if (threadIdx.x == 0) {
        for (int i = 0; i < NBAR; ++i) {
            const bool row_threads_arrive = (i >= P_FULL && i < P_FULL + 2) || (i >= O_EMPTY && i < O_EMPTY + 2);
            mbar_init(bar(i), row_threads_arrive ? 4 : 1);   // one arrival per row warp, else one commit / expect_tx
        }
        wait_ctl_init(abort_flag, p.wait_cap_us);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);
    const uint32_t tS[2] = {tmem_base, tmem_base + 128};
    const uint32_t tO[2] = {tmem_base + 256, tmem_base + 384};

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            const int hk = h / p.group;
            const int qrow = seq_row(p.q, p.S, b, q0, h);
            mbar_expect_tx(bar(Q_FULL), TILE_BYTES);
            for (int half = 0; half < 2; ++half)
                tma_load_3d(sQ + half * HALF_BYTES, &tmQ, bar(Q_FULL), half * 64, h % p.q.hblk, qrow);
            bool ok = true;
            for (int j = 0; j < n_steps && ok; ++j) {
                const int st = j & 1;
                const uint32_t ph = (uint32_t)(j >> 1) & 1;
                const int krow = seq_row(p.k, p.S, b, s0 + j * KT, hk);
                if (!mbar_wait(bar(K_EMPTY + st), ph ^ 1, abort_flag, p.status)) { ok = false; break; }
                mbar_expect_tx(bar(K_FULL + st), TILE_BYTES);
                for (int half = 0; half < 2; ++half)
                    tma_load_3d(sK + st * TILE_BYTES + half * HALF_BYTES, &tmK, bar(K_FULL + st), half * 64, hk % p.k.hblk, krow);
                if (!mbar_wait(bar(V_EMPTY + st), ph ^ 1, abort_flag, p.status)) { ok = false; break; }
                mbar_expect_tx(bar(V_FULL + st), TILE_BYTES);
                for (int half = 0; half < 2; ++half)
                    tma_load_3d(sV + st * TILE_BYTES + half * HALF_BYTES, &tmV, bar(V_FULL + st), half * 64, hk % p.k.hblk, krow);
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer: the whole warp runs the loop, one elected lane issues =================
        {
            const uint32_t leader = elect_one();
            // S = Q K^T: M=128, N=128, A and B K-major.  O' = P V: A from TMEM, B MN-major.
            constexpr uint32_t FMT = F16 ? 0u : 1u;   // operand format of the instruction descriptor: f16 = 0, bf16 = 1
            const uint32_t idesc_qk = (1u << 4) | (FMT << 7) | (FMT << 10) | ((uint32_t)(KT >> 3) << 17) | ((uint32_t)(QT >> 4) << 24);
            const uint32_t idesc_pv = idesc_qk | (1u << 16);
            auto issue_qk = [&](int j) {
                const int st = j & 1;
                const uint32_t kaddr = sK + st * TILE_BYTES;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {   // 16 d per instruction; d 0..63 in the first half, 64..127 in the second
                    const uint32_t off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;
                    umma_ss_w(tS[st], desc_sw128(sQ + off, 16), desc_sw128(kaddr + off, 16), idesc_qk, kk > 0, leader);
                }
                commit1_w(bar(S_FULL + st), leader);
                commit1_w(bar(K_EMPTY + st), leader);
            };
            bool ok = mbar_wait(bar(Q_FULL), 0, abort_flag, p.status);
            if (ok) ok = mbar_wait(bar(K_FULL + 0), 0, abort_flag, p.status);
            if (ok) {
                tc_fence_after();
                issue_qk(0);
            }
            for (int j = 0; j < n_steps && ok; ++j) {
                const int st = j & 1;
                const uint32_t ph = (uint32_t)(j >> 1) & 1;
                if (j + 1 < n_steps) {
                    if (!mbar_wait(bar(K_FULL + (st ^ 1)), (uint32_t)((j + 1) >> 1) & 1, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after();
                    issue_qk(j + 1);   // overwrites the S/P buffer of step j-1: ordered behind P V of step j-1 on the tensor pipe
                }
                if (!mbar_wait(bar(P_FULL + st), ph, abort_flag, p.status)) { ok = false; break; }
                if (!mbar_wait(bar(V_FULL + st), ph, abort_flag, p.status)) { ok = false; break; }
                if (!mbar_wait(bar(O_EMPTY + st), ph ^ 1, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t vaddr = sV + st * TILE_BYTES;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)     // 16 keys per instruction: 8 TMEM columns of packed bf16 P, 2048 bytes of V
                    umma_ts_w(tO[st], tS[st] + kk * 8, desc_sw128(vaddr + kk * 2048, HALF_BYTES), idesc_pv, kk > 0, leader);
                commit1_w(bar(O_FULL + st), leader);
                commit1_w(bar(V_EMPTY + st), leader);
            }
        }
    } else {
        // ================= row threads: softmax and the running (O~, m, l) =================
        const int q = warp & 3;
        const int r = q * 32 + lane;                 // query row inside the tile == TMEM lane
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        float o[D];
#pragma unroll
        for (int i = 0; i < D; ++i) o[i] = 0.f;
        float m_run = -INFINITY, l_run = 0.f, alpha_prev = 0.f;
        bool ok = true;

        auto fold = [&](int st, float alpha) {   // O~ <- O~ * alpha + O'
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t v[32];
                tmem_ld32(tO[st] + lane_addr + c * 32, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) o[c * 32 + i] = fmaf(o[c * 32 + i], alpha, __uint_as_float(v[i]));
            }
        };

        for (int j = 0; j < n_steps && ok; ++j) {
            const int st = j & 1;
            const uint32_t ph = (uint32_t)(j >> 1) & 1;
            if (!mbar_wait(bar(S_FULL + st), ph, abort_flag, p.status)) { ok = false; break; }
            tc_fence_after();
            const bool diag = p.causal && (j == n_steps - 1);
            const int kmax = q0 + r - (s0 + j * KT); // columns c > kmax of this tile lie after the query row
            // ---- pass 1: row maximum ----
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four independent chains, not one of 128 links
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t v[32];
                tmem_ld32(tS[st] + lane_addr + c * 32, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float s = __uint_as_float(v[i]);
                    if (diag && c * 32 + i > kmax) s = -INFINITY;
                    mx4[i & 3] = fmaxf(mx4[i & 3], s);
                }
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            const float m_new = fmaxf(m_run, mx * p.scale_log2e);
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;           // e^(-inf - -inf) := 0
            const float alpha = (m_run == -INFINITY) ? 0.f : ex2(m_run - m_use);
            // ---- pass 2: P = 2^(S*scale - m), row sum, P written over S as packed bf16 ----
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t v[32];
                tmem_ld32(tS[st] + lane_addr + c * 32, v);
                tmem_ld_wait();
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float p0 = ex2(fmaf(__uint_as_float(v[i]), p.scale_log2e, -m_use));
                    float p1 = ex2(fmaf(__uint_as_float(v[i + 1]), p.scale_log2e, -m_use));
                    if (diag && c * 32 + i > kmax) p0 = 0.f;
                    if (diag && c * 32 + i + 1 > kmax) p1 = 0.f;
                    sum += p0 + p1;
                    pk[i / 2] = ja_pack16<F16>(p0, p1);
                }
                tmem_st16(tS[st] + lane_addr + c * 16, pk);   // columns [16c, 16c+16): S columns already consumed
            }
            l_run = l_run * alpha + sum;
            m_run = m_new;
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(P_FULL + st));
            // ---- fold the partial of the previous step while the tensor pipe computes P V of this one ----
            if (j > 0) {
                const int ps = st ^ 1;
                if (!mbar_wait(bar(O_FULL + ps), (uint32_t)((j - 1) >> 1) & 1, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                fold(ps, alpha_prev);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(O_EMPTY + ps));
            }
            alpha_prev = alpha;
        }
        if (ok && n_steps > 0) {
            const int ls = (n_steps - 1) & 1;
            if (mbar_wait(bar(O_FULL + ls), (uint32_t)((n_steps - 1) >> 1) & 1, abort_flag, p.status)) {
                tc_fence_after();
                fold(ls, alpha_prev);
                // ---- O = O~ / l, one rounding, 256 contiguous bytes per row ----
                const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
                const int64_t cell = (int64_t)seq_row(p.q, p.S, b, q0 + r, h) * p.q.hblk + h % p.q.hblk;
                char* dst = p.o_base + cell * (D * 2);
                if (p.lse_base) p.lse_base[cell] = (m_run + log2f(l_run)) * 0.6931471805599453f;   // scores were kept in base 2
#pragma unroll
                for (int g = 0; g < 16; ++g) {
                    uint4 ov;
                    uint32_t* po = reinterpret_cast<uint32_t*>(&ov);
#pragma unroll
                    for (int e = 0; e < 4; ++e) po[e] = ja_pack16<F16>(o[g * 8 + 2 * e] * inv, o[g * 8 + 2 * e + 1] * inv);
                    *reinterpret_cast<uint4*>(dst + g * 16) = ov;
                }
            }
        }
    }
    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

// ---- row-thread arithmetic: 3-input max and packed f32x2 math keep the instruction count per score low ----
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// maximum of one row of scores (128 fp32 bit patterns): four chains of 3-input maxima
__device__ __forceinline__ float row_max128(const uint32_t (&v)[128]) {
    float m0 = __uint_as_float(v[0]), m1 = __uint_as_float(v[1]), m2 = __uint_as_float(v[2]), m3 = __uint_as_float(v[3]);
#pragma unroll
    for (int i = 4; i + 7 < 128; i += 8) {
        m0 = max3(m0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
        m1 = max3(m1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
        m2 = max3(m2, __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
        m3 = max3(m3, __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
    }
    m0 = max3(m0, __uint_as_float(v[124]), __uint_as_float(v[125]));
    m1 = max3(m1, __uint_as_float(v[126]), __uint_as_float(v[127]));
    return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}

// 2^x for a pair of exponents on the FMA pipe (no special-function unit): x = n + f with n = round(x), f in [-1/2, 1/2];
// 2^f by a cubic fitted to a relative error of 7.5e-5 (bf16 keeps 8 bits of P); n is added to the exponent field. x is
// clamped at -126 so that the exponent field cannot wrap; scores above the offset by more than 2^8 never reach here (lazy
// rescale keeps x <= 8).
__device__ __forceinline__ void exp2_poly_pair(uint64_t x2, float& p0, float& p1) {
    float x0, x1;
    unpack2(x2, x0, x1);
    x0 = fmaxf(x0, -126.f);
    x1 = fmaxf(x1, -126.f);
    const uint64_t x = pack2(x0, x1);
    const uint64_t magic = pack2(12582912.f, 12582912.f);        // 1.5 * 2^23: adding it rounds x to an integer in the low mantissa bits
    const uint64_t t = add2(x, magic);
    const uint64_t n = add2(t, pack2(-12582912.f, -12582912.f));
    const uint64_t f = fma2(n, pack2(-1.f, -1.f), x);
    uint64_t r = fma2(pack2(0.05517162f, 0.05517162f), f, pack2(0.24261113f, 0.24261113f));
    r = fma2(r, f, pack2(0.69326097f, 0.69326097f));
    r = fma2(r, f, pack2(0.99992806f, 0.99992806f));
    float r0, r1, t0, t1;
    unpack2(r, r0, r1);
    unpack2(t, t0, t1);
    p0 = __int_as_float(__float_as_int(r0) + (__float_as_int(t0) << 23));
    p1 = __int_as_float(__float_as_int(r1) + (__float_as_int(t1) << 23));
}

// One row of P = 2^(S * scale - m) for 128 keys as 64 packed bf16 (or f16) pairs in registers; returns the row sum (f32, of the
// unrounded values); a score of -inf (a masked key) gives exactly 0. POLY: which pairs of every group of eight keys take the
// FMA-pipe exponential instead of ex2 -- 0 none, 1 one of four, 2 two of four, 3 one of eight -- interleaved so that both
// pipes stay busy.
template <int POLY, bool F16>
__device__ __forceinline__ float row_exp_pack128(const uint32_t (&v)[128], float scale, float m_used, uint32_t (&pk)[64]) {
    const uint64_t sc2 = pack2(scale, scale), nm2 = pack2(-m_used, -m_used);
    uint64_t sum_a = pack2(0.f, 0.f), sum_b = pack2(0.f, 0.f);
#pragma unroll
    for (int cc = 0; cc < 16; ++cc) {
#pragma unroll
        for (int i = 0; i < 8; i += 2) {
            const int col = cc * 8 + i;
            const uint64_t x2 = fma2(pack2(__uint_as_float(v[col]), __uint_as_float(v[col + 1])), sc2, nm2);
            float p0, p1;
            const bool poly = (POLY == 1 && i == 6) || (POLY == 2 && (i == 2 || i == 6)) || (POLY == 3 && i == 6 && (cc & 1));
            if (poly) {
                exp2_poly_pair(x2, p0, p1);
            } else {
                unpack2(x2, p0, p1);
                p0 = ex2(p0);
                p1 = ex2(p1);
            }
            if (i & 2) sum_a = add2(sum_a, pack2(p0, p1));
            else sum_b = add2(sum_b, pack2(p0, p1));
            pk[col / 2] = ja_pack16<F16>(p0, p1);
        }
    }
    float a0, a1, b0, b1;
    unpack2(sum_a, a0, a1);
    unpack2(sum_b, b0, b1);
    return (a0 + a1) + (b0 + b1);
}

// ---------------------------------------------------------------------------------------------------------
// Two query tiles per CTA. The CTA owns 256 query rows of one (batch, head) as two independent 128-row output key tiles
// A and B that share every K_j / V_j tile it loads; while the row threads of one tile exponentiate, the tensor pipe works
// on the other tile, and each scheduler holds two row warps.
//   warp 0 TMA producer, warp 1 MMA issuer (runs converged, one elected lane issues; the steady state is straight-line
//   code: a branch or a move to uniform registers between two tcgen05.mma costs the issuing thread ~40 cycles against
//   64 cycles of tensor-pipe time for M128 N128 K16), warps 2..5 rows of A, warps 6..9 rows of B (one thread per row).
//   TMEM: S of A at 0, S of B at 128, O~ of A at 256, O~ of B at 384 (fp32, 128 columns each). O~ is ACCUMULATED IN TENSOR
//   MEMORY by the P V products. The running maximum used as the exponent offset is only raised when a row's new maximum
//   exceeds it by more than 2^8 (P stays <= 256, exact in the final O~/l); only then is the row's O~ rescaled in place.
//   P goes to the P V product through SHARED memory (a 128-byte-swizzled K-major tile, the layout TMA gives Q): the row
//   threads copy S into registers and release the S columns at once, so the next Q K^T of the tile runs WHILE they
//   exponentiate.
//   Shared memory: Q_A, Q_B, P_A, P_B and THREE K / V slots that K_0, K_1, V_0, K_2, V_1, ... pass through in the order
//   the products consume them (7 tiles = 224 KiB). O leaves through the tile's P buffer and two TMA stores.
// PERSIST: one CTA per SM takes work items (one item = the pair of tiles of one (batch, head)), heaviest first, from a
//   counter in global memory: the producer thread claims the next item and hands its number to the other roles through a
//   two-entry queue in shared memory, and runs ahead into the next item as soon as the Q buffers are free, so the next
//   item's Q and first K tile load, and its first Q K^T run, while the row threads finish this item. Barrier phases follow
//   running counters (items; key steps per tile). Otherwise one CTA per item, handed out by the hardware in grid order.
// VAR selects row-thread variants ("attn_variant"; all verified against the oracle): bits 0-1 = POLY of row_exp_pack128, bit 2 =
//   exponentiate into registers first and wait for the P tile only before storing. Default 1: a quarter of the exponentials
//   on the FMA pipe (B4 S2048 H32 causal, same run: POLY 0 0.1430 ms, one of eight 0.1405, one of four 0.1403, two of four
//   0.1509; exponentials first 0.1542).
// Timing-only ablations of this kernel before the masked loops were merged (B4 S2048 H32 causal, 0.163 ms on the box of
//   that run): no P stores -6 %, no exponentials -7 %, QK^T or P V reduced to one instruction of eight -6 % / 0 %, no K / V
//   loads -10 %, no output stage -3 %; all of them together still left 0.067 ms: the row threads' own instruction stream (two
//   row warps per scheduler, several hundred instructions per row and key tile, issued in order) and the hand-offs between
//   the roles bound the kernel, not one of the units. Also measured and not kept: on the diagonal tile, skipping the keys
//   that no row of a warp may see (half of that tile's exponentials on average): 2-3 % slower; TMA prefetches into L2
//   (the next item's Q and first K / V tiles, claimed one item early, and the tiles two key steps ahead): 20 % slower --
//   the prefetches queue in front of the loads the products wait for; claiming one item early alone: 2 % slower; issuing
//   the tensor-memory loads of the next key step's scores before handing P over (when they are already complete): 20 %
//   slower; a fourth group of four warps that takes O~ / l and the stores off the row warps (register allotments moved
//   between the groups with setmaxnreg, output written straight from registers): 6 % slower -- the output stage is not
//   what an item waits for. Not possible: P in f16 from ex2.approx.f16x2 (two exponentials per instruction) against bf16
//   V -- tcgen05.mma kind::f16 with different formats for A and B is an illegal instruction.
//   The output written from the row threads' registers straight to global memory (no staging in the P tile, no wait for
//   its TMA stores at the next item's first key step): 0.1495 ms against 0.1399.
//   With f16 relations, exponentials in half precision (ex2.approx.f16x2: two per instruction, the result already the
//   packed operand, the row sum from f16 partial sums): 0.1558 ms against 0.1405 -- half the special-function work
//   buys nothing, the conversions and the sum cost more.
//   TWO threads per query row (sixteen row warps, 64 keys each, the halves of a row agreeing on its maximum through shared
//   memory at every key step; registers moved to the row warps with setmaxnreg): 0.1618 ms against 0.1399, 2.12 against
//   1.79 ms on one sequence of 16384 rows. Halving the row threads' instruction chains does not shorten a key step:
//   what a step waits for are the hand-offs themselves (commit -> barrier -> wake, the tensor-memory loads, P ready ->
//   issue), and with S and O~ of two tiles the 512 columns of tensor memory are full -- a third tile to overlap them
//   with does not fit at d = 128.
//   Built, verified against the oracle and dropped for the same reason as the shared-memory analysis below suggested it:
//   FOUR tiles on a pair of CTAs, both products as tcgen05.mma.cta_group::2 with M = 256 and the K / V tile split between
//   the two SMs (each SM then reads and is filled with half of every K / V tile: a quarter less traffic on the
//   shared-memory port per product). B4 S2048 causal 0.230 ms against 0.140, one sequence of 16384 rows 2.79 against
//   1.80 ms: every key step then has two hand-offs that cross the cluster (the peer's P ready -> the leader's MMA warp;
//   the products' commit -> the peer's row warps), and their latency sits on the chain that already bounds the kernel.
//   Counters of the steady state: per 128 x 128 x 128 product pair the two smem x smem products read 128 KiB of shared
//   memory (1024 cycles of its 128 B/clk port, as long as the products themselves take), the P stores and the K / V fills
//   add half as much again: the shared-memory port, not a pipe, bounds long sequences (tensor-core reads 53 % + stores
//   19 % of its cycles over a whole launch of B4 S2048).
constexpr int NUM_THREADS2 = 320;
constexpr int SMEM_BYTES2 = 7 * TILE_BYTES + 1024 + 256;

// {next item, CTAs finished} pairs for launches of the persistent form: a launch takes the next pair of the ring, and its
// last CTA zeroes the pair again, so a pair is ready for reuse (also by a replay of a captured launch) as soon as its kernel
// has finished. 128 launches would have to be in flight at once (or 128 captured launches alive in graphs that replay
// concurrently) for two of them to share a pair.
constexpr int ATTN_QUEUES = 256;
__device__ int32_t g_attn_queues[2 * ATTN_QUEUES];

struct AttnItem {
    int q0, h, b, s0, n_a, n_b;
};
// item number `rank` in launch order (ja_attn_decode_cta: heaviest pairs first inside sections of (batch, head) pairs);
// false past the end
__device__ __forceinline__ bool attn_item(const AttnTcParams& p, int rank, AttnItem* it) {
    const int hb = p.H * p.B, n_pairs = p.S / (2 * QT);
    if (rank >= n_pairs * hb) return false;
    int slot, bh;
    ja_attn_decode_cta(rank, n_pairs, hb, p.sect, &slot, &bh);
    const int pr = p.n_order ? (int)p.order[slot] : n_pairs - 1 - slot;
    it->h = bh % p.H;
    it->b = bh / p.H;
    it->q0 = pr * 2 * QT;
    int s1;
    sequence_of(p, it->q0, it->s0, s1);
    it->n_a = p.causal ? (it->q0 + QT - it->s0) / KT : (s1 - it->s0) / KT;
    it->n_b = p.causal ? (it->q0 + 2 * QT - it->s0) / KT : (s1 - it->s0) / KT;
    return true;
}

template <bool PERSIST, int VAR, bool F16>
__global__ void __launch_bounds__(NUM_THREADS2, 1)
attention_tc2_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                     const __grid_constant__ AttnTcParams p) {
    constexpr int POLY = VAR & 3;
    constexpr bool WAIT_FIRST = (VAR & 4) == 0;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t sQ = base, sKV = base + 2 * TILE_BYTES, sP = base + 5 * TILE_BYTES;
    uint8_t* pP = smem + 5 * TILE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 7 * TILE_BYTES);
    const uint32_t bar0 = smem_u32(bars);
    enum { Q_FULL = 0, Q_EMPTY = 1, KV_FULL = 2, KV_EMPTY = 5, S_FULL = 8, S_FREE = 10, P_FULL = 12, P_EMPTY = 14, O_FULL = 16,
           O_STAGED = 18, O_READ = 20, P_STORED = 22, ITEM_FULL = 24, ITEM_EMPTY = 26, NBAR = 28 };
    auto bar = [&](int i) { return bar0 + 8u * i; };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NBAR);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);   // two words: abort flag, wait limit
    volatile int* item_rank = reinterpret_cast<volatile int*>(tmem_slot + 3);    // [2]: the item numbers in flight

    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0), lane = threadIdx.x % 32;
    // consumers of the item queue (MMA warp, row warps): wait for entry k, read it, release it
    auto next_item = [&](int k, AttnItem* it) -> bool {
        if (!PERSIST) return k == 0 && attn_item(p, (int)blockIdx.x, it);
        const int e = k & 1;
        if (!mbar_wait(bar(ITEM_FULL + e), (uint32_t)(k >> 1) & 1, abort_flag, p.status)) return false;
        const int rank = item_rank[e];
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(ITEM_EMPTY + e));
        return attn_item(p, rank, it);
    };

    if (threadIdx.x == 0) {
        for (int i = 0; i < NBAR; ++i) {
            const bool row_warps_arrive = (i >= S_FREE && i < S_FREE + 2) || (i >= P_FULL && i < P_FULL + 2) ||
                                          (i >= O_STAGED && i < O_STAGED + 2) || (i >= O_READ && i < O_READ + 2);
            mbar_init(bar(i), row_warps_arrive ? 4 : (i >= ITEM_EMPTY && i < ITEM_EMPTY + 2) ? 9 : 1);
        }
        wait_ctl_init(abort_flag, p.wait_cap_us);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            int li = 0;                       // K / V tiles loaded so far: ring slot li % 3, phase (li / 3) & 1
            bool ok = true;
            AttnItem it;
            for (int item = 0; ok; ++item) {
                int rank;
                if (PERSIST) {
                    // claim the next item and publish its number (entry item & 1 of the queue, free once all nine consumer
                    // warps have read what it held two items ago)
                    const int e = item & 1;
                    if (item >= 2 && !mbar_wait(bar(ITEM_EMPTY + e), (uint32_t)((item >> 1) - 1) & 1, abort_flag, p.status)) break;
                    rank = atomicAdd(p.queue, 1);
                    item_rank[e] = rank;
                    mbar_arrive(bar(ITEM_FULL + e));
                } else {
                    if (item > 0) break;
                    rank = (int)blockIdx.x;
                }
                if (!attn_item(p, rank, &it)) break;
                const int hk = it.h / p.group;
                // the Q buffers are free once the previous item's last Q K^T has read them
                if (item > 0 && !mbar_wait(bar(Q_EMPTY), (uint32_t)(item - 1) & 1, abort_flag, p.status)) break;
                mbar_expect_tx(bar(Q_FULL), 2 * TILE_BYTES);
                for (int t = 0; t < 2; ++t) {
                    const int qrow_t = seq_row(p.q, p.S, it.b, it.q0 + t * QT, it.h);
                    for (int half = 0; half < 2; ++half)
                        tma_load_3d(sQ + t * TILE_BYTES + half * HALF_BYTES, &tmQ, bar(Q_FULL), half * 64, it.h % p.q.hblk, qrow_t);
                }
                // K / V tiles in the order the products consume them: K_0, then for every step j: K_{j+1} (if any), V_j
                auto load = [&](const CUtensorMap* tm, int j) {
                    const int sl = li % 3;
                    const uint32_t ph = (uint32_t)(li / 3) & 1;
                    if (!mbar_wait(bar(KV_EMPTY + sl), ph ^ 1, abort_flag, p.status)) { ok = false; return; }
                    const int krow = seq_row(p.k, p.S, it.b, it.s0 + j * KT, hk);
                    mbar_expect_tx(bar(KV_FULL + sl), TILE_BYTES);
                    for (int half = 0; half < 2; ++half)
                        tma_load_3d(sKV + sl * TILE_BYTES + half * HALF_BYTES, tm, bar(KV_FULL + sl), half * 64, hk % p.k.hblk, krow);
                    ++li;
                };
                load(&tmK, 0);
                for (int j = 0; j < it.n_b && ok; ++j) {
                    if (j + 1 < it.n_b) load(&tmK, j + 1);
                    if (ok) load(&tmV, j);
                }
            }
            if (PERSIST) {   // the last CTA to get here leaves the counter pair as it found it
                __threadfence();
                if (atomicAdd(p.queue + 1, 1) == (int)gridDim.x - 1) {
                    p.queue[0] = 0;
                    p.queue[1] = 0;
                    __threadfence();
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer: the whole warp runs the loop, one elected lane issues =================
        const uint32_t leader = elect_one();
        constexpr uint32_t FMT = F16 ? 0u : 1u;   // operand format of the instruction descriptor: f16 = 0, bf16 = 1
        const uint32_t idesc_qk = (1u << 4) | (FMT << 7) | (FMT << 10) | ((uint32_t)(KT >> 3) << 17) | ((uint32_t)(QT >> 4) << 24);
        const uint32_t idesc_pv = idesc_qk | (1u << 16);
        auto issue_qk = [&](int t, int sl) {          // S_t = Q_t K^T, K in slot sl
            const uint32_t kaddr = sKV + sl * TILE_BYTES, qaddr = sQ + t * TILE_BYTES;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {          // 16 d per instruction; d 0..63 in the first half, 64..127 in the second
                const uint32_t off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;
                umma_ss_w(tmem_base + t * 128, desc_sw128(qaddr + off, 16), desc_sw128(kaddr + off, 16), idesc_qk, kk > 0, leader);
            }
            commit1_w(bar(S_FULL + t), leader);
        };
        auto issue_pv = [&](int t, int sl, bool first) {   // O~_t (+)= P_t V, P in shared memory (K-major), V in slot sl (MN-major)
            const uint32_t vaddr = sKV + sl * TILE_BYTES, paddr = sP + t * TILE_BYTES;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;
                umma_ss_w(tmem_base + 256 + t * 128, desc_sw128(paddr + off, 16), desc_sw128(vaddr + kk * 2048, HALF_BYTES), idesc_pv,
                          (!first || kk > 0) ? 1u : 0u, leader);
            }
            commit1_w(bar(P_EMPTY + t), leader);
            commit1_w(bar(O_FULL + t), leader);
        };
        int li = 0;
        int cs[2] = {0, 0};                   // key steps of each tile in all items so far
        bool ok = true;
        AttnItem it;
        for (int item = 0; ok && next_item(item, &it); ++item) {
            const int n_of[2] = {it.n_a, it.n_b};
            ok = mbar_wait(bar(Q_FULL), (uint32_t)item & 1, abort_flag, p.status);
            {
                const int sl = li % 3;
                if (ok) ok = mbar_wait(bar(KV_FULL + sl), (uint32_t)(li / 3) & 1, abort_flag, p.status);
                for (int t = 0; t < 2 && ok; ++t) {
                    // S_t is free once the row threads hold the scores of the tile's previous key step (of the previous item)
                    if (cs[t] > 0 && !mbar_wait(bar(S_FREE + t), (uint32_t)(cs[t] - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after();
                    issue_qk(t, sl);
                }
                if (!ok) break;
                commit1_w(bar(KV_EMPTY + sl), leader);
                if (it.n_b == 1) commit1_w(bar(Q_EMPTY), leader);
                ++li;
            }
            for (int j = 0; j < it.n_b && ok; ++j) {
                if (j + 1 < it.n_b) {
                    const int sl = li % 3;
                    if (!mbar_wait(bar(KV_FULL + sl), (uint32_t)(li / 3) & 1, abort_flag, p.status)) { ok = false; break; }
                    for (int t = 0; t < 2 && ok; ++t) {
                        if (j + 1 < n_of[t]) {
                            // the row threads have copied S_t of step j into registers: its columns may be overwritten
                            if (!mbar_wait(bar(S_FREE + t), (uint32_t)(cs[t] + j) & 1, abort_flag, p.status)) { ok = false; break; }
                            tc_fence_after();
                            issue_qk(t, sl);
                        }
                    }
                    if (!ok) break;
                    commit1_w(bar(KV_EMPTY + sl), leader);
                    if (j + 2 == it.n_b) commit1_w(bar(Q_EMPTY), leader);   // that was the item's last Q K^T
                    ++li;
                }
                const int sl = li % 3;
                if (!mbar_wait(bar(KV_FULL + sl), (uint32_t)(li / 3) & 1, abort_flag, p.status)) { ok = false; break; }
                for (int t = 0; t < 2 && ok; ++t) {
                    if (j < n_of[t]) {
                        if (!mbar_wait(bar(P_FULL + t), (uint32_t)(cs[t] + j) & 1, abort_flag, p.status)) { ok = false; break; }
                        // the first P V of an item overwrites O~: the row threads must have read the previous item's
                        if (j == 0 && item > 0 && !mbar_wait(bar(O_READ + t), (uint32_t)(item - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                        tc_fence_after();
                        issue_pv(t, sl, j == 0);
                    }
                }
                if (!ok) break;
                commit1_w(bar(KV_EMPTY + sl), leader);
                ++li;
            }
            cs[0] += it.n_a;
            cs[1] += it.n_b;
        }
    } else {
        // ================= row threads =================
        const int t = (warp - 2) >> 2;                     // tile: 0 = A, 1 = B
        const int q = warp & 3;                            // TMEM lane group of this warp
        const int r = q * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        const uint32_t tS = tmem_base + t * 128 + lane_addr, tO = tmem_base + 256 + t * 128 + lane_addr;
        uint8_t* prow = pP + t * TILE_BYTES + r * 128;     // this row inside each 64-key half of the P tile
        const int sw = r & 7;                              // 128-byte swizzle: 16-byte chunk c of row r lives at chunk c ^ (r & 7)
        int cs = 0;                                        // key steps of this tile in all items so far
        bool ok = true;
        AttnItem it;
        for (int item = 0; ok && next_item(item, &it); ++item) {
            const int n_t = t == 0 ? it.n_a : it.n_b;
            const int qrow = it.q0 + t * QT + r;
            float m_used = -INFINITY, l_run = 0.f;
            for (int j = 0; j < n_t && ok; ++j) {
                const int c = cs + j;
                if (!mbar_wait(bar(S_FULL + t), (uint32_t)c & 1, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                const bool diag = p.causal && (j == n_t - 1);
                const int kmax = qrow - (it.s0 + j * KT);
                uint32_t v[128];
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) tmem_ld32(tS + cc * 32, v + cc * 32);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(S_FREE + t));   // S_t is in registers: the next Q K^T of this tile may run
                if (diag) {   // Keys after the query row score -inf: they lose every maximum and exponentiate to exactly 0, so ONE copy of
                              // the maximum / exponential code serves masked and unmasked tiles. (A masked variant of both loops --
                              // a select per score inside them, the maximum as one chain of 128 dependent selects -- cost 12 % of
                              // the kernel on B4 S2048: the chain sits on every item's critical path, and the second copy of the
                              // unrolled loops on the instruction cache.)
#pragma unroll
                    for (int i = 0; i < 128; ++i)
                        if (i > kmax) v[i] = 0xff800000u;
                }
                const float mx = row_max128(v);
                const float m_new = mx * p.scale_log2e;        // finite: the first key of a sequence is never masked
                // lazy rescale: raise the offset only when the row maximum outgrew it by more than 2^8
                float alpha = 1.f;
                bool need = false;
                if (j == 0) m_used = m_new;
                else if (m_new > m_used + 8.f) { alpha = ex2(m_used - m_new); m_used = m_new; need = true; }
                const bool rescale = __any_sync(0xffffffffu, need);
                // Two things have to hold before P of this step may be stored: the P V of the tile's previous key step has
                // read the P tile (P_EMPTY; O~ then also holds every product so far), and at the first step of an item the
                // TMA stores of the previous item's output, which was staged in the P tile, have read it (P_STORED).
                auto wait_p_tile = [&]() -> bool {
                    if (c > 0 && !mbar_wait(bar(P_EMPTY + t), (uint32_t)(c - 1) & 1, abort_flag, p.status)) return false;
                    if (j == 0 && item > 0 && !mbar_wait(bar(P_STORED + t), (uint32_t)(item - 1) & 1, abort_flag, p.status)) return false;
                    return true;
                };
                if (WAIT_FIRST || rescale) {
                    if (!wait_p_tile()) { ok = false; break; }
                }
                if (rescale) {
                    tc_fence_after();
#pragma unroll 1
                    for (int cc = 0; cc < 16; ++cc) {   // rare path: small chunks keep the register footprint of the hot path low
                        uint32_t o[8];
                        tmem_ld8(tO + cc * 8, o);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 8; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st8(tO + cc * 8, o);
                    }
                    tmem_st_wait();
                    tc_fence_before();
                    l_run *= alpha;
                }
                uint32_t pk[64];
                l_run += row_exp_pack128<POLY, F16>(v, p.scale_log2e, m_used, pk);
                if (!(WAIT_FIRST || rescale)) {
                    if (!wait_p_tile()) { ok = false; break; }
                }
#pragma unroll
                for (int cc = 0; cc < 16; ++cc)          // 16 chunks of 8 keys = 16 bytes of bf16
                    *reinterpret_cast<uint4*>(prow + (cc >> 3) * HALF_BYTES + (((cc & 7) ^ sw) << 4)) =
                        make_uint4(pk[cc * 4], pk[cc * 4 + 1], pk[cc * 4 + 2], pk[cc * 4 + 3]);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads P through the async proxy
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(P_FULL + t));
            }
            if (!ok) break;
            // ---- the item's output: O = O~ / l through the tile's P buffer (its last P V has read it once O_FULL fires) and two
            // TMA stores -- 16-byte stores from 32 lanes to 32 different rows would write half-filled sectors
            if (!mbar_wait(bar(O_FULL + t), (uint32_t)(cs + n_t - 1) & 1, abort_flag, p.status)) { ok = false; break; }
            tc_fence_after();
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            if (p.lse_base) {
                const int64_t cell = (int64_t)seq_row(p.q, p.S, it.b, qrow, it.h) * p.q.hblk + it.h % p.q.hblk;
                p.lse_base[cell] = (m_used + log2f(l_run)) * 0.6931471805599453f;   // l is relative to the offset m_used
            }
#pragma unroll 1
            for (int cc = 0; cc < 4; ++cc) {   // not unrolled: the output stage runs once per item, and code size costs instruction fetches
                uint32_t o[32];
                tmem_ld32(tO + cc * 32, o);
                tmem_ld_wait();
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    uint4 ov;
                    uint32_t* po = reinterpret_cast<uint32_t*>(&ov);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        po[e] = ja_pack16<F16>(__uint_as_float(o[g * 8 + 2 * e]) * inv, __uint_as_float(o[g * 8 + 2 * e + 1]) * inv);
                    const int ch = cc * 4 + g;                      // 16-byte chunk 0..15 of the row
                    *reinterpret_cast<uint4*>(prow + (ch >> 3) * HALF_BYTES + (((ch & 7) ^ sw) << 4)) = ov;
                }
            }
            tc_fence_before();
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar(O_READ + t));        // O~ of this tile may be overwritten by the next item's first P V
                mbar_arrive(bar(O_STAGED + t));
            }
            if (q == 0 && lane == 0) {
                if (!mbar_wait(bar(O_STAGED + t), (uint32_t)item & 1, abort_flag, p.status)) { ok = false; }
                else {
                    const int orow = seq_row(p.q, p.S, it.b, it.q0 + t * QT, it.h);
                    for (int half = 0; half < 2; ++half)
                        tma_store_3d(&tmO, sP + t * TILE_BYTES + half * HALF_BYTES, half * 64, it.h % p.q.hblk, orow);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // shared memory may be reused after this
                    mbar_arrive(bar(P_STORED + t));  // the P tile may be written again
                }
            }
            ok = __all_sync(0xffffffffu, ok);
            cs += n_t;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

// "bshd" relation with uniform blocks along b and h as a rank-3 tensor (d, head in block, row of hblk x 128 cells)
ja_status_t encode_rows(const RelView& v, bool f16, CUtensorMap* tm) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return ja_fail(JA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const int64_t hb = v.bs[2];
    const int64_t rows = v.extent[0] * v.extent[1] * v.nblk[2];
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)hb, (cuuint64_t)rows};
    cuuint64_t strides[2] = {(cuuint64_t)(D * 2), (cuuint64_t)(hb * D * 2)};
    cuuint32_t box[3] = {64, 1, 128};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult res = enc(tm, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, v.base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                       CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (res != CUDA_SUCCESS) return ja_fail(JA_ERR_CUDA, "cuTensorMapEncodeTiled (bshd rows) failed with code %d", (int)res);
    return JA_OK;
}

bool fill_geom(const RelView& v, const int32_t* host_split, SeqGeom* g) {
    if (!v.bs[0] || !v.bs[2] || v.nblk[3] != 1) return false;
    g->bblk = (int32_t)v.bs[0];
    g->hblk = (int32_t)v.bs[2];
    g->nhb = v.nblk[2];
    g->sblk = (int32_t)v.bs[1];
    g->nsb = v.nblk[1];
    if (!g->sblk) {
        if (g->nsb > MAX_SB || !host_split) return false;
        for (int i = 0; i <= g->nsb; ++i) g->split[i] = host_split[i];
    }
    return true;
}

}  // namespace


// After a device-side failure (a bounded wait that expired) a persistent launch may have left its work counter non-zero:
// put every counter pair of the current device back to zero. Called by ja_stream_status when it reports such a failure;
// the stream is idle then.
void ja_attention_reset_queues() {
    void* q = nullptr;
    if (cudaGetSymbolAddress(&q, g_attn_queues) == cudaSuccess && q) cudaMemset(q, 0, sizeof(int32_t) * 2 * ATTN_QUEUES);
}

namespace {

template <bool PERSIST>
ja_status_t launch_two_tiles(int variant, bool f16, dim3 grid, cudaStream_t st, const CUtensorMap& tq, const CUtensorMap& tk,
                             const CUtensorMap& tv, const CUtensorMap& to, const AttnTcParams& p) {
    if (f16) {   // f16 cells: the default row-thread variant only
        JA_CUDA(cudaFuncSetAttribute(attention_tc2_kernel<PERSIST, 1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES2));
        attention_tc2_kernel<PERSIST, 1, true><<<grid, NUM_THREADS2, SMEM_BYTES2, st>>>(tq, tk, tv, to, p);
        return JA_OK;
    }
#define JA_ATTN_LAUNCH(V)                                                                                                          \
    case V: {                                                                                                                      \
        JA_CUDA(cudaFuncSetAttribute(attention_tc2_kernel<PERSIST, V, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES2)); \
        attention_tc2_kernel<PERSIST, V, false><<<grid, NUM_THREADS2, SMEM_BYTES2, st>>>(tq, tk, tv, to, p);                      \
        return JA_OK;                                                                                                              \
    }
    switch (variant) {
        JA_ATTN_LAUNCH(0)
        JA_ATTN_LAUNCH(1)
        JA_ATTN_LAUNCH(3)
        JA_ATTN_LAUNCH(4)
        default: return ja_fail(JA_ERR_INVALID_ARG, "unknown attention variant %d", variant);
    }
#undef JA_ATTN_LAUNCH
}

}  // namespace

// Returns JA_OK and sets *launched when a tensor-memory kernel took the job; leaves *launched false when the tiling does
// not fit (every q / k split point and sequence end must be a multiple of 128 rows, blocks uniform along b and h, at most
// MAX_SB sequence blocks when they are irregular). The four tensor maps are encoded once per (spec, relations) tuple and
// kept in a.cache.
ja_status_t ja_launch_attention_tc(const AttnArgs& a, cudaStream_t st, bool* launched) {
    *launched = false;
    if (a.align % 128 || !a.rows_layout) return JA_OK;
    AttnTcParams p;
    memset(&p, 0, sizeof p);
    if (!fill_geom(a.q, a.q_split, &p.q) || !fill_geom(a.k, a.k_split, &p.k)) return JA_OK;
    static_assert(sizeof(CUtensorMap) == 128, "AttnTcCache holds four 128-byte tensor maps");
    AttnTcCache local;
    AttnTcCache* cache = a.cache ? a.cache : &local;
    CUtensorMap* maps = reinterpret_cast<CUtensorMap*>(cache->maps);
    if (!cache->valid) {
        ja_status_t s;
        if ((s = encode_rows(a.q, a.f16, &maps[0])) != JA_OK) return s;
        if ((s = encode_rows(a.k, a.f16, &maps[1])) != JA_OK) return s;
        if ((s = encode_rows(a.v, a.f16, &maps[2])) != JA_OK) return s;
        if ((s = encode_rows(a.o, a.f16, &maps[3])) != JA_OK) return s;
        cache->valid = true;
    }
    const CUtensorMap &tq = maps[0], &tk = maps[1], &tv = maps[2], &to = maps[3];
    const JaConfig& cfg = ja_config();
    p.o_base = a.o.base;
    p.lse_base = reinterpret_cast<float*>(a.lse.base);
    p.status = ja_device_status_word(st);
    if (!p.status) return ja_fail(JA_ERR_CUDA, "cannot resolve the device status word");
    p.wait_cap_us = (uint32_t)cfg.wait_cap_us;
    p.B = a.B; p.S = a.S; p.H = a.H;
    p.group = a.group;
    p.causal = a.causal;
    p.n_ends = a.n_ends;
    bool pair_ok = a.S % (2 * QT) == 0;
    for (int i = 0; i < a.n_ends; ++i) {
        p.ends[i] = a.ends[i];
        if (a.ends[i] % (2 * QT)) pair_ok = false;
    }
    p.scale_log2e = a.scale * 1.4426950408889634f;
    const bool two_tiles = pair_ok && cfg.attn_one_tile != 1;
    // packed sequences: the work of a tile is its distance from the start of its own sequence, not its index
    const int rows_per_cta = two_tiles ? 2 * QT : QT, n_cta_tiles = a.S / rows_per_cta;
    if (a.n_ends > 1 && n_cta_tiles <= MAX_ORDER) {
        std::vector<std::pair<int, int>> w(n_cta_tiles);   // (-steps, tile)
        for (int t = 0; t < n_cta_tiles; ++t) {
            const int q0 = t * rows_per_cta;
            int s0 = 0, s1 = a.S;
            for (int i = 0; i < a.n_ends; ++i) {
                if (a.ends[i] <= q0) s0 = a.ends[i];
                else { s1 = a.ends[i]; break; }
            }
            w[t] = {-(a.causal ? q0 + rows_per_cta - s0 : s1 - s0), t};
        }
        std::sort(w.begin(), w.end());
        p.n_order = n_cta_tiles;
        for (int t = 0; t < n_cta_tiles; ++t) p.order[t] = (uint16_t)w[t].second;
    }
    const int sms = ja_sm_count();
    // tiles of different weight (causal band, packed sequences): one section, i.e. heaviest first across all (batch, head)
    // pairs; equal tiles: sections that fill the GPU once, so that CTAs running together share K / V tiles through L2
    p.sect = (a.causal || a.n_ends > 1) ? a.H * a.B : std::max(1, (sms + n_cta_tiles - 1) / n_cta_tiles);
    if (cfg.attn_section >= 1) p.sect = cfg.attn_section;
    p.sect = std::min(p.sect, a.H * a.B);
    if (two_tiles) {
        const int64_t items = (int64_t)a.H * a.B * (a.S / (2 * QT));
        // persistent over work items where items are short (no sequence longer than 4096 rows); beyond that the hardware's
        // hand-out of one CTA per item balances as well and the queue buys nothing
        int longest = a.S;
        if (a.n_ends > 0) {
            longest = a.ends[0];
            for (int i = 1; i < a.n_ends; ++i) longest = std::max(longest, a.ends[i] - a.ends[i - 1]);
        }
        const bool persist = cfg.attn_persistent >= 0 ? cfg.attn_persistent == 1 : longest <= 4096;
        const int variant = cfg.attn_variant >= 0 ? cfg.attn_variant : 1;
        ja_status_t s;
        if (persist) {
            int32_t* queues = nullptr;
            if (cudaGetSymbolAddress((void**)&queues, g_attn_queues) != cudaSuccess || !queues)
                return ja_fail(JA_ERR_CUDA, "cannot resolve the attention work queues");
            // launches recorded into a CUDA graph keep their pair for as long as the graph lives: they draw from the upper half
            // of the ring, launches that run at once from the lower half, so a replay never shares a pair with an eager launch
            static std::atomic<unsigned> next_queue{0}, next_captured{0};
            cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
            if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) cap = cudaStreamCaptureStatusNone;
            const unsigned half = ATTN_QUEUES / 2;
            const unsigned slot = cap == cudaStreamCaptureStatusActive ? half + next_captured.fetch_add(1) % half : next_queue.fetch_add(1) % half;
            p.queue = queues + 2 * slot;
            s = launch_two_tiles<true>(variant, a.f16, dim3((unsigned)std::min<int64_t>(items, sms), 1, 1), st, tq, tk, tv, to, p);
        } else {
            s = launch_two_tiles<false>(variant, a.f16, dim3((unsigned)items, 1, 1), st, tq, tk, tv, to, p);
        }
        if (s != JA_OK) return s;
    } else {
        dim3 grid((unsigned)((int64_t)a.H * a.B * (a.S / QT)), 1, 1);
        if (a.f16) {
            JA_CUDA(cudaFuncSetAttribute(attention_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
            attention_tc_kernel<true><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(tq, tk, tv, p);
        } else {
            JA_CUDA(cudaFuncSetAttribute(attention_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
            attention_tc_kernel<false><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(tq, tk, tv, p);
        }
    }
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    *launched = true;
    return JA_OK;
}
