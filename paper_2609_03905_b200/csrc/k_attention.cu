// Dot-product attention as a join-agg: "bqhd,bkhd,bkhd->bqhd", f = ATTENTION, (+) = online softmax.
//
// One CTA owns one output key tile: QT query rows of one (batch, head). It walks the function specs that
// share that output key -- the key/value blocks kb that survive the causal band predicate -- in ascending
// order. For each joined tuple (Q block, K block, V block) the concrete operator computes the partial
// triple (O~, m, l) of the block pair; the running triple kept in registers is combined with it by
//     m* = max(m, m'),  O~ <- O~ e^(m-m*) + O~' e^(m'-m*),  l <- l e^(m-m*) + l' e^(m'-m*)
// which is the aggregation operator of the spec. O = O~/l is written once, to the key's offset in the
// output relation. Scores and probabilities never reach HBM.
//
// Grouped-query attention: query head h joins key/value head h / group. Packed sequences: an output key tile
// joins only key/value tiles of its own sequence [s0, s1) (Example 3.10).
//
// This file holds the mma.sync form (m16n8k16, bf16 in, fp32 accumulate; operands staged in shared memory with
// cp.async under an XOR swizzle and read with ldmatrix). It serves tilings the tensor-memory kernel cannot
// take (64-row blocks); everything else is dispatched to the tcgen05 kernel.
// RAGGED form of the same kernel: ANY split points of the sequence index, any sequence length and any sequence ends. Output
// key tiles are then 64 consecutive positions wherever they fall: a tile may straddle blocks and packed sequences and run
// past the end of the index, so every row is located on its own (block lookup per row), rows past the end are zero, and
// the selection predicate of the spec -- same sequence, and not after the query when causal -- is applied per score.
#include <stdlib.h>

#include <algorithm>

#include "ja_device.cuh"

namespace {

constexpr int D = 128;     // head dimension (extent of the unsplit last index)
constexpr int KT = 64;     // key rows per inner step
constexpr int ROW_BYTES = D * 2;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// F16: operands are f16 instead of bf16 (same fragments, f32 accumulate)
template <bool F16>
__device__ __forceinline__ void mma_16bit(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    if (F16)
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    else
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// byte address inside a [rows][128] bf16 tile whose 16-byte chunks are XOR-swizzled by the row
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * ROW_BYTES + ((chunk ^ (row & 7)) << 4)); }

// pointer to cell (b, s, h, 0) of a "bshd" relation, and the byte pitch between consecutive s inside the block
__device__ __forceinline__ const char* row_ptr(const RelView& v, int b, int s, int h, int64_t* pitch) {
    const int bb = ja_find_blk(v, 0, b), sb = ja_find_blk(v, 1, s), hb = ja_find_blk(v, 2, h);
    const int64_t blo = v.splits[0][bb], slo = v.splits[1][sb], hlo = v.splits[2][hb];
    const int64_t sw = v.splits[1][sb + 1] - slo, hw = v.splits[2][hb + 1] - hlo;
    const int64_t flat = ((int64_t)bb * v.nblk[1] + sb) * v.nblk[2] + hb;
    *pitch = hw * D * 2;
    return v.base + v.blk_off[flat] + ((((int64_t)(b - blo) * sw + (s - slo)) * hw + (h - hlo)) * D) * 2;
}

// the packed sequence [s0, s1) that holds position pos (the whole index when sequences are not packed)
__device__ __forceinline__ void seq_bounds(const AttnArgs& a, int pos, int& s0, int& s1) {
    s0 = 0;
    s1 = a.S;
    for (int i = 0; i < a.n_ends; ++i) {
        if (a.ends[i] <= pos) s0 = a.ends[i];
        else { s1 = a.ends[i]; break; }
    }
}

template <int QT, bool F16, bool RAGGED>
__global__ void __launch_bounds__(QT * 2, 1) attention_kernel(AttnArgs a) {
    constexpr int NW = QT / 16;        // warps; each owns 16 query rows
    constexpr int NT = NW * 32;
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* sQ = smem;                          // QT x 128 (reused to stage O)
    uint8_t* sK = smem + QT * ROW_BYTES;         // 2 x KT x 128
    uint8_t* sV = sK + 2 * KT * ROW_BYTES;       // 2 x KT x 128
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int g = lane / 4, t4 = lane % 4;

    const int n_qt = (a.S + QT - 1) / QT;
    int slot, bh;
    ja_attn_decode_cta((int)blockIdx.x, n_qt, a.H * a.B, a.sect, &slot, &bh);
    const int qt = n_qt - 1 - slot;              // heaviest output keys (most surviving tuples) first
    const int h = bh % a.H, b = bh / a.H;
    const int q0 = qt * QT;
    const int hk = h / a.group;                  // key/value head joined with this query head
    int s0, s1;                                  // the packed sequence the tile's first row lies in (RAGGED: later rows may lie in later ones)
    seq_bounds(a, q0, s0, s1);
    const int q_last = min(q0 + QT, a.S) - 1;    // last position of the tile that exists
    if (RAGGED) {
        int unused;
        seq_bounds(a, q_last, unused, s1);       // the key walk ends where the last row's sequence ends
    }

    // ---- stage Q, read its A fragments ---------------------------------------------------------------------
    {
        int64_t pitch;
        const char* qp = RAGGED ? nullptr : row_ptr(a.q, b, q0, h, &pitch);  // a q tile never leaves its block (QT divides qblk)
        for (int i = tid; i < QT * 16; i += NT) {
            int r = i / 16, c = i % 16;
            if (!RAGGED) cp_async16(smem_u32(sQ) + swz(r, c), qp + (int64_t)r * pitch + c * 16);
            else if (q0 + r < a.S) cp_async16(smem_u32(sQ) + swz(r, c), row_ptr(a.q, b, q0 + r, h, &pitch) + c * 16);
            else *reinterpret_cast<uint4*>(sQ + swz(r, c)) = make_uint4(0u, 0u, 0u, 0u);
        }
        cp_async_commit();
    }
    // number of 64-row key steps this output key joins with: keys [s0, q0 + QT) when causal, else [s0, s1)
    const int k_end = a.causal ? min(s1, (RAGGED ? q_last + 1 : q0 + QT)) : s1;
    const int n_steps = (k_end - s0 + KT - 1) / KT;

    auto load_kv = [&](int step, int buf) {
        const int k0 = s0 + step * KT;  // a 64-row step never straddles a key block (64 divides every split point)
        int64_t pk = 0, pv = 0;
        const char* kp = RAGGED ? nullptr : row_ptr(a.k, b, k0, hk, &pk);
        const char* vp = RAGGED ? nullptr : row_ptr(a.v, b, k0, hk, &pv);
        const uint32_t dk = smem_u32(sK) + buf * KT * ROW_BYTES, dv = smem_u32(sV) + buf * KT * ROW_BYTES;
        for (int i = tid; i < KT * 16; i += NT) {
            int r = i / 16, c = i % 16;
            if (!RAGGED) {
                cp_async16(dk + swz(r, c), kp + (int64_t)r * pk + c * 16);
                cp_async16(dv + swz(r, c), vp + (int64_t)r * pv + c * 16);
            } else if (k0 + r < a.S) {   // every row on its own: a step may straddle key blocks
                cp_async16(dk + swz(r, c), row_ptr(a.k, b, k0 + r, hk, &pk) + c * 16);
                cp_async16(dv + swz(r, c), row_ptr(a.v, b, k0 + r, hk, &pv) + c * 16);
            } else {                     // past the end of the index: zeros (their scores are masked, 0 * V must not be NaN)
                const uint32_t off = swz(r, c);
                *reinterpret_cast<uint4*>(sK + buf * KT * ROW_BYTES + off) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4*>(sV + buf * KT * ROW_BYTES + off) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        cp_async_commit();
    };
    load_kv(0, 0);

    cp_async_wait<1>();  // Q has landed
    __syncthreads();
    uint32_t qf[8][4];
    {
        const int r = warp * 16 + (lane % 8) + 8 * ((lane / 8) % 2);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const int chunk = ks * 2 + lane / 16;
            ldmatrix_x4(smem_u32(sQ) + swz(r, chunk), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
        }
    }

    float o[16][4];
#pragma unroll
    for (int n = 0; n < 16; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const float sl2 = a.scale * 1.4426950408889634f;  // scores are kept in the base-2 exponent domain
    const int row0 = q0 + warp * 16 + g;              // sequence position of this thread's first row (second: +8)
    int rs0[2] = {0, 0}, rs1[2] = {0, 0};             // RAGGED: keys [rs0, rs1) are the sequence of each of the two rows; empty past the end
    if (RAGGED) {
#pragma unroll
        for (int r = 0; r < 2; ++r)
            if (row0 + 8 * r < a.S) seq_bounds(a, row0 + 8 * r, rs0[r], rs1[r]);
    }

    for (int step = 0; step < n_steps; ++step) {
        const int buf = step & 1;
        if (step + 1 < n_steps) { load_kv(step + 1, buf ^ 1); cp_async_wait<1>(); }
        else cp_async_wait<0>();
        __syncthreads();
        const uint32_t kbase = smem_u32(sK) + buf * KT * ROW_BYTES, vbase = smem_u32(sV) + buf * KT * ROW_BYTES;

        // ---- S = Q K^T for 16 rows x 64 keys -------------------------------------------------------------------
        float s[8][4];
#pragma unroll
        for (int n = 0; n < 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {  // pairs of 8-key tiles
                const int mi = lane / 8;
                const int krow = np * 16 + (mi / 2) * 8 + (lane % 8);
                const int chunk = ks * 2 + (mi % 2);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(kbase + swz(krow, chunk), b0, b1, b2, b3);
                mma_16bit<F16>(s[2 * np], qf[ks], b0, b1);
                mma_16bit<F16>(s[2 * np + 1], qf[ks], b2, b3);
            }
        }
        // ---- scale, causal band inside the diagonal block, row max ---------------------------------------------
        const int k0 = s0 + step * KT;
        const bool diag = a.causal && (k0 + KT - 1 > q0 + warp * 16);
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int n = 0; n < 8; ++n) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float v = s[n][e] * sl2;
                if (RAGGED) {
                    const int key = k0 + n * 8 + 2 * t4 + (e & 1);
                    const int row = row0 + 8 * (e >> 1);
                    if (key < rs0[e >> 1] || key >= rs1[e >> 1] || (a.causal && key > row)) v = -INFINITY;
                } else if (diag) {
                    const int key = k0 + n * 8 + 2 * t4 + (e & 1);
                    const int row = row0 + 8 * (e >> 1);
                    if (key > row) v = -INFINITY;
                }
                s[n][e] = v;
                mx[e >> 1] = fmaxf(mx[e >> 1], v);
            }
        }
        float alpha[2], m_use[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            const float m_new = fmaxf(m_run[r], mx[r]);
            m_use[r] = (m_new == -INFINITY) ? 0.f : m_new;               // e^(-inf - -inf) := 0
            alpha[r] = (m_run[r] == -INFINITY) ? 0.f : exp2f(m_run[r] - m_use[r]);
            m_run[r] = m_new;
        }
        // ---- P = 2^(S - m), row sums, O~ <- O~ alpha ----------------------------------------------------------------
        float ls[2] = {0.f, 0.f};
        uint32_t pf[4][4];
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            float p0 = exp2f(s[n][0] - m_use[0]), p1 = exp2f(s[n][1] - m_use[0]);
            float p2 = exp2f(s[n][2] - m_use[1]), p3 = exp2f(s[n][3] - m_use[1]);
            ls[0] += p0 + p1;
            ls[1] += p2 + p3;
            pf[n / 2][(n % 2) * 2 + 0] = ja_pack16<F16>(p0, p1);
            pf[n / 2][(n % 2) * 2 + 1] = ja_pack16<F16>(p2, p3);
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) l_run[r] = l_run[r] * alpha[r] + ls[r];
#pragma unroll
        for (int n = 0; n < 16; ++n) {
            o[n][0] *= alpha[0]; o[n][1] *= alpha[0];
            o[n][2] *= alpha[1]; o[n][3] *= alpha[1];
        }
        // ---- O~ += P V ----------------------------------------------------------------------------------------------
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {      // 16 keys per step
#pragma unroll
            for (int np = 0; np < 8; ++np) {  // pairs of 8-wide d tiles
                const int mi = lane / 8;
                const int vrow = ks * 16 + (mi % 2) * 8 + (lane % 8);
                const int chunk = np * 2 + (mi / 2);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(vbase + swz(vrow, chunk), b0, b1, b2, b3);
                mma_16bit<F16>(o[2 * np], pf[ks], b0, b1);
                mma_16bit<F16>(o[2 * np + 1], pf[ks], b2, b3);
            }
        }
        __syncthreads();  // everyone is done with this buffer before it is refilled
    }

    // ---- finish: O = O~ / l, stage through shared memory, 16-byte stores --------------------------------------------
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    }
    const float inv0 = l_run[0] > 0.f ? 1.f / l_run[0] : 0.f, inv1 = l_run[1] > 0.f ? 1.f / l_run[1] : 0.f;
    if (a.lse.base && t4 == 0) {   // second output: log of the softmax denominator (scores were kept in base 2)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            if (RAGGED && row0 + 8 * r >= a.S) continue;
            const int64_t x[3] = {b, row0 + 8 * r, h};
            *reinterpret_cast<float*>(a.lse.base + ja_elem_off(a.lse, x)) = (m_run[r] + log2f(l_run[r])) * 0.6931471805599453f;
        }
    }
    {
        const int r_lo = warp * 16 + g, r_hi = r_lo + 8;
#pragma unroll
        for (int n = 0; n < 16; ++n) {
            // columns n*8 + 2*t4, +1  -> chunk n, byte (2*t4)*2 inside it
            *reinterpret_cast<uint32_t*>(sQ + swz(r_lo, n) + t4 * 4) = ja_pack16<F16>(o[n][0] * inv0, o[n][1] * inv0);
            *reinterpret_cast<uint32_t*>(sQ + swz(r_hi, n) + t4 * 4) = ja_pack16<F16>(o[n][2] * inv1, o[n][3] * inv1);
        }
    }
    __syncthreads();
    {
        int64_t pitch;
        char* op = RAGGED ? nullptr : const_cast<char*>(row_ptr(a.o, b, q0, h, &pitch));
        for (int i = tid; i < QT * 16; i += NT) {
            int r = i / 16, c = i % 16;
            if (RAGGED) {
                if (q0 + r >= a.S) continue;
                op = const_cast<char*>(row_ptr(a.o, b, q0 + r, h, &pitch)) - (int64_t)r * pitch;
            }
            *reinterpret_cast<uint4*>(op + (int64_t)r * pitch + c * 16) = *reinterpret_cast<const uint4*>(sQ + swz(r, c));
        }
    }
}

}  // namespace

ja_status_t ja_launch_attention(const AttnArgs& a, cudaStream_t st) {
    if (ja_config().attn_mma_sync != 1) {
        bool launched = false;
        ja_status_t s = ja_launch_attention_tc(a, st, &launched);
        if (s != JA_OK || launched) return s;
    }
    const bool ragged = a.align % 64 != 0;       // some split point, sequence end or the length itself is not a multiple of 64 rows
    const int QT = (a.align % 128 == 0) ? 128 : 64;
    const int n_qt = (a.S + QT - 1) / QT;
    AttnArgs a2 = a;
    a2.sect = (a.causal || a.n_ends > 1) ? a.H * a.B : std::min<int>(a.H * a.B, std::max(1, (ja_sm_count() + n_qt - 1) / n_qt));
    dim3 grid((unsigned)((int64_t)a.H * a.B * n_qt), 1, 1);
    const int smem = QT * ROW_BYTES + 4 * KT * ROW_BYTES;
#define JA_ATTN_SYNC(Q, F, R)                                                                                          \
    do {                                                                                                              \
        JA_CUDA(cudaFuncSetAttribute(attention_kernel<Q, F, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)); \
        attention_kernel<Q, F, R><<<grid, 2 * Q, smem, st>>>(a2);                                                    \
    } while (0)
    if (ragged) {
        if (a.f16) JA_ATTN_SYNC(64, true, true);
        else JA_ATTN_SYNC(64, false, true);
    } else if (QT == 128) {
        if (a.f16) JA_ATTN_SYNC(128, true, false);
        else JA_ATTN_SYNC(128, false, false);
    } else {
        if (a.f16) JA_ATTN_SYNC(64, true, false);
        else JA_ATTN_SYNC(64, false, false);
    }
#undef JA_ATTN_SYNC
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}
