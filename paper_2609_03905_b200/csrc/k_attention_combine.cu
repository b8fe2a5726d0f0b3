// The online-softmax aggregation of the attention join-agg as a step of its own (Definition 3.7 step 2 when the function
// specs of one output key were executed apart -- over disjoint ranges of the key index, Section 5.1 -- and each left a
// normalised partial result O_c together with lse_c, the log of its softmax denominator):
//     lse = log sum_c exp(lse_c),   O = sum_c exp(lse_c - lse) O_c,
// which is (O~, m, l) (+) (O~', m', l') written for results that were already divided by their l (O_c = O~_c / l_c,
// lse_c = m_c + log l_c). Copies are combined in ascending order in f32 and O is rounded once. A copy whose lse is -inf
// (no key of its range joined with the row) contributes nothing; a row with no key at all gets O = 0 and lse = -inf.
// The partial results are m separate relations (each the output pair of one ja_execute over its key range), at most eight.
// One 16-byte vector of a (batch, position, head) row of 128 cells per lane; every row of every relation is located
// through its key table, so the partial relations and the outputs may be tiled in any way, each its own. HBM-bound:
// m + 1 rows moved.
#include <stdlib.h>
#include <string.h>

#include "ja_device.cuh"

namespace {

constexpr int MAX_COPIES = 8;
struct CombineParams {
    RelView op[MAX_COPIES], lp[MAX_COPIES];   // partial outputs [b,s,h,d] and their lse [b,s,h] (f32), one relation per copy
    RelView o, l;                             // output [b,s,h,d], its lse [b,s,h] (f32, optional)
    int32_t m, has_l;
    int64_t B, S, H;
    // FAST form: every O relation has the tiling of o and every lse relation that of o's first three indices, all blocks of
    // one shape. A payload then is a run of rows in one common order: row i lies in block i / rows_per_blk.
    int64_t rows_per_blk, o_blk_stride, l_blk_stride;
};

// one 16-byte vector of a row: 4 f32 cells or 8 16-bit cells
template <typename T> struct Vec16 { static constexpr int CELLS = 16 / (int)sizeof(T); };
template <typename T> __device__ __forceinline__ void unpack_vec(const uint4& v, float (&f)[Vec16<T>::CELLS]);
template <> __device__ __forceinline__ void unpack_vec<float>(const uint4& v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
template <bool F16> __device__ __forceinline__ void unpack_vec16(const uint4& v, float (&f)[8]) {
    const float2 a = ja_unpack16<F16>(v.x), b = ja_unpack16<F16>(v.y), c = ja_unpack16<F16>(v.z), d = ja_unpack16<F16>(v.w);
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
}
template <> __device__ __forceinline__ void unpack_vec<__nv_bfloat16>(const uint4& v, float (&f)[8]) { unpack_vec16<false>(v, f); }
template <> __device__ __forceinline__ void unpack_vec<__half>(const uint4& v, float (&f)[8]) { unpack_vec16<true>(v, f); }
template <typename T> __device__ __forceinline__ uint4 pack_vec(const float (&f)[Vec16<T>::CELLS]);
template <> __device__ __forceinline__ uint4 pack_vec<float>(const float (&f)[4]) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
template <> __device__ __forceinline__ uint4 pack_vec<__nv_bfloat16>(const float (&f)[8]) {
    return make_uint4(ja_pack16<false>(f[0], f[1]), ja_pack16<false>(f[2], f[3]), ja_pack16<false>(f[4], f[5]), ja_pack16<false>(f[6], f[7]));
}
template <> __device__ __forceinline__ uint4 pack_vec<__half>(const float (&f)[8]) {
    return make_uint4(ja_pack16<true>(f[0], f[1]), ja_pack16<true>(f[2], f[3]), ja_pack16<true>(f[4], f[5]), ja_pack16<true>(f[6], f[7]));
}

// MC: capacity in copies (2, 4 or 8). A lane holds one 16-byte vector of a row, so a row of 128 cells takes 16 lanes (16-bit
// cells) or 32 (f32) and a warp-wide load covers RPL = 2 or 1 rows; a warp takes R = 2 (MC = 2) or 1 such loads per copy and
// round, kept packed in registers until they are used. More rows per round (R = 8 / MC: 4 KiB in flight per warp) cost more in
// registers, and so in resident warps, than they brought: 45.9 / 75.0 us against 37.0 / 58.7 for m = 2 / 4 on
// 4 x 2048 x 32 rows of bf16.
template <typename T, bool FAST, int MC>
__global__ void __launch_bounds__(256) attention_combine_kernel(const CombineParams p) {
    constexpr int R = (MAX_COPIES / MC + 1) / 2, CELLS = Vec16<T>::CELLS, LPR = 128 / CELLS, RPL = 32 / LPR, ROWS = R * RPL;
    const int lane = threadIdx.x & 31, sub = lane / LPR, col = (lane % LPR) * 16;      // col: byte offset of the lane's vector in its row
    const uint32_t warps = gridDim.x * 8u, n_rows = (uint32_t)(p.B * p.S * p.H);   // the host keeps the row count below 2^31
    for (uint32_t row0 = (blockIdx.x * 8u + (threadIdx.x >> 5)) * ROWS; row0 < n_rows; row0 += warps * ROWS) {
        // FAST: rows are counted in payload order, the same in every relation; otherwise `row` is the flat (b, s, h) and every
        // relation's key table is asked
        int64_t xd[R][4], o_off[R], l_off[R];     // (b, s, h) for the statistics relations, (b, s, h, 0) for the rows of cells
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const uint32_t row = min(row0 + r * RPL + sub, n_rows - 1);     // rows past the end repeat the last one and are not stored
            xd[r][0] = xd[r][1] = xd[r][2] = xd[r][3] = 0;
            o_off[r] = l_off[r] = 0;
            if (FAST) {
                const uint32_t blk = row / (uint32_t)p.rows_per_blk, rin = row - blk * (uint32_t)p.rows_per_blk;
                o_off[r] = (int64_t)blk * p.o_blk_stride + (int64_t)rin * (128 * (int)sizeof(T));
                l_off[r] = (int64_t)blk * p.l_blk_stride + (int64_t)rin * 4;
            } else {
                const uint32_t H = (uint32_t)p.H, S = (uint32_t)p.S;
                xd[r][2] = row % H;
                xd[r][1] = (row / H) % S;
                xd[r][0] = row / (H * S);
            }
        }
        // every load of the round first: the statistics and the rows of cells of all copies, none depends on another
        float lc[R][MC];
        uint4 raw[R][MC];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int c = 0; c < MC; ++c) {
                lc[r][c] = -INFINITY;
                raw[r][c] = make_uint4(0u, 0u, 0u, 0u);
                if (c < p.m) {
                    lc[r][c] = *reinterpret_cast<const float*>(p.lp[c].base + (FAST ? l_off[r] : ja_elem_off(p.lp[c], xd[r])));
                    raw[r][c] = *reinterpret_cast<const uint4*>(p.op[c].base + (FAST ? o_off[r] : ja_elem_off(p.op[c], xd[r])) + col);
                }
            }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < MC; ++c) mx = fmaxf(mx, lc[r][c]);
            float sum = 0.f;
            if (mx > -INFINITY) {
#pragma unroll
                for (int c = 0; c < MC; ++c)
                    if (c < p.m) sum += __expf(lc[r][c] - mx);
            }
            const float lse = mx > -INFINITY ? mx + __logf(sum) : -INFINITY;
            // the weighted sum of the partial rows, ascending copy order
            float acc[CELLS];
#pragma unroll
            for (int e = 0; e < CELLS; ++e) acc[e] = 0.f;
            if (mx > -INFINITY) {
#pragma unroll
                for (int c = 0; c < MC; ++c) {
                    if (c >= p.m) continue;
                    const float w = __expf(lc[r][c] - lse);
                    if (w == 0.f) continue;      // also keeps a copy that holds nothing valid (lse = -inf, cells unspecified) out of the sum
                    float f[CELLS];
                    unpack_vec<T>(raw[r][c], f);
#pragma unroll
                    for (int e = 0; e < CELLS; ++e) acc[e] = fmaf(w, f[e], acc[e]);
                }
            }
            if (row0 + r * RPL + sub < n_rows) {
                *reinterpret_cast<uint4*>(p.o.base + (FAST ? o_off[r] : ja_elem_off(p.o, xd[r])) + col) = pack_vec<T>(acc);
                if (p.has_l && col == 0) *reinterpret_cast<float*>(p.l.base + (FAST ? l_off[r] : ja_elem_off(p.l, xd[r]))) = lse;
            }
        }
    }
}

}  // namespace

// m <= 8 copies; every relation is on the device and validated by the caller
ja_status_t ja_launch_attention_combine(const ja_relation* const* op, const ja_relation* const* lp, int m, const ja_relation* o,
                                        const ja_relation* l, cudaStream_t st) {
    if (m < 1 || m > MAX_COPIES) return ja_fail(JA_ERR_UNSUPPORTED, "between 1 and %d partial results", MAX_COPIES);
    CombineParams p;
    memset(&p, 0, sizeof p);
    for (int c = 0; c < m; ++c) {
        p.op[c] = ja_view(op[c]);
        p.lp[c] = ja_view(lp[c]);
    }
    p.o = ja_view(o);
    if (l) p.l = ja_view(l);
    p.has_l = l ? 1 : 0;
    p.m = m;
    p.B = o->extent[0]; p.S = o->extent[1]; p.H = o->extent[2];
    // one tiling with blocks of one shape everywhere: rows are addressed by arithmetic on their number in payload order
    bool fast = o->equal_blocks && o->nblocks > 0;
    auto same = [](const ja_relation* a, const ja_relation* b, int rank) {
        for (int d = 0; d < rank; ++d)
            if (a->splits[d] != b->splits[d]) return false;
        return a->equal_blocks;
    };
    const int64_t l_stride = lp[0]->nblocks > 1 ? lp[0]->blk_off[1] - lp[0]->blk_off[0] : 0;
    for (int c = 0; c < m && fast; ++c) {
        fast = same(op[c], o, 4) && same(lp[c], o, 3) && lp[c]->nblocks == o->nblocks &&
               (lp[c]->nblocks > 1 ? lp[c]->blk_off[1] - lp[c]->blk_off[0] : 0) == l_stride;
    }
    if (fast && l) fast = same(l, o, 3) && l->nblocks == o->nblocks && (l->nblocks > 1 ? l->blk_off[1] - l->blk_off[0] : 0) == l_stride;
    if (fast) {
        p.rows_per_blk = o->bs[0] * o->bs[1] * o->bs[2];
        p.o_blk_stride = o->nblocks > 1 ? o->blk_off[1] - o->blk_off[0] : 0;
        p.l_blk_stride = l_stride;
    }
    const int rows_per_warp = (m <= 2 ? 2 : 1) * (o->dtype == JA_F32 ? 1 : 2);
    const int64_t n_rows = p.B * p.S * p.H, want = (n_rows + 8 * rows_per_warp - 1) / (8 * rows_per_warp), cap = (int64_t)ja_sm_count() * 16;
    if (n_rows >= (1ll << 31)) return ja_fail(JA_ERR_UNSUPPORTED, "more than 2^31 (batch, position, head) rows");
    const unsigned grid = (unsigned)(want < cap ? (want > 0 ? want : 1) : cap);
#define JA_COMBINE_MC(T, MC)                                                          \
    do {                                                                              \
        if (fast) attention_combine_kernel<T, true, MC><<<grid, 256, 0, st>>>(p);    \
        else attention_combine_kernel<T, false, MC><<<grid, 256, 0, st>>>(p);        \
    } while (0)
#define JA_COMBINE(T)                                                                 \
    do {                                                                              \
        if (m <= 2) JA_COMBINE_MC(T, 2);                                              \
        else if (m <= 4) JA_COMBINE_MC(T, 4);                                         \
        else JA_COMBINE_MC(T, 8);                                                     \
    } while (0)
    if (o->dtype == JA_F32) JA_COMBINE(float);
    else if (o->dtype == JA_F16) JA_COMBINE(__half);
    else JA_COMBINE(__nv_bfloat16);
#undef JA_COMBINE_MC
#undef JA_COMBINE
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}
