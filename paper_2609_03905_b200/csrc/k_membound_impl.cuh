// Memory-bound join-aggs on the block-key layout.
//
//  * flat key-aligned maps ("X,X->X": ADD, SILU_MUL): operands tiled identically have identical payload
//    layouts, so the join on block keys and on in-block cells is a walk over the payloads in lockstep.
//  * row-structured forms ("Rj..."): a team of threads owns one row key R; the row's cells live in the
//    nblk(j) blocks that share R's block key, and the team walks them in ascending j -- for the reductions
//    (SQUARE/SUM, IDENT/MAX, EXP_SUB/SUM) that walk IS the aggregation over the function specs that share an
//    output key (Definition 3.7); the partial never leaves registers.
//
// All loads/stores are 128-bit when the tiling allows (every split of j a multiple of the vector width).
#pragma once

#include <stdlib.h>
#include <string.h>

#include "ja_device.cuh"

namespace {

// ---------------------------------------------------------------------------------------------------
// flat maps
// ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ float silu_mul_f(float a, float b) { return a / (1.f + __expf(-a)) * b; }

template <int FN>
__device__ __forceinline__ float flat_fn(float a, float b) {
    return FN == JA_FN_ADD ? a + b : silu_mul_f(a, b);
}

// eight 16-bit cells per 16-byte vector; F16: false = bf16, true = f16
template <int FN, bool F16>
__global__ void __launch_bounds__(256) flat_16bit_kernel(const uint4* __restrict__ a, const uint4* __restrict__ b,
                                                         uint4* __restrict__ out, int64_t n_vec) {
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * 256) {
        uint4 va = a[i], vb = b[i], vo;
        const uint32_t* pa = reinterpret_cast<const uint32_t*>(&va);
        const uint32_t* pb = reinterpret_cast<const uint32_t*>(&vb);
        uint32_t* po = reinterpret_cast<uint32_t*>(&vo);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float2 fa = ja_unpack16<F16>(pa[k]), fb = ja_unpack16<F16>(pb[k]);
            po[k] = ja_pack16<F16>(flat_fn<FN>(fa.x, fb.x), flat_fn<FN>(fa.y, fb.y));
        }
        out[i] = vo;
    }
}

template <int FN>
__global__ void __launch_bounds__(256) flat_f32_kernel(const float4* __restrict__ a, const float4* __restrict__ b,
                                                       float4* __restrict__ out, int64_t n_vec) {
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * 256) {
        float4 va = a[i], vb = b[i], vo;
        vo.x = flat_fn<FN>(va.x, vb.x); vo.y = flat_fn<FN>(va.y, vb.y);
        vo.z = flat_fn<FN>(va.z, vb.z); vo.w = flat_fn<FN>(va.w, vb.w);
        out[i] = vo;
    }
}

// ---------------------------------------------------------------------------------------------------
// row-structured forms
// ---------------------------------------------------------------------------------------------------
template <typename T, int VEC>
struct alignas(sizeof(T) * VEC) Vec {
    T e[VEC];
};

struct RowCtx {
    int64_t lead_flat;  // flat block key over the leading dimensions
    int64_t lead_in;    // row offset inside that block (row-major over the block's leading extents)
    int pos;            // coordinate of the second index (RoPE position)
    int64_t stat_off;   // byte offset of this row's cell in a statistics relation keyed by R
};

// 32-bit coordinate arithmetic (extents are < 2^31): 64-bit division is a long software routine and would
// dominate these memory-bound kernels. On uniform tilings every lookup is arithmetic -- no table is read.
__device__ __forceinline__ void dim_lookup(const RelView& v, int d, int x, int* b, int* lo, int* w) {
    if (v.bs[d]) {
        const int bs = (int)v.bs[d];
        const int bb = (int)((uint32_t)x / (uint32_t)bs);
        *b = bb;
        *lo = bb * bs;
        *w = min(bs, (int)v.extent[d] - bb * bs);
        return;
    }
    int l = 0, h = v.nblk[d] - 1;
    while (l < h) {
        int mid = (l + h + 1) >> 1;
        if (v.splits[d][mid] <= (int64_t)x) l = mid;
        else h = mid - 1;
    }
    *b = l;
    *lo = (int)v.splits[d][l];
    *w = (int)v.splits[d][l + 1] - *lo;
}
__device__ __forceinline__ int64_t blk_offset(const RelView& v, int64_t flat) {
    return v.blk_stride ? flat * v.blk_stride : v.blk_off[flat];
}

__device__ __forceinline__ RowCtx row_ctx(const RelView& x, const RelView& stat, bool has_stat, int64_t row) {
    RowCtx c;
    int lead[JA_MAX_RANK] = {0, 0, 0, 0};
    uint32_t rem = (uint32_t)row;
    for (int d = x.rank - 2; d >= 0; --d) {
        const uint32_t e = (uint32_t)x.extent[d];
        const uint32_t qd = rem / e;
        lead[d] = (int)(rem - qd * e);
        rem = qd;
    }
    c.lead_flat = 0;
    c.lead_in = 0;
    for (int d = 0; d < x.rank - 1; ++d) {
        int b, lo, w;
        dim_lookup(x, d, lead[d], &b, &lo, &w);
        c.lead_flat = c.lead_flat * x.nblk[d] + b;
        c.lead_in = c.lead_in * w + (lead[d] - lo);
    }
    c.pos = lead[1];
    // the statistics relation is keyed by the same leading indices with the same splits
    c.stat_off = has_stat ? blk_offset(stat, c.lead_flat) + c.lead_in * stat.esize : 0;
    return c;
}

// byte offset of the vector starting at column `col` of the row
__device__ __forceinline__ int64_t vec_off(const RelView& x, const RowCtx& c, int col) {
    const int last = x.rank - 1;
    int b, l, w;
    dim_lookup(x, last, col, &b, &l, &w);
    return blk_offset(x, c.lead_flat * x.nblk[last] + b) + (c.lead_in * w + (col - l)) * x.esize;
}

template <bool IS_MAX>
__device__ __forceinline__ float team_reduce(float v, int team, float* smem, int row_in_cta, int lane_t) {
    const int w = team < 32 ? team : 32;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        if (o < w) {
            float other = __shfl_xor_sync(0xffffffffu, v, o);
            v = IS_MAX ? fmaxf(v, other) : v + other;
        }
    }
    if (team > 32) {  // uniform across the CTA: every thread takes this branch or none does
        const int warps = team / 32;
        __syncthreads();
        if ((lane_t & 31) == 0) smem[row_in_cta * 8 + lane_t / 32] = v;
        __syncthreads();
        float r = smem[row_in_cta * 8];
        for (int k = 1; k < warps; ++k) {
            float other = smem[row_in_cta * 8 + k];
            r = IS_MAX ? fmaxf(r, other) : r + other;
        }
        v = r;
    }
    return v;
}

// OP semantics: see RowOp in ja_internal.h. VPT > 0: the row stays in registers between passes (VPT vectors
// per thread). VPT == 0: streaming fallback for long or unaligned rows, later passes re-read the row.
template <typename T, int VEC, int VPT, int OP>
__global__ void __launch_bounds__(256) row_kernel(RowArgs a, int64_t n_rows, int team) {
    __shared__ float red[64];
    constexpr bool RES = VPT > 0;
    constexpr int NV = RES ? VPT : 1;
    using V = Vec<T, VEC>;
    const int rpc = 256 / team;
    const int row_in_cta = threadIdx.x / team, lane_t = threadIdx.x % team;
    const int last = a.x.rank - 1;
    const int n = (int)a.x.extent[last];
    const int64_t row = (int64_t)blockIdx.x * rpc + row_in_cta;
    const bool live = row < n_rows;
    constexpr bool HAS_STAT = (OP == ROW_SUMSQ || OP == ROW_MAX || OP == ROW_EXPSUM || OP == ROW_RMS_SCALE ||
                               OP == ROW_EXP_SUB_DIV);
    RowCtx ctx = row_ctx(a.x, a.s0, HAS_STAT, live ? row : 0);

    V raw[NV];
    // ---- pass 0: load (resident mode) -------------------------------------------------------------------
    if (RES) {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int col = (k * team + lane_t) * VEC;
            if (live && col < n) raw[k] = *reinterpret_cast<const V*>(a.x.base + vec_off(a.x, ctx, col));
        }
    }
    // iterate over this thread's vectors: f(col, value)
    auto for_each = [&](auto f) {
        if (RES) {
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int col = (k * team + lane_t) * VEC;
                if (live && col < n) f(col, raw[k]);
            }
        } else if (live) {
            for (int col = lane_t * VEC; col < n; col += team * VEC) {
                V v = *reinterpret_cast<const V*>(a.x.base + vec_off(a.x, ctx, col));
                f(col, v);
            }
        }
    };

    float m = 0.f, l = 0.f, rstd = 0.f;
    // ---- reductions ----------------------------------------------------------------------------------------
    if (OP == ROW_SUMSQ || OP == ROW_RMSNORM) {
        float s = 0.f;
        for_each([&](int, const V& v) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) { float f = ja_to_float(v.e[e]); s = fmaf(f, f, s); }
        });
        s = team_reduce<false>(s, team, red, row_in_cta, lane_t);
        if (OP == ROW_SUMSQ) {
            if (live && lane_t == 0) *reinterpret_cast<float*>(a.s0.base + ctx.stat_off) = s;
            return;
        }
        rstd = 1.0f / sqrtf(s / (float)n + a.eps);
    }
    if (OP == ROW_MAX || OP == ROW_SOFTMAX) {
        float mx = -INFINITY;
        for_each([&](int, const V& v) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) mx = fmaxf(mx, ja_to_float(v.e[e]));
        });
        m = team_reduce<true>(mx, team, red, row_in_cta, lane_t);
        if (OP == ROW_MAX) {
            if (live && lane_t == 0) *reinterpret_cast<float*>(a.s0.base + ctx.stat_off) = m;
            return;
        }
    }
    if (OP == ROW_EXPSUM || OP == ROW_EXP_SUB_DIV) m = live ? *reinterpret_cast<const float*>(a.s0.base + ctx.stat_off) : 0.f;
    if (OP == ROW_EXPSUM || OP == ROW_SOFTMAX) {
        float s = 0.f;
        for_each([&](int, const V& v) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) s += __expf(ja_to_float(v.e[e]) - m);
        });
        l = team_reduce<false>(s, team, red, row_in_cta, lane_t);
        if (OP == ROW_EXPSUM) {
            if (live && lane_t == 0) *reinterpret_cast<float*>(a.s1.base + ctx.stat_off) = l;
            return;
        }
    }
    if (OP == ROW_EXP_SUB_DIV) l = live ? *reinterpret_cast<const float*>(a.s1.base + ctx.stat_off) : 1.f;
    if (OP == ROW_RMS_SCALE) {
        float ss = live ? *reinterpret_cast<const float*>(a.s0.base + ctx.stat_off) : 1.f;
        rstd = 1.0f / sqrtf(ss / (float)n + a.eps);
    }
    // ---- map + store ---------------------------------------------------------------------------------------
    const float inv_l = (OP == ROW_SOFTMAX || OP == ROW_EXP_SUB_DIV) ? 1.0f / l : 0.f;
    for_each([&](int col, const V& v) {
        V o;
        if (OP == ROW_RMS_SCALE || OP == ROW_RMSNORM) {
            int cb, glo, gw;
            dim_lookup(a.g, 0, col, &cb, &glo, &gw);
            const int64_t goff = blk_offset(a.g, cb) + (col - glo) * a.g.esize;
            V g = *reinterpret_cast<const V*>(a.g.base + goff);
#pragma unroll
            for (int e = 0; e < VEC; ++e) o.e[e] = ja_from_float<T>(ja_to_float(v.e[e]) * rstd * ja_to_float(g.e[e]));
        } else if (OP == ROW_SOFTMAX || OP == ROW_EXP_SUB_DIV) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) o.e[e] = ja_from_float<T>(__expf(ja_to_float(v.e[e]) - m) * inv_l);
        } else if (OP == ROW_ROPE) {
            const float2* tab = a.rope_table + (ctx.pos * a.rope_d + (col % a.rope_d)) / 2;
#pragma unroll
            for (int e = 0; e + 1 < VEC; e += 2) {
                float2 cs = tab[e / 2];
                float x0 = ja_to_float(v.e[e]), x1 = ja_to_float(v.e[e + 1]);
                o.e[e] = ja_from_float<T>(x0 * cs.x - x1 * cs.y);
                o.e[e + 1] = ja_from_float<T>(x0 * cs.y + x1 * cs.x);
            }
        }
        *reinterpret_cast<V*>(a.y.base + vec_off(a.y, ctx, col)) = o;  // y is tiled exactly like x
    });
}

// ---------------------------------------------------------------------------------------------------
// fast path: equal-sized blocks in every dimension. The payload offset of cell (row, col) separates into
//     rowpart(row) + colpart(col),   rowpart = row-block strip + row inside the block, colpart = column block + column
// so a thread computes colpart once for its fixed set of columns, a team computes rowpart once per row, and the
// inner loops contain no division and no table lookup. CTAs are persistent over rows.
// ---------------------------------------------------------------------------------------------------
struct FastGeom {
    int n, bsc, nbc;            // row length, column-block width, column blocks
    int blk_elems;              // elements between consecutive blocks of x / y (equal shapes, padding included)
    int lead_rank;              // leading dimensions (1..3)
    int lead_ext[3], lead_bs[3], lead_nb[3];
    int stat_blk_bytes;         // bytes between consecutive blocks of a statistics relation
    int g_blk_bytes;            // bytes between consecutive blocks of the gain vector
    int rope_d;
};

template <typename T, int VEC, int VPT, int OP>
__global__ void __launch_bounds__(256, (VPT <= 2 ? 4 : (VPT <= 4 ? 3 : 1))) row_fast_kernel(RowArgs a, FastGeom g, int64_t n_rows, int team) {
    __shared__ float red[64];
    using V = Vec<T, VEC>;
    const int rpc = blockDim.x / team;
    const int row_in_cta = threadIdx.x / team, lane_t = threadIdx.x % team;
    constexpr bool HAS_G = (OP == ROW_RMS_SCALE || OP == ROW_RMSNORM);
    constexpr bool KEEP_EXP = (OP == ROW_SOFTMAX);

    int colpart[VPT];
    int gpart[HAS_G ? VPT : 1];   // byte offset of the matching cells of the gain vector
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int col = (k * team + lane_t) * VEC;
        colpart[k] = -1;
        if (col < g.n) {
            const int cb = (int)((uint32_t)col / (uint32_t)g.bsc);
            const int ci = col - cb * g.bsc;
            colpart[k] = cb * g.blk_elems + ci;
            if (HAS_G) gpart[k] = cb * g.g_blk_bytes + ci * (int)sizeof(T);
        }
    }
    const int64_t strip = (int64_t)g.nbc * g.blk_elems;  // elements in one strip of column blocks

    // rowpart, statistics offset and position of one row
    struct RowGeom { int64_t rowpart, stat_off; int pos; bool live; };
    auto geom = [&](int64_t row) {
        RowGeom rg;
        rg.live = row < n_rows;
        uint32_t rem = (uint32_t)(rg.live ? row : 0);
        int lead_flat = 0, lead_in = 0;
        int c[3] = {0, 0, 0};
#pragma unroll
        for (int d = 2; d >= 0; --d) {
            if (d < g.lead_rank) {
                const uint32_t q = rem / (uint32_t)g.lead_ext[d];
                c[d] = (int)(rem - q * (uint32_t)g.lead_ext[d]);
                rem = q;
            }
        }
#pragma unroll
        for (int d = 0; d < 3; ++d) {
            if (d < g.lead_rank) {
                const int b = (int)((uint32_t)c[d] / (uint32_t)g.lead_bs[d]);
                lead_flat = lead_flat * g.lead_nb[d] + b;
                lead_in = lead_in * g.lead_bs[d] + (c[d] - b * g.lead_bs[d]);
            }
        }
        rg.pos = c[1];
        rg.rowpart = (int64_t)lead_flat * strip + (int64_t)lead_in * g.bsc;
        rg.stat_off = (int64_t)lead_flat * g.stat_blk_bytes + (int64_t)lead_in * 4;
        return rg;
    };

    // software pipeline over rows: the loads of the next row are in flight while this row is reduced and written
    const int64_t row_step = (int64_t)gridDim.x * rpc;
    RowGeom cur = geom((int64_t)blockIdx.x * rpc + row_in_cta);
    V raw[VPT], nxt[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k)
        if (cur.live && colpart[k] >= 0) raw[k] = *reinterpret_cast<const V*>(reinterpret_cast<const T*>(a.x.base) + cur.rowpart + colpart[k]);

    for (int64_t row0 = (int64_t)blockIdx.x * rpc; row0 < n_rows; row0 += row_step) {
        const bool live = cur.live;
        const int pos = cur.pos;
        const int64_t stat_off = cur.stat_off;
        T* yrow = reinterpret_cast<T*>(a.y.base) + cur.rowpart;
        RowGeom nx = geom(row0 + row_step + row_in_cta);
#pragma unroll
        for (int k = 0; k < VPT; ++k)
            if (nx.live && colpart[k] >= 0) nxt[k] = *reinterpret_cast<const V*>(reinterpret_cast<const T*>(a.x.base) + nx.rowpart + colpart[k]);
        auto advance = [&]() {
#pragma unroll
            for (int k = 0; k < VPT; ++k) raw[k] = nxt[k];
            cur = nx;
        };

        float m = 0.f, l = 0.f, rstd = 0.f;
        float ex[KEEP_EXP ? VPT * VEC : 1];
        if (OP == ROW_SUMSQ || OP == ROW_RMSNORM) {
            float s = 0.f;
#pragma unroll
            for (int k = 0; k < VPT; ++k)
                if (live && colpart[k] >= 0) {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) { float f = ja_to_float(raw[k].e[e]); s = fmaf(f, f, s); }
                }
            s = team_reduce<false>(s, team, red, row_in_cta, lane_t);
            if (OP == ROW_SUMSQ) {
                if (live && lane_t == 0) *reinterpret_cast<float*>(a.s0.base + stat_off) = s;
                advance();
                continue;
            }
            rstd = 1.0f / sqrtf(s / (float)g.n + a.eps);
        }
        if (OP == ROW_MAX || OP == ROW_SOFTMAX) {
            float mx = -INFINITY;
#pragma unroll
            for (int k = 0; k < VPT; ++k)
                if (live && colpart[k] >= 0) {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) mx = fmaxf(mx, ja_to_float(raw[k].e[e]));
                }
            m = team_reduce<true>(mx, team, red, row_in_cta, lane_t);
            if (OP == ROW_MAX) {
                if (live && lane_t == 0) *reinterpret_cast<float*>(a.s0.base + stat_off) = m;
                advance();
                continue;
            }
        }
        if (OP == ROW_EXPSUM || OP == ROW_EXP_SUB_DIV) m = live ? *reinterpret_cast<const float*>(a.s0.base + stat_off) : 0.f;
        if (OP == ROW_EXPSUM || OP == ROW_SOFTMAX) {
            float s = 0.f;
#pragma unroll
            for (int k = 0; k < VPT; ++k)
                if (live && colpart[k] >= 0) {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        const float p = __expf(ja_to_float(raw[k].e[e]) - m);
                        if (KEEP_EXP) ex[k * VEC + e] = p;
                        s += p;
                    }
                }
            l = team_reduce<false>(s, team, red, row_in_cta, lane_t);
            if (OP == ROW_EXPSUM) {
                if (live && lane_t == 0) *reinterpret_cast<float*>(a.s1.base + stat_off) = l;
                advance();
                continue;
            }
        }
        if (OP == ROW_EXP_SUB_DIV) l = live ? *reinterpret_cast<const float*>(a.s1.base + stat_off) : 1.f;
        if (OP == ROW_RMS_SCALE) {
            const float ss = live ? *reinterpret_cast<const float*>(a.s0.base + stat_off) : 1.f;
            rstd = 1.0f / sqrtf(ss / (float)g.n + a.eps);
        }
        const float inv_l = (OP == ROW_SOFTMAX || OP == ROW_EXP_SUB_DIV) ? 1.0f / l : 0.f;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            if (!(live && colpart[k] >= 0)) continue;
            V o;
            if (HAS_G) {
                const V gv = *reinterpret_cast<const V*>(a.g.base + gpart[HAS_G ? k : 0]);
#pragma unroll
                for (int e = 0; e < VEC; ++e)
                    o.e[e] = ja_from_float<T>(ja_to_float(raw[k].e[e]) * rstd * ja_to_float(gv.e[e]));
            } else if (OP == ROW_SOFTMAX) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) o.e[e] = ja_from_float<T>(ex[KEEP_EXP ? k * VEC + e : 0] * inv_l);
            } else if (OP == ROW_EXP_SUB_DIV) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) o.e[e] = ja_from_float<T>(__expf(ja_to_float(raw[k].e[e]) - m) * inv_l);
            } else if (OP == ROW_ROPE) {
                const int col = (k * team + lane_t) * VEC;
                const float2* tab = a.rope_table + (pos * g.rope_d + (col % g.rope_d)) / 2;
#pragma unroll
                for (int e = 0; e + 1 < VEC; e += 2) {
                    const float2 cs = tab[e / 2];
                    const float x0 = ja_to_float(raw[k].e[e]), x1 = ja_to_float(raw[k].e[e + 1]);
                    o.e[e] = ja_from_float<T>(x0 * cs.x - x1 * cs.y);
                    o.e[e + 1] = ja_from_float<T>(x0 * cs.y + x1 * cs.x);
                }
            }
            *reinterpret_cast<V*>(yrow + colpart[k]) = o;
        }
        advance();
    }
}

template <typename T, int VEC, int VPT, int OP>
void launch_fast_v(const RowArgs& a, const FastGeom& g, int64_t n_rows, int team, cudaStream_t st) {
    // a CTA is one team when rows need several warps (its barrier then couples only the warps of one row), and four
    // independent single-warp teams otherwise
    const int block = team >= 64 ? team : 128;
    const int rpc = block / team;
    int64_t want = (n_rows + rpc - 1) / rpc;
    // persistent: exactly as many CTAs as are resident at once
    static int resident = 0;   // per template instance
    if (resident == 0) {
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, row_fast_kernel<T, VEC, VPT, OP>, block, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
        resident = per_sm * ja_sm_count();
    }
    unsigned grid = (unsigned)(want < resident ? want : resident);
    row_fast_kernel<T, VEC, VPT, OP><<<grid, block, 0, st>>>(a, g, n_rows, team);
}

// returns false if the shape does not fit the fast path (caller falls back to the generic kernel)
template <typename T, int OP>
bool launch_fast(const RowArgs& a, const FastGeom& g, int64_t n_rows, cudaStream_t st) {
    constexpr int VEC = 16 / (int)sizeof(T);
    // few vectors per thread (two register sets: the row being processed and the prefetched next row);
    // rows longer than one warp's share take 2, 4 or 8 warps
    // measured on B200: maps that write a row back run best with 2 vectors per thread, pure reductions with 4
    constexpr bool REDUCE_ONLY = (OP == ROW_SUMSQ || OP == ROW_MAX || OP == ROW_EXPSUM);
    int team = 32;
    while (team < 256 && g.n > team * VEC * (REDUCE_ONLY ? 4 : 2)) team *= 2;
    { const int t = ja_config().row_team; if (t >= 32 && t <= 256 && (t & (t - 1)) == 0) team = t; }
    const int vpt = (g.n + team * VEC - 1) / (team * VEC);
    if (vpt <= 1) launch_fast_v<T, VEC, 1, OP>(a, g, n_rows, team, st);
    else if (vpt <= 2) launch_fast_v<T, VEC, 2, OP>(a, g, n_rows, team, st);
    else if (vpt <= 4) launch_fast_v<T, VEC, 4, OP>(a, g, n_rows, team, st);
    else if (vpt <= 8) launch_fast_v<T, VEC, 8, OP>(a, g, n_rows, team, st);
    else if (vpt <= 16) launch_fast_v<T, VEC, 16, OP>(a, g, n_rows, team, st);
    else return false;
    return true;
}

template <typename T>
bool launch_fast_op(RowOp op, const RowArgs& a, const FastGeom& g, int64_t n_rows, cudaStream_t st) {
    switch (op) {
        case ROW_SUMSQ: return launch_fast<T, ROW_SUMSQ>(a, g, n_rows, st);
        case ROW_MAX: return launch_fast<T, ROW_MAX>(a, g, n_rows, st);
        case ROW_EXPSUM: return launch_fast<T, ROW_EXPSUM>(a, g, n_rows, st);
        case ROW_RMS_SCALE: return launch_fast<T, ROW_RMS_SCALE>(a, g, n_rows, st);
        case ROW_EXP_SUB_DIV: return launch_fast<T, ROW_EXP_SUB_DIV>(a, g, n_rows, st);
        case ROW_RMSNORM: return launch_fast<T, ROW_RMSNORM>(a, g, n_rows, st);
        case ROW_SOFTMAX: return launch_fast<T, ROW_SOFTMAX>(a, g, n_rows, st);
        case ROW_ROPE: return launch_fast<T, ROW_ROPE>(a, g, n_rows, st);
    }
    return false;
}

template <typename T, int VEC, int OP>
ja_status_t launch_row_t(const RowArgs& a, int64_t n_rows, int64_t n, cudaStream_t st) {
    // team: the smallest power of two (32..256) that keeps at most 4 vectors per thread (few registers, many
    // resident warps), else up to 16 vectors at 256 threads, else stream
    int team = 32;
    while (team < 256 && n > (int64_t)team * VEC * 4) team *= 2;
    int64_t vpt = (n + (int64_t)team * VEC - 1) / ((int64_t)team * VEC);
    const int rpc = 256 / team;
    unsigned grid = (unsigned)((n_rows + rpc - 1) / rpc);
    if (vpt <= 1) row_kernel<T, VEC, 1, OP><<<grid, 256, 0, st>>>(a, n_rows, team);
    else if (vpt <= 2) row_kernel<T, VEC, 2, OP><<<grid, 256, 0, st>>>(a, n_rows, team);
    else if (vpt <= 4) row_kernel<T, VEC, 4, OP><<<grid, 256, 0, st>>>(a, n_rows, team);
    else if (vpt <= 8) row_kernel<T, VEC, 8, OP><<<grid, 256, 0, st>>>(a, n_rows, team);
    else if (vpt <= 16 && VEC > 1) row_kernel<T, VEC, 16, OP><<<grid, 256, 0, st>>>(a, n_rows, team);
    else row_kernel<T, VEC, 0, OP><<<grid, 256, 0, st>>>(a, n_rows, team);
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}

template <typename T, int OP>
ja_status_t launch_row_vec(const RowArgs& a, int vec, int64_t n_rows, int64_t n, cudaStream_t st) {
    constexpr int FULL = 16 / (int)sizeof(T);
    if (vec == FULL) return launch_row_t<T, FULL, OP>(a, n_rows, n, st);
    if (vec == 2) return launch_row_t<T, 2, OP>(a, n_rows, n, st);
    return launch_row_t<T, 1, OP>(a, n_rows, n, st);
}

template <typename T>
ja_status_t launch_row_op(RowOp op, const RowArgs& a, int vec, int64_t n_rows, int64_t n, cudaStream_t st) {
    switch (op) {
        case ROW_SUMSQ: return launch_row_vec<T, ROW_SUMSQ>(a, vec, n_rows, n, st);
        case ROW_MAX: return launch_row_vec<T, ROW_MAX>(a, vec, n_rows, n, st);
        case ROW_EXPSUM: return launch_row_vec<T, ROW_EXPSUM>(a, vec, n_rows, n, st);
        case ROW_RMS_SCALE: return launch_row_vec<T, ROW_RMS_SCALE>(a, vec, n_rows, n, st);
        case ROW_EXP_SUB_DIV: return launch_row_vec<T, ROW_EXP_SUB_DIV>(a, vec, n_rows, n, st);
        case ROW_RMSNORM: return launch_row_vec<T, ROW_RMSNORM>(a, vec, n_rows, n, st);
        case ROW_SOFTMAX: return launch_row_vec<T, ROW_SOFTMAX>(a, vec, n_rows, n, st);
        case ROW_ROPE: return launch_row_vec<T, ROW_ROPE>(a, vec, n_rows, n, st);
    }
    return ja_fail(JA_ERR_INVALID_ARG, "unknown row op");
}

template <typename T>
ja_status_t launch_row_typed(RowOp op, const RowArgs& a, cudaStream_t st) {
    const ja_dtype_t dt = JaDtypeOf<T>::value;
    const int last = a.x.rank - 1;
    const int64_t n = a.x.extent[last];
    int64_t n_rows = 1;
    for (int d = 0; d < last; ++d) n_rows *= a.x.extent[d];
    if (n_rows >= (1ll << 31) || n >= (1ll << 31)) return ja_fail(JA_ERR_UNSUPPORTED, "row-structured join-agg: extents must be < 2^31");
    const int full = dt == JA_F32 ? 4 : 8;
    const int es = dt == JA_F32 ? 4 : 2;
    // ---- fast path: every block of x (and of g, and of the statistics relations) has the same shape --------
    const bool has_g = (op == ROW_RMS_SCALE || op == ROW_RMSNORM);
    const bool has_stat = (op == ROW_SUMSQ || op == ROW_MAX || op == ROW_EXPSUM || op == ROW_RMS_SCALE || op == ROW_EXP_SUB_DIV);
    const bool has_y = !(op == ROW_SUMSQ || op == ROW_MAX || op == ROW_EXPSUM);
    if (a.x.blk_stride != 0 && a.x.bs[last] % full == 0 && (!has_y || a.y.blk_stride == a.x.blk_stride) &&
        (!has_g || a.g.blk_stride != 0) && (!has_stat || a.s0.blk_stride != 0) &&
        (int64_t)a.x.nblk[last] * (a.x.blk_stride / es) < (1ll << 31)) {
        FastGeom g;
        memset(&g, 0, sizeof g);
        g.n = (int)n; g.bsc = (int)a.x.bs[last]; g.nbc = a.x.nblk[last];
        g.blk_elems = (int)(a.x.blk_stride / es);
        g.lead_rank = last;
        for (int d = 0; d < last; ++d) { g.lead_ext[d] = (int)a.x.extent[d]; g.lead_bs[d] = (int)a.x.bs[d]; g.lead_nb[d] = a.x.nblk[d]; }
        g.stat_blk_bytes = has_stat ? (int)a.s0.blk_stride : 0;
        g.g_blk_bytes = has_g ? (int)a.g.blk_stride : 0;
        g.rope_d = a.rope_d > 0 ? a.rope_d : 2;
        bool ok = launch_fast_op<T>(op, a, g, n_rows, st);
        if (ok) {
            ja_count_launch();
            JA_CUDA(cudaGetLastError());
            return JA_OK;
        }
    }
    // ---- generic path: any tiling, key tables read on the device ----------------------------------------------
    int vec = 1;
    if (a.x.bs[last] != 0 && a.x.bs[last] % full == 0 && n % full == 0) vec = full;
    else if (op == ROW_ROPE) vec = 2;
    return launch_row_op<T>(op, a, vec, n_rows, n, st);
}

}  // namespace
