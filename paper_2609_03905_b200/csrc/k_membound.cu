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

template <int FN>
__global__ void __launch_bounds__(256) flat_bf16_kernel(const uint4* __restrict__ a, const uint4* __restrict__ b,
                                                        uint4* __restrict__ out, int64_t n_vec) {
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * 256) {
        uint4 va = a[i], vb = b[i], vo;
        const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&va);
        const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&vb);
        __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&vo);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float2 fa = __bfloat1622float2(pa[k]), fb = __bfloat1622float2(pb[k]);
            po[k] = __floats2bfloat162_rn(flat_fn<FN>(fa.x, fb.x), flat_fn<FN>(fa.y, fb.y));
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
    int64_t pos;        // coordinate of the second index (RoPE position)
    int64_t stat_off;   // byte offset of this row's cell in a statistics relation keyed by R
};

__device__ __forceinline__ RowCtx row_ctx(const RelView& x, const RelView& stat, bool has_stat, int64_t row) {
    RowCtx c;
    int64_t lead[JA_MAX_RANK] = {0, 0, 0, 0};
    int64_t rem = row;
    for (int d = x.rank - 2; d >= 0; --d) {
        lead[d] = rem % x.extent[d];
        rem /= x.extent[d];
    }
    c.lead_flat = 0;
    c.lead_in = 0;
    for (int d = 0; d < x.rank - 1; ++d) {
        int b = ja_find_blk(x, d, lead[d]);
        int64_t lo = x.splits[d][b], w = x.splits[d][b + 1] - lo;
        c.lead_flat = c.lead_flat * x.nblk[d] + b;
        c.lead_in = c.lead_in * w + (lead[d] - lo);
    }
    c.pos = lead[1];
    c.stat_off = has_stat ? ja_elem_off(stat, lead) : 0;
    return c;
}

// byte offset of the vector starting at column `col` of the row; also the column-block index and its lower bound
__device__ __forceinline__ int64_t vec_off(const RelView& x, const RowCtx& c, int64_t col, int* cb, int64_t* lo) {
    const int last = x.rank - 1;
    int b = ja_find_blk(x, last, col);
    int64_t l = x.splits[last][b], w = x.splits[last][b + 1] - l;
    *cb = b;
    *lo = l;
    return x.blk_off[c.lead_flat * x.nblk[last] + b] + (c.lead_in * w + (col - l)) * x.esize;
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
    const int64_t n = a.x.extent[last];
    const int64_t row = (int64_t)blockIdx.x * rpc + row_in_cta;
    const bool live = row < n_rows;
    constexpr bool HAS_STAT = (OP == ROW_SUMSQ || OP == ROW_MAX || OP == ROW_EXPSUM || OP == ROW_RMS_SCALE ||
                               OP == ROW_EXP_SUB_DIV);
    RowCtx ctx = row_ctx(a.x, a.s0, HAS_STAT, live ? row : 0);

    V raw[NV];
    int64_t offs[NV];
    // ---- pass 0: load (resident mode) -------------------------------------------------------------------
    if (RES) {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            int64_t col = ((int64_t)k * team + lane_t) * VEC;
            offs[k] = -1;
            if (live && col < n) {
                int cb; int64_t lo;
                offs[k] = vec_off(a.x, ctx, col, &cb, &lo);
                raw[k] = *reinterpret_cast<const V*>(a.x.base + offs[k]);
            }
        }
    }
    // iterate over this thread's vectors: f(k, col, byte offset, value)
    auto for_each = [&](auto f) {
        if (RES) {
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                int64_t col = ((int64_t)k * team + lane_t) * VEC;
                if (offs[k] >= 0) f(col, offs[k], raw[k]);
            }
        } else if (live) {
            for (int64_t col = (int64_t)lane_t * VEC; col < n; col += (int64_t)team * VEC) {
                int cb; int64_t lo;
                int64_t off = vec_off(a.x, ctx, col, &cb, &lo);
                V v = *reinterpret_cast<const V*>(a.x.base + off);
                f(col, off, v);
            }
        }
    };

    float m = 0.f, l = 0.f, rstd = 0.f;
    // ---- reductions ----------------------------------------------------------------------------------------
    if (OP == ROW_SUMSQ || OP == ROW_RMSNORM) {
        float s = 0.f;
        for_each([&](int64_t, int64_t, const V& v) {
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
        for_each([&](int64_t, int64_t, const V& v) {
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
        for_each([&](int64_t, int64_t, const V& v) {
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
    for_each([&](int64_t col, int64_t off, const V& v) {
        V o;
        if (OP == ROW_RMS_SCALE || OP == ROW_RMSNORM) {
            int cb = ja_find_blk(a.g, 0, col);
            int64_t goff = a.g.blk_off[cb] + (col - a.g.splits[0][cb]) * a.g.esize;
            V g = *reinterpret_cast<const V*>(a.g.base + goff);
#pragma unroll
            for (int e = 0; e < VEC; ++e) o.e[e] = ja_from_float<T>(ja_to_float(v.e[e]) * rstd * ja_to_float(g.e[e]));
        } else if (OP == ROW_SOFTMAX || OP == ROW_EXP_SUB_DIV) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) o.e[e] = ja_from_float<T>(__expf(ja_to_float(v.e[e]) - m) * inv_l);
        } else if (OP == ROW_ROPE) {
            const float2* tab = a.rope_table + ctx.pos * (n / 2) + col / 2;
#pragma unroll
            for (int e = 0; e + 1 < VEC; e += 2) {
                float2 cs = tab[e / 2];
                float x0 = ja_to_float(v.e[e]), x1 = ja_to_float(v.e[e + 1]);
                o.e[e] = ja_from_float<T>(x0 * cs.x - x1 * cs.y);
                o.e[e + 1] = ja_from_float<T>(x0 * cs.y + x1 * cs.x);
            }
        }
        *reinterpret_cast<V*>(a.y.base + off) = o;  // y is tiled exactly like x: same offset
    });
}

template <typename T, int VEC, int OP>
ja_status_t launch_row_t(const RowArgs& a, int64_t n_rows, int64_t n, cudaStream_t st) {
    // team: the smallest power of two (32..256) that keeps at most 8 vectors per thread, else 16, else stream
    int team = 32;
    while (team < 256 && n > (int64_t)team * VEC * 8) team *= 2;
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

}  // namespace

ja_status_t ja_launch_flat(ja_fn_t fn, const void* a, const void* b, void* out, int64_t n_elems, ja_dtype_t dt,
                           cudaStream_t st) {
    // payload sizes are multiples of 128 bytes, so whole 16-byte vectors cover them exactly
    const int64_t n_vec = n_elems * (dt == JA_F32 ? 4 : 2) / 16;
    int64_t want = (n_vec + 255) / 256;
    unsigned grid = (unsigned)(want < (int64_t)148 * 32 ? (want > 0 ? want : 1) : (int64_t)148 * 32);
    if (dt == JA_BF16) {
        if (fn == JA_FN_ADD) flat_bf16_kernel<JA_FN_ADD><<<grid, 256, 0, st>>>((const uint4*)a, (const uint4*)b, (uint4*)out, n_vec);
        else flat_bf16_kernel<JA_FN_SILU_MUL><<<grid, 256, 0, st>>>((const uint4*)a, (const uint4*)b, (uint4*)out, n_vec);
    } else {
        if (fn == JA_FN_ADD) flat_f32_kernel<JA_FN_ADD><<<grid, 256, 0, st>>>((const float4*)a, (const float4*)b, (float4*)out, n_vec);
        else flat_f32_kernel<JA_FN_SILU_MUL><<<grid, 256, 0, st>>>((const float4*)a, (const float4*)b, (float4*)out, n_vec);
    }
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}

ja_status_t ja_launch_row(RowOp op, const RowArgs& a, ja_dtype_t dt, cudaStream_t st) {
    const int last = a.x.rank - 1;
    const int64_t n = a.x.extent[last];
    int64_t n_rows = 1;
    for (int d = 0; d < last; ++d) n_rows *= a.x.extent[d];
    // widest vector every column split allows (the host mirrors of the split tables are not kept in the view,
    // so the caller's tiling is probed through the uniform block size when there is one)
    const int full = dt == JA_F32 ? 4 : 8;
    int vec = 1;
    if (a.x.bs[last] != 0 && a.x.bs[last] % full == 0 && n % full == 0) vec = full;
    else if (op == ROW_ROPE) vec = 2;
    return dt == JA_F32 ? launch_row_op<float>(op, a, vec, n_rows, n, st)
                        : launch_row_op<__nv_bfloat16>(op, a, vec, n_rows, n, st);
}
