// Row statistics as join-aggs whose output is only the statistic: "Rj->R" SQUARE / SUM (sum of squares), IDENT / MAX
// (row maximum) and "Rj,R->R" EXP_SUB / SUM (sum of exp(x - m)). The function specs of one output key are the column
// blocks of one row; nothing is written but one f32 per row, so the kernel is a pure read stream: no staging through
// shared memory, no barrier, one warp per row with the loads of a chunk (eight 16-byte vectors per lane) in flight before
// the first use, four CTAs of eight warps per SM. Relations with uniform blocks whose width is a whole number of 16-byte
// vectors. The partial sums of a row are combined in a fixed order (lane-wise over ascending columns, then the
// butterfly over lanes), so a launch is deterministic.
// HBM-bound: n cells read per row. Where it is used (L2 flushed before every launch, against the bulk-copy pipelined
// kernel of k_row_tma_impl.cuh on the same inputs): sum of squares of 8192 x 4096 bf16 (67 MB) 16.7 us against 18.6 --
// a launch that short is mostly ramp, and this form has nothing to set up; row maximum and sum of exponentials of
// 32 x 2048 x 2048 (268 MB) 49.9 / 66.2 us against 47.3 / 65.3, so those two stay with the pipelined kernel unless the
// switch "row_reduce" is 1. Both forms read at most ~5.5 TB/s (what the register file or the stages can keep in flight),
// and the sum of exponentials pays about half of its special-function time on top in either form. Measured and not kept:
// issuing the loads of the next chunk before reducing this one (two buffers in registers halve what is in flight: 17.4 /
// 51.4 / 71.9 us), sixteen vectors per lane (occupancy halves: 20.5 / 72.9 / 92.7), and asking for the warp's next row
// with one bulk L2 prefetch per column block (21.3 / 69.7 / 88.2: the prefetches queue in front of the loads); a quarter or
// half of the exponentials as a degree-5 polynomial on the FMA pipe instead of ex2.approx (73.8 / 83.5 us against 66.2: what
// the sum of exponentials pays on top of the row maximum is instruction issue, not the special-function unit); the scale,
// the subtraction and the two running sums as packed f32x2 instructions (64.4 us against 66.2, sum of squares unchanged: not
// worth a second code path).
#include <stdlib.h>
#include <string.h>

#include "ja_device.cuh"

namespace {

struct ReduceGeom {
    int n, bsc, nbc;            // row length, column-block width, column blocks (cells)
    int64_t blk_elems;          // cells between consecutive blocks (equal shapes, padding included)
    int lead_rank;              // leading (row) dimensions, 1..3
    int lead_ext[3], lead_bs[3], lead_nb[3];
    int stat_blk_bytes;         // bytes between consecutive blocks of the statistics relations
    int64_t n_rows;
};

template <typename T> struct Cells;
template <> struct Cells<float> {
    static constexpr int VEC = 4;
    static __device__ __forceinline__ void widen(const uint4& v, float (&f)[4]) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
};
template <> struct Cells<__nv_bfloat16> {
    static constexpr int VEC = 8;
    static __device__ __forceinline__ void widen(const uint4& v, float (&f)[8]) {   // bf16 -> f32 is a shift or a mask
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            f[2 * e] = __uint_as_float(w[e] << 16);
            f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
        }
    }
};
template <> struct Cells<__half> {
    static constexpr int VEC = 8;
    static __device__ __forceinline__ void widen(const uint4& v, float (&f)[8]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 t = ja_unpack16<true>(w[e]);
            f[2 * e] = t.x;
            f[2 * e + 1] = t.y;
        }
    }
};

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <typename T, int OP>
__global__ void __launch_bounds__(256) row_reduce_kernel(const char* __restrict__ x, const char* __restrict__ s_in,
                                                         char* __restrict__ s_out, const ReduceGeom g) {
    constexpr int VEC = Cells<T>::VEC;
    constexpr bool IS_MAX = OP == ROW_MAX;
    constexpr int UNROLL = 8;                                // 16-byte loads in flight per lane
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int nvec = g.n / VEC;                              // 16-byte vectors per row
    const int64_t strip = (int64_t)g.nbc * g.blk_elems;      // cells in one strip of column blocks
    // first cell of a row and the byte offset of its statistic (row-major over the leading indices)
    auto locate = [&](int64_t row, int64_t* stat_off) -> const T* {
        uint32_t rem = (uint32_t)row;
        int c[3] = {0, 0, 0};
#pragma unroll
        for (int d = 2; d >= 0; --d)
            if (d < g.lead_rank) {
                const uint32_t q = rem / (uint32_t)g.lead_ext[d];
                c[d] = (int)(rem - q * (uint32_t)g.lead_ext[d]);
                rem = q;
            }
        int lead_flat = 0, lead_in = 0;
#pragma unroll
        for (int d = 0; d < 3; ++d)
            if (d < g.lead_rank) {
                const int b = (int)((uint32_t)c[d] / (uint32_t)g.lead_bs[d]);
                lead_flat = lead_flat * g.lead_nb[d] + b;
                lead_in = lead_in * g.lead_bs[d] + (c[d] - b * g.lead_bs[d]);
            }
        *stat_off = (int64_t)lead_flat * g.stat_blk_bytes + (int64_t)lead_in * 4;
        return reinterpret_cast<const T*>(x) + (int64_t)lead_flat * strip + (int64_t)lead_in * g.bsc;
    };
    int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    for (; row < g.n_rows; row += warps) {
        int64_t stat_off;
        const T* xrow = locate(row, &stat_off);
        float neg_m2 = 0.f;                                  // EXP_SUB: -m log2(e), exp(x - m) = 2^(x log2e - m log2e)
        if (OP == ROW_EXPSUM) neg_m2 = -*reinterpret_cast<const float*>(s_in + stat_off) * 1.4426950408889634f;

        float acc0 = IS_MAX ? -INFINITY : 0.f, acc1 = acc0;
        // this lane's vectors are lane, lane + 32, ...: column block and offset inside it advance by 32 vectors a step
        int cb = (lane * VEC) / g.bsc, ci = lane * VEC - cb * g.bsc;
        for (int v0 = lane; v0 < nvec; v0 += 32 * UNROLL) {
            uint4 buf[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (v0 + 32 * u < nvec) buf[u] = __ldg(reinterpret_cast<const uint4*>(xrow + (int64_t)cb * g.blk_elems + ci));
                ci += 32 * VEC;
                while (ci >= g.bsc) { ci -= g.bsc; ++cb; }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (v0 + 32 * u >= nvec) continue;
                float f[VEC];
                Cells<T>::widen(buf[u], f);
#pragma unroll
                for (int e = 0; e < VEC; e += 2) {
                    if (OP == ROW_SUMSQ) {
                        acc0 = fmaf(f[e], f[e], acc0);
                        acc1 = fmaf(f[e + 1], f[e + 1], acc1);
                    } else if (OP == ROW_MAX) {
                        acc0 = fmaxf(acc0, f[e]);
                        acc1 = fmaxf(acc1, f[e + 1]);
                    } else {
                        acc0 += ex2_approx(fmaf(f[e], 1.4426950408889634f, neg_m2));
                        acc1 += ex2_approx(fmaf(f[e + 1], 1.4426950408889634f, neg_m2));
                    }
                }
            }
        }
        float r = IS_MAX ? fmaxf(acc0, acc1) : acc0 + acc1;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float t = __shfl_xor_sync(0xffffffffu, r, o);
            r = IS_MAX ? fmaxf(r, t) : r + t;
        }
        if (lane == 0) *reinterpret_cast<float*>(s_out + stat_off) = r;
    }
}

template <typename T, int OP>
ja_status_t launch_reduce(const RowArgs& a, const ReduceGeom& g, cudaStream_t st) {
    static int per_sm = 0;   // per template instance
    if (per_sm == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, row_reduce_kernel<T, OP>, 256, 0) != cudaSuccess || n < 1) n = 1;
        per_sm = n;
    }
    const int64_t want = (g.n_rows + 7) / 8;                 // eight rows (warps) per CTA
    const int64_t resident = (int64_t)per_sm * ja_sm_count();
    const unsigned grid = (unsigned)(want < resident ? want : resident);
    const char* s_in = OP == ROW_EXPSUM ? a.s0.base : nullptr;
    char* s_out = OP == ROW_EXPSUM ? a.s1.base : a.s0.base;
    row_reduce_kernel<T, OP><<<grid, 256, 0, st>>>(a.x.base, s_in, s_out, g);
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}

template <typename T>
ja_status_t launch_reduce_op(RowOp op, const RowArgs& a, const ReduceGeom& g, cudaStream_t st) {
    switch (op) {
        case ROW_SUMSQ: return launch_reduce<T, ROW_SUMSQ>(a, g, st);
        case ROW_MAX: return launch_reduce<T, ROW_MAX>(a, g, st);
        default: return launch_reduce<T, ROW_EXPSUM>(a, g, st);
    }
}

}  // namespace

// Sets *launched when this form took the job: a statistics-only row join-agg over relations with uniform blocks of whole
// 16-byte vectors; leaves it false (and launches nothing) otherwise.
ja_status_t ja_launch_row_reduce(RowOp op, const RowArgs& a, ja_dtype_t dt, cudaStream_t st, bool* launched) {
    *launched = false;
    if (op != ROW_SUMSQ && op != ROW_MAX && op != ROW_EXPSUM) return JA_OK;
    const int sw = ja_config().row_reduce;
    if (sw == 0) return JA_OK;
    const int last = a.x.rank - 1;
    const int vec = dt == JA_F32 ? 4 : 8, es = dt == JA_F32 ? 4 : 2;
    if (last < 1 || last > 3 || a.x.blk_stride == 0 || a.s0.blk_stride == 0 || (op == ROW_EXPSUM && a.s1.blk_stride != a.s0.blk_stride))
        return JA_OK;
    if (a.x.bs[last] == 0 || a.x.bs[last] % vec != 0 || a.x.extent[last] % vec != 0 || a.x.blk_stride % 16 != 0) return JA_OK;
    int64_t n_rows = 1;
    for (int d = 0; d < last; ++d) {
        if (a.x.bs[d] == 0) return JA_OK;
        n_rows *= a.x.extent[d];
    }
    if (n_rows >= (1ll << 31) || a.x.extent[last] >= (1ll << 31)) return JA_OK;
    // by default only the sum of squares (see the measurements at the top), and only where one warp per row fills the GPU
    if (sw < 0 && (op != ROW_SUMSQ || n_rows < (int64_t)ja_sm_count() * 16)) return JA_OK;
    ReduceGeom g;
    memset(&g, 0, sizeof g);
    g.n = (int)a.x.extent[last];
    g.bsc = (int)a.x.bs[last];
    g.nbc = a.x.nblk[last];
    g.blk_elems = a.x.blk_stride / es;
    g.lead_rank = last;
    for (int d = 0; d < last; ++d) { g.lead_ext[d] = (int)a.x.extent[d]; g.lead_bs[d] = (int)a.x.bs[d]; g.lead_nb[d] = a.x.nblk[d]; }
    g.stat_blk_bytes = (int)a.s0.blk_stride;
    g.n_rows = n_rows;
    ja_status_t s = dt == JA_F32   ? launch_reduce_op<float>(op, a, g, st)
                    : dt == JA_F16 ? launch_reduce_op<__half>(op, a, g, st)
                                   : launch_reduce_op<__nv_bfloat16>(op, a, g, st);
    if (s == JA_OK) *launched = true;
    return s;
}
