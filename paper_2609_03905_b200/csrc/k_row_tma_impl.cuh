// Row-structured join-aggs ("Rj..." forms) on uniform tilings, staged through shared memory by bulk asynchronous
// copies. These operators move a few bytes per flop, so the only thing that matters is how many bytes are in flight:
// a thread that loads its cells into registers, reduces and stores keeps a few hundred bytes in flight; a ring of
// shared-memory stages filled by cp.async.bulk keeps 100-200 KiB in flight per SM with one issuing thread.
//
// A relation with uniform blocks is a rank-4 tensor (column in block, row in block, column block, strip of blocks), so
// one tiled TMA copy fetches the R rows of a work unit out of ALL the column blocks they cross (boxes are at most 256
// cells wide: a unit is bsc/bw copies in and as many out). Few, large copies matter: this part's TMA unit spends
// about 0.1 us per copy whatever its size.
//
//   warps 0..7  consumers: warp w owns rows w, w+8, ... of the stage. It walks the row's column blocks in ascending
//               order -- for the reductions (SQUARE/SUM, IDENT/MAX, EXP_SUB/SUM) that walk is the aggregation over the
//               function specs that share the row's output key -- and, for the maps, writes the result over the input
//               in shared memory.
//   warp 8      loader: one thread issues the TMA loads of a unit into a free stage (mbarrier complete_tx).
//   warp 9      storer (maps only): when the eight consumer warps are done with a stage, one thread issues the TMA
//               stores of the stage and frees it once the copies have read shared memory.
// Every mbarrier wait is bounded; on expiry the CTA records JA_ERR_TIMEOUT, waits (bounded) for its loads in flight
// and leaves through the normal exit.
#pragma once

#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <type_traits>

#include "ja_device.cuh"
#include "ja_ptx.cuh"

namespace {

using namespace ja_ptx;

constexpr int CONSUMER_WARPS = 8;
constexpr int NUM_THREADS = (CONSUMER_WARPS + 2) * 32;
constexpr int MAX_STAGES = 6;

struct RowTmaGeom {
    int n, bsc, nbc;             // row length, column-block width, column blocks (cells)
    int rows_per_blk;            // rows (flattened leading coordinates) inside one block
    int chunks_per_blk;          // work units per strip of nbc blocks
    int R;                       // rows per unit (the last unit of a block may hold fewer)
    int stages;
    int wpr;                     // consumer warps per row (1, 2, 4 or 8); R * wpr >= 8 whenever wpr > 1
    int64_t n_units;
    int64_t blk_bytes;           // bytes between consecutive blocks of x / y
    int bw, nh;                  // TMA box width in cells (divides bsc, at most 256) and boxes per unit: bsc / bw
    int seg_bytes;               // shared-memory bytes of one column block inside a box: R * bw * sizeof(T)
    int half_bytes;              // one box: nbc * seg_bytes
    int stage_bytes;             // nh * half_bytes
    int stat_blk_bytes;          // bytes between consecutive blocks of a statistics relation
    int g_blk_bytes;             // bytes between consecutive blocks of the gain vector
    float eps;
    uint32_t wait_cap_us;        // limit of every bounded wait
};

__device__ __forceinline__ void tma_store_4d(const CUtensorMap* tm, uint32_t src, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(tm), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <typename T, int VEC> struct alignas(sizeof(T) * VEC) RVec { T e[VEC]; };

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// A row is owned by a team of wpr warps (1, 2, 4 or 8): long rows are split so that all eight consumer warps work on the
// few rows a stage can hold. A team reduction is a warp reduction, one partial per warp in shared memory, an mbarrier
// (bounded wait) and a sum / max over the partials in a fixed order, so every warp of the team gets the same bits.
struct Team {
    int wpr, sub;            // warps per row; this warp's index inside its team
    float* red;              // [2][8] partials of this team (two buffers: consecutive reductions alternate)
    uint32_t bar;            // the team's mbarrier (count wpr)
    uint32_t count;          // reductions done so far by this warp
    volatile int* abort_flag;
    int32_t* status;
    bool ok;
};

template <bool IS_MAX>
__device__ __forceinline__ float team_reduce(Team& t, float v, int lane) {
    v = IS_MAX ? warp_max(v) : warp_sum(v);
    if (t.wpr == 1) return v;
    float* buf = t.red + (t.count & 1) * 8;
    if (lane == 0) {
        buf[t.sub] = v;
        mbar_arrive(t.bar);
    }
    if (!mbar_wait(t.bar, t.count & 1, t.abort_flag, t.status)) t.ok = false;
    ++t.count;
    float r = buf[0];
    for (int i = 1; i < t.wpr; ++i) r = IS_MAX ? fmaxf(r, buf[i]) : r + buf[i];
    return r;
}

// ---- one row, any cell type: plain scalar arithmetic --------------------------------------------------------
template <typename T, int OP, int VPL>
__device__ __forceinline__ void row_generic(const RowArgs& a, const RowTmaGeom& g, uint8_t* rowp, const int (&off)[VPL],
                                            const uint8_t* g_s, int64_t stat_off, float pre0, float pre1, int lane, Team& team) {
    constexpr int VEC = 16 / (int)sizeof(T);
    using V = RVec<T, VEC>;
    constexpr bool HAS_G = (OP == ROW_RMS_SCALE || OP == ROW_RMSNORM);
    constexpr bool HAS_Y = !(OP == ROW_SUMSQ || OP == ROW_MAX || OP == ROW_EXPSUM);
    constexpr bool KEEP_EXP = (OP == ROW_SOFTMAX);
    float m = 0.f, l = 0.f, rstd = 0.f;
    float ex[KEEP_EXP ? VPL * VEC : 1];
    if (OP == ROW_SUMSQ || OP == ROW_RMSNORM) {
        float sacc = 0.f;
#pragma unroll
        for (int k = 0; k < VPL; ++k)
            if (off[k] >= 0) {
                const V v = *reinterpret_cast<const V*>(rowp + off[k]);
#pragma unroll
                for (int e = 0; e < VEC; ++e) { const float f = ja_to_float(v.e[e]); sacc = fmaf(f, f, sacc); }
            }
        sacc = team_reduce<false>(team, sacc, lane);
        if (OP == ROW_SUMSQ) {
            if (lane == 0 && team.sub == 0) *reinterpret_cast<float*>(a.s0.base + stat_off) = sacc;
            return;
        }
        rstd = 1.0f / sqrtf(sacc / (float)g.n + g.eps);
    }
    if (OP == ROW_MAX || OP == ROW_SOFTMAX) {
        float mx = -INFINITY;
#pragma unroll
        for (int k = 0; k < VPL; ++k)
            if (off[k] >= 0) {
                const V v = *reinterpret_cast<const V*>(rowp + off[k]);
#pragma unroll
                for (int e = 0; e < VEC; ++e) mx = fmaxf(mx, ja_to_float(v.e[e]));
            }
        m = team_reduce<true>(team, mx, lane);
        if (OP == ROW_MAX) {
            if (lane == 0 && team.sub == 0) *reinterpret_cast<float*>(a.s0.base + stat_off) = m;
            return;
        }
    }
    if (OP == ROW_EXPSUM || OP == ROW_EXP_SUB_DIV) m = pre0;
    if (OP == ROW_EXPSUM || OP == ROW_SOFTMAX) {
        float sacc = 0.f;
#pragma unroll
        for (int k = 0; k < VPL; ++k)
            if (off[k] >= 0) {
                const V v = *reinterpret_cast<const V*>(rowp + off[k]);
#pragma unroll
                for (int e = 0; e < VEC; ++e) {
                    const float p = __expf(ja_to_float(v.e[e]) - m);
                    if (KEEP_EXP) ex[k * VEC + e] = p;
                    sacc += p;
                }
            }
        l = team_reduce<false>(team, sacc, lane);
        if (OP == ROW_EXPSUM) {
            if (lane == 0 && team.sub == 0) *reinterpret_cast<float*>(a.s1.base + stat_off) = l;
            return;
        }
    }
    if (OP == ROW_EXP_SUB_DIV) l = pre1;
    if (OP == ROW_RMS_SCALE) {
        const float ss = pre0;
        rstd = 1.0f / sqrtf(ss / (float)g.n + g.eps);
    }
    const float inv_l = (OP == ROW_SOFTMAX || OP == ROW_EXP_SUB_DIV) ? 1.0f / l : 0.f;
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        if (off[k] < 0) continue;
        V o;
        if (HAS_G) {
            const V v = *reinterpret_cast<const V*>(rowp + off[k]);
            const V gv = *reinterpret_cast<const V*>(g_s + (size_t)((k * team.wpr + team.sub) * 32 + lane) * 16);
#pragma unroll
            for (int e = 0; e < VEC; ++e) o.e[e] = ja_from_float<T>(ja_to_float(v.e[e]) * rstd * ja_to_float(gv.e[e]));
        } else if (OP == ROW_SOFTMAX) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) o.e[e] = ja_from_float<T>(ex[KEEP_EXP ? k * VEC + e : 0] * inv_l);
        } else if (OP == ROW_EXP_SUB_DIV) {
            const V v = *reinterpret_cast<const V*>(rowp + off[k]);
#pragma unroll
            for (int e = 0; e < VEC; ++e) o.e[e] = ja_from_float<T>(__expf(ja_to_float(v.e[e]) - m) * inv_l);
        }
        if (HAS_Y) *reinterpret_cast<V*>(rowp + off[k]) = o;
    }
}

// ---- one row of bf16 cells: the same arithmetic with few instructions per cell -----------------------------------
// bf16 -> f32 is a shift or a mask; MAX runs on packed bf16 pairs (exact); products, sums and the exponent argument
// run on packed f32 pairs. exp(x - m) is ex2(x log2e - m log2e), one multiply-add and one special-function op.
__device__ __forceinline__ uint64_t pk2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void upk2(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t x, uint64_t y, uint64_t z) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(x), "l"(y), "l"(z));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t x, uint64_t y) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(x), "l"(y));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t x, uint64_t y) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(x), "l"(y));
    return d;
}
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint64_t widen(uint32_t w) { return pk2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u)); }
__device__ __forceinline__ uint32_t narrow(uint64_t v) {   // two f32 -> packed bf16, round to nearest even
    float lo, hi;
    upk2(v, lo, hi);
    const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&t);
}

// FULL: every lane owns VPL valid vectors of the row (the row length is exactly VPL * warps-per-row * 32 vectors), so the walk
// over them is straight-line code that the compiler can interleave; otherwise each vector is guarded.
template <int OP, int VPL, bool FULL>
__device__ __forceinline__ void row_bf16(const RowArgs& a, const RowTmaGeom& g, uint8_t* rowp, const int (&off)[VPL], const uint8_t* g_s,
                                         int64_t stat_off, float pre0, float pre1, int lane, Team& team) {
    constexpr bool HAS_G = (OP == ROW_RMS_SCALE || OP == ROW_RMSNORM);
    constexpr bool KEEP_EXP = (OP == ROW_SOFTMAX);
    constexpr float LOG2E = 1.4426950408889634f;
    float m = 0.f, l = 0.f, rstd = 0.f;
    uint64_t ex[KEEP_EXP ? VPL * 4 : 1];
    if (OP == ROW_SUMSQ || OP == ROW_RMSNORM) {
        uint64_t acc0 = pk2(0.f, 0.f), acc1 = pk2(0.f, 0.f);
#pragma unroll
        for (int k = 0; k < VPL; ++k)
            if (FULL || off[k] >= 0) {
                const uint4 v = *reinterpret_cast<const uint4*>(rowp + off[k]);
                const uint64_t f0 = widen(v.x), f1 = widen(v.y), f2 = widen(v.z), f3 = widen(v.w);
                acc0 = fma2(f0, f0, acc0);
                acc1 = fma2(f1, f1, acc1);
                acc0 = fma2(f2, f2, acc0);
                acc1 = fma2(f3, f3, acc1);
            }
        float s0, s1, s2, s3;
        upk2(acc0, s0, s1);
        upk2(acc1, s2, s3);
        const float sacc = team_reduce<false>(team, (s0 + s1) + (s2 + s3), lane);
        if (OP == ROW_SUMSQ) {
            if (lane == 0 && team.sub == 0) *reinterpret_cast<float*>(a.s0.base + stat_off) = sacc;
            return;
        }
        rstd = 1.0f / sqrtf(sacc / (float)g.n + g.eps);
    }
    if (OP == ROW_MAX || OP == ROW_SOFTMAX) {
        __nv_bfloat162 mx = __float2bfloat162_rn(-INFINITY);
#pragma unroll
        for (int k = 0; k < VPL; ++k)
            if (FULL || off[k] >= 0) {
                const uint4 v = *reinterpret_cast<const uint4*>(rowp + off[k]);
                const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
                mx = __hmax2(__hmax2(mx, h[0]), __hmax2(h[1], __hmax2(h[2], h[3])));
            }
        const float2 mf = __bfloat1622float2(mx);
        m = team_reduce<true>(team, fmaxf(mf.x, mf.y), lane);
        if (OP == ROW_MAX) {
            if (lane == 0 && team.sub == 0) *reinterpret_cast<float*>(a.s0.base + stat_off) = m;
            return;
        }
    }
    if (OP == ROW_EXPSUM || OP == ROW_EXP_SUB_DIV) m = pre0;
    const uint64_t sc2 = pk2(LOG2E, LOG2E), nm2 = pk2(-m * LOG2E, -m * LOG2E);
    auto exp_pair = [&](uint32_t w) {
        float t0, t1;
        upk2(fma2(widen(w), sc2, nm2), t0, t1);
        return pk2(ex2f(t0), ex2f(t1));
    };
    if (OP == ROW_EXPSUM || OP == ROW_SOFTMAX) {
        uint64_t acc0 = pk2(0.f, 0.f), acc1 = pk2(0.f, 0.f);
#pragma unroll
        for (int k = 0; k < VPL; ++k)
            if (FULL || off[k] >= 0) {
                const uint4 v = *reinterpret_cast<const uint4*>(rowp + off[k]);
                const uint64_t e0 = exp_pair(v.x), e1 = exp_pair(v.y), e2 = exp_pair(v.z), e3 = exp_pair(v.w);
                if (KEEP_EXP) { ex[k * 4] = e0; ex[k * 4 + 1] = e1; ex[k * 4 + 2] = e2; ex[k * 4 + 3] = e3; }
                acc0 = add2(acc0, e0);
                acc1 = add2(acc1, e1);
                acc0 = add2(acc0, e2);
                acc1 = add2(acc1, e3);
            }
        float s0, s1, s2, s3;
        upk2(acc0, s0, s1);
        upk2(acc1, s2, s3);
        l = team_reduce<false>(team, (s0 + s1) + (s2 + s3), lane);
        if (OP == ROW_EXPSUM) {
            if (lane == 0 && team.sub == 0) *reinterpret_cast<float*>(a.s1.base + stat_off) = l;
            return;
        }
    }
    if (OP == ROW_EXP_SUB_DIV) l = pre1;
    if (OP == ROW_RMS_SCALE) {
        const float ss = pre0;
        rstd = 1.0f / sqrtf(ss / (float)g.n + g.eps);
    }
    const float scale = (OP == ROW_SOFTMAX || OP == ROW_EXP_SUB_DIV) ? 1.0f / l : rstd;
    const uint64_t scale2 = pk2(scale, scale);
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        if (!FULL && off[k] < 0) continue;
        uint4 o;
        if (HAS_G) {
            const uint4 v = *reinterpret_cast<const uint4*>(rowp + off[k]);
            const uint4 gv = *reinterpret_cast<const uint4*>(g_s + (size_t)((k * team.wpr + team.sub) * 32 + lane) * 16);
            o.x = narrow(mul2(mul2(widen(v.x), scale2), widen(gv.x)));
            o.y = narrow(mul2(mul2(widen(v.y), scale2), widen(gv.y)));
            o.z = narrow(mul2(mul2(widen(v.z), scale2), widen(gv.z)));
            o.w = narrow(mul2(mul2(widen(v.w), scale2), widen(gv.w)));
        } else if (OP == ROW_SOFTMAX) {
            o.x = narrow(mul2(ex[KEEP_EXP ? k * 4 : 0], scale2));
            o.y = narrow(mul2(ex[KEEP_EXP ? k * 4 + 1 : 0], scale2));
            o.z = narrow(mul2(ex[KEEP_EXP ? k * 4 + 2 : 0], scale2));
            o.w = narrow(mul2(ex[KEEP_EXP ? k * 4 + 3 : 0], scale2));
        } else {   // ROW_EXP_SUB_DIV
            const uint4 v = *reinterpret_cast<const uint4*>(rowp + off[k]);
            o.x = narrow(mul2(exp_pair(v.x), scale2));
            o.y = narrow(mul2(exp_pair(v.y), scale2));
            o.z = narrow(mul2(exp_pair(v.z), scale2));
            o.w = narrow(mul2(exp_pair(v.w), scale2));
        }
        *reinterpret_cast<uint4*>(rowp + off[k]) = o;
    }
}

// VPL = 16-byte vectors per lane covering one row (lane + 32 k, k < VPL)
// CTAs per SM: two, so that sixteen consumer warps share an SM's issue slots and special-function unit; one for the
// softmax of very long rows, whose exponentials fill the register file
template <typename T, int OP, int VPL> constexpr int ctas_per_sm() { return (OP == ROW_SOFTMAX && VPL * sizeof(T) >= 32) ? 1 : 2; }

template <typename T, int OP, int VPL>
__global__ void __launch_bounds__(NUM_THREADS, (ctas_per_sm<T, OP, VPL>())) row_tma_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY, RowArgs a, RowTmaGeom g,
               int32_t* status) {
    constexpr int VEC = 16 / (int)sizeof(T);
    using V = RVec<T, VEC>;
    constexpr bool HAS_G = (OP == ROW_RMS_SCALE || OP == ROW_RMSNORM);
    constexpr bool HAS_Y = !(OP == ROW_SUMSQ || OP == ROW_MAX || OP == ROW_EXPSUM);
    extern __shared__ uint8_t smem_raw[];
    // [stages][nh][nbc][R][bw] cells, then the gain vector [n], then the barriers
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t s_stage0 = (raw + 127u) & ~127u;
    uint8_t* smem = smem_raw + (s_stage0 - raw);
    uint8_t* g_s = smem + (size_t)g.stages * g.stage_bytes;
    const size_t g_bytes = HAS_G ? ((size_t)g.n * sizeof(T) + 127) / 128 * 128 : 0;
    uint64_t* bars = reinterpret_cast<uint64_t*>(g_s + g_bytes);
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto done_bar = [&](int s) { return bar0 + 8u * (MAX_STAGES + s); };       // consumers -> storer
    auto free_bar = [&](int s) { return bar0 + 8u * (2 * MAX_STAGES + s); };   // storer (or consumers) -> loader
    auto team_bar = [&](int t) { return bar0 + 8u * (3 * MAX_STAGES + t); };
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 3 * MAX_STAGES + CONSUMER_WARPS);
    float* red_all = reinterpret_cast<float*>(bars + 3 * MAX_STAGES + CONSUMER_WARPS + 1);   // [8 teams][2][8]

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(done_bar(s), CONSUMER_WARPS);
            mbar_init(free_bar(s), HAS_Y ? 1 : CONSUMER_WARPS);
        }
        for (int t = 0; t < CONSUMER_WARPS; ++t) mbar_init(team_bar(t), (uint32_t)g.wpr);
        wait_ctl_init(abort_flag, g.wait_cap_us);   // two words: the slot is eight bytes wide
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (HAS_G && warp < CONSUMER_WARPS) {   // the gain vector, dense, once per CTA; the loader is already fetching rows meanwhile
        for (int v = threadIdx.x; v * VEC < g.n; v += CONSUMER_WARPS * 32) {
            const int col = v * VEC, cb = col / g.bsc, ci = col - cb * g.bsc;
            *reinterpret_cast<V*>(g_s + (size_t)col * sizeof(T)) =
                *reinterpret_cast<const V*>(a.g.base + (int64_t)cb * g.g_blk_bytes + (int64_t)ci * sizeof(T));
        }
        asm volatile("bar.sync 1, %0;" ::"n"(CONSUMER_WARPS * 32) : "memory");
    }

    const int64_t first = blockIdx.x, step = gridDim.x;
    const int row_seg_bytes = g.bw * (int)sizeof(T);    // bytes of one row inside one column block of a box

    // unit -> (strip of blocks, first row inside the block, rows)
    auto unit_geom = [&](int64_t u, int64_t* lb, int* r0, int* rows) {
        *lb = u / g.chunks_per_blk;
        const int ch = (int)(u - *lb * g.chunks_per_blk);
        *r0 = ch * g.R;
        *rows = min(g.R, g.rows_per_blk - *r0);
    };

    if (warp == CONSUMER_WARPS) {
        // ================= loader =================
        if (lane == 0) {
            bool ok = true;
            int64_t i = 0;
            for (int64_t u = first; u < g.n_units && ok; u += step, ++i) {
                const int s = (int)(i % g.stages);
                const uint32_t ph = (uint32_t)(i / g.stages) & 1;
                if (i >= g.stages && !mbar_wait(free_bar(s), ph ^ 1, abort_flag, status)) { ok = false; break; }
                int64_t lb;
                int r0, rows;
                unit_geom(u, &lb, &r0, &rows);
                mbar_expect_tx(full_bar(s), (uint32_t)g.stage_bytes);   // whole boxes: rows past the block's end arrive as zeros
                const uint32_t dst = s_stage0 + (uint32_t)s * g.stage_bytes;
                for (int h = 0; h < g.nh; ++h) tma_load_4d<1>(dst + h * g.half_bytes, &tmX, full_bar(s), h * g.bw, r0, 0, (int)lb);
            }
            if (!ok) {   // loads already issued still write shared memory: wait (bounded) for them before leaving
                for (int64_t j = i > g.stages ? i - g.stages : 0; j < i; ++j) {
                    const uint64_t t0 = global_ns();
                    while (!mbar_try_wait(full_bar((int)(j % g.stages)), (uint32_t)(j / g.stages) & 1) && global_ns() - t0 < 200000000ull) {}
                }
            }
        }
    } else if (warp == CONSUMER_WARPS + 1) {
        // ================= storer =================
        if (HAS_Y && lane == 0) {
            bool ok = true;
            int64_t i = 0;
            for (int64_t u = first; u < g.n_units && ok; u += step, ++i) {
                const int s = (int)(i % g.stages);
                const uint32_t ph = (uint32_t)(i / g.stages) & 1;
                if (!mbar_wait(done_bar(s), ph, abort_flag, status)) { ok = false; break; }
                int64_t lb;
                int r0, rows;
                unit_geom(u, &lb, &r0, &rows);
                const uint32_t src = s_stage0 + (uint32_t)s * g.stage_bytes;
                for (int h = 0; h < g.nh; ++h) tma_store_4d(&tmY, src + h * g.half_bytes, h * g.bw, r0, 0, (int)lb);   // rows past the block's end are clipped
                bulk_commit();
                bulk_wait_read0();                 // the copies have read the stage: it may be refilled
                mbar_arrive(free_bar(s));
            }
            bulk_wait0();
        }
    } else {
        // ================= consumers =================
        int off[VPL];   // byte offset of this lane's k-th vector inside a row of the stage (column block + column), or -1
        const bool full_rows = (int64_t)VPL * g.wpr * 32 * VEC == (int64_t)g.n;   // no lane has a vector past the end of the row
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            const int col = ((k * g.wpr + warp % g.wpr) * 32 + lane) * VEC;
            off[k] = -1;
            if (col < g.n) {
                const int cb = col / g.bsc, ci = col - cb * g.bsc, h = ci / g.bw;
                off[k] = h * g.half_bytes + cb * g.seg_bytes + (ci - h * g.bw) * (int)sizeof(T);
            }
        }
        Team team;
        team.wpr = g.wpr;
        team.sub = warp % g.wpr;
        const int tid = warp / g.wpr, n_teams = CONSUMER_WARPS / g.wpr;
        team.red = red_all + tid * 16;
        team.bar = team_bar(tid);
        team.count = 0;
        team.abort_flag = abort_flag;
        team.status = status;
        team.ok = true;
        // Input statistics of a row (m for EXP_SUB, m and l for EXP_SUB_DIV, the sum of squares for RMS_SCALE) are loaded one
        // unit AHEAD: a row's arithmetic cannot start without them, and a load issued when the row's turn comes is a cold
        // global access in front of every row. (On the 268 MB exp-SUM join-agg this measured the same as loading them in
        // place, 65 us: that kernel is bound by its warps' own dependent instruction chains -- one CTA per SM takes 94 us,
        // two 65 us, three, with two stages each instead of three, 72 us.)
        constexpr bool PRE0 = (OP == ROW_EXPSUM || OP == ROW_EXP_SUB_DIV || OP == ROW_RMS_SCALE), PRE1 = (OP == ROW_EXP_SUB_DIV);
        constexpr int MAXR = 4;   // rows of one unit that one team handles: at most 32 rows per unit over 8 teams
        float nxt0[MAXR], nxt1[MAXR];
        auto prefetch_stats = [&](int64_t u) {
#pragma unroll
            for (int q = 0; q < MAXR; ++q) { nxt0[q] = 0.f; nxt1[q] = 0.f; }
            if (!PRE0 || u >= g.n_units) return;
            int64_t lb;
            int r0, rows;
            unit_geom(u, &lb, &r0, &rows);
#pragma unroll
            for (int q = 0; q < MAXR; ++q) {
                const int r = tid + q * n_teams;
                if (r < rows) {
                    const int64_t so = lb * g.stat_blk_bytes + (int64_t)(r0 + r) * 4;
                    nxt0[q] = *reinterpret_cast<const float*>(a.s0.base + so);
                    if (PRE1) nxt1[q] = *reinterpret_cast<const float*>(a.s1.base + so);
                }
            }
        };
        prefetch_stats(first);
        int64_t i = 0;
        for (int64_t u = first; u < g.n_units && team.ok; u += step, ++i) {
            const int s = (int)(i % g.stages);
            const uint32_t ph = (uint32_t)(i / g.stages) & 1;
            float cur0[MAXR], cur1[MAXR];
#pragma unroll
            for (int q = 0; q < MAXR; ++q) { cur0[q] = nxt0[q]; cur1[q] = nxt1[q]; }
            prefetch_stats(u + step);
            if (!mbar_wait(full_bar(s), ph, abort_flag, status)) { team.ok = false; break; }
            int64_t lb;
            int r0, rows;
            unit_geom(u, &lb, &r0, &rows);
            uint8_t* stage = smem + (size_t)s * g.stage_bytes;
#pragma unroll
            for (int q = 0; q < MAXR; ++q) {
                const int r = tid + q * n_teams;
                if (r >= rows || !team.ok) break;
                uint8_t* rowp = stage + (size_t)r * row_seg_bytes;
                const int64_t stat_off = lb * g.stat_blk_bytes + (int64_t)(r0 + r) * 4;
                if constexpr (std::is_same<T, __nv_bfloat16>::value) {
                    if (full_rows) row_bf16<OP, VPL, true>(a, g, rowp, off, g_s, stat_off, cur0[q], cur1[q], lane, team);
                    else row_bf16<OP, VPL, false>(a, g, rowp, off, g_s, stat_off, cur0[q], cur1[q], lane, team);
                }
                else row_generic<T, OP, VPL>(a, g, rowp, off, g_s, stat_off, cur0[q], cur1[q], lane, team);
            }
            if (!team.ok) break;
            if (HAS_Y) fence_async_smem();    // this thread's writes to the stage become visible to the bulk stores
            __syncwarp();
            if (lane == 0) mbar_arrive(HAS_Y ? done_bar(s) : free_bar(s));
        }
    }
}

struct RowMaps { CUtensorMap x, y; };

template <typename T, int OP, int VPL>
ja_status_t launch_v(const RowMaps& tm, const RowArgs& a, RowTmaGeom g, int g_bytes, int sms, int32_t* status, cudaStream_t st,
                     bool* launched) {
    constexpr int CTAS = ctas_per_sm<T, OP, VPL>();
    const int budget = (CTAS == 2 ? 110 : 220) * 1024 - g_bytes;
    g.stages = (int)std::min<int64_t>(MAX_STAGES, budget / g.stage_bytes);
    if (g.stages < 2) { *launched = false; return JA_OK; }
    static bool configured[64] = {};   // per template instance and device
    int dev = 0;
    cudaGetDevice(&dev);
    if (!configured[dev & 63]) {
        JA_CUDA(cudaFuncSetAttribute(row_tma_kernel<T, OP, VPL>, cudaFuncAttributeMaxDynamicSharedMemorySize, 222 * 1024));
        configured[dev & 63] = true;
    }
    const int smem_bytes = g.stages * g.stage_bytes + g_bytes + (3 * MAX_STAGES + CONSUMER_WARPS + 2) * 8 + CONSUMER_WARPS * 16 * 4 + 128;
    const unsigned grid = (unsigned)std::min<int64_t>(g.n_units, (int64_t)sms * CTAS);
    row_tma_kernel<T, OP, VPL><<<grid, NUM_THREADS, smem_bytes, st>>>(tm.x, tm.y, a, g, status);
    return JA_OK;
}

template <typename T, int OP>
ja_status_t launch_op(const RowMaps& tm, const RowArgs& a, const RowTmaGeom& g, int vpl, int g_bytes, int sms, int32_t* status,
                      cudaStream_t st, bool* launched) {
    *launched = true;
    if (vpl <= 1) return launch_v<T, OP, 1>(tm, a, g, g_bytes, sms, status, st, launched);
    if (vpl <= 2) return launch_v<T, OP, 2>(tm, a, g, g_bytes, sms, status, st, launched);
    if (vpl <= 4) return launch_v<T, OP, 4>(tm, a, g, g_bytes, sms, status, st, launched);
    if (vpl <= 8) return launch_v<T, OP, 8>(tm, a, g, g_bytes, sms, status, st, launched);
    if (vpl <= 16) return launch_v<T, OP, 16>(tm, a, g, g_bytes, sms, status, st, launched);
    *launched = false;
    return JA_OK;
}

template <typename T>
ja_status_t launch_t(RowOp op, const RowMaps& tm, const RowArgs& a, const RowTmaGeom& g, int vpl, int g_bytes, int sms,
                     int32_t* status, cudaStream_t st, bool* launched) {
    switch (op) {
        case ROW_SUMSQ: return launch_op<T, ROW_SUMSQ>(tm, a, g, vpl, g_bytes, sms, status, st, launched);
        case ROW_MAX: return launch_op<T, ROW_MAX>(tm, a, g, vpl, g_bytes, sms, status, st, launched);
        case ROW_EXPSUM: return launch_op<T, ROW_EXPSUM>(tm, a, g, vpl, g_bytes, sms, status, st, launched);
        case ROW_RMS_SCALE: return launch_op<T, ROW_RMS_SCALE>(tm, a, g, vpl, g_bytes, sms, status, st, launched);
        case ROW_EXP_SUB_DIV: return launch_op<T, ROW_EXP_SUB_DIV>(tm, a, g, vpl, g_bytes, sms, status, st, launched);
        case ROW_RMSNORM: return launch_op<T, ROW_RMSNORM>(tm, a, g, vpl, g_bytes, sms, status, st, launched);
        case ROW_SOFTMAX: return launch_op<T, ROW_SOFTMAX>(tm, a, g, vpl, g_bytes, sms, status, st, launched);
        default: break;
    }
    *launched = false;
    return JA_OK;
}

// x / y with uniform blocks as the rank-4 tensor (column in block, row in block, column block, strip), box (bw, R, nbc, 1)
ja_status_t encode_rows4(const RelView& v, const RowTmaGeom& g, int64_t n_lead, ja_dtype_t dt, CUtensorMap* tm) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return ja_fail(JA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const int es = dt == JA_F32 ? 4 : 2;
    cuuint64_t dims[4] = {(cuuint64_t)g.bsc, (cuuint64_t)g.rows_per_blk, (cuuint64_t)g.nbc, (cuuint64_t)n_lead};
    cuuint64_t strides[3] = {(cuuint64_t)g.bsc * es, (cuuint64_t)g.blk_bytes, (cuuint64_t)g.blk_bytes * g.nbc};
    cuuint32_t box[4] = {(cuuint32_t)g.bw, (cuuint32_t)g.R, (cuuint32_t)g.nbc, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUtensorMapDataType cell = dt == JA_F32   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                     : dt == JA_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                                    : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    CUresult res = enc(tm, cell, 4, v.base, dims, strides, box,
                       estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (res != CUDA_SUCCESS) return ja_fail(JA_ERR_CUDA, "cuTensorMapEncodeTiled (row strips) failed with code %d", (int)res);
    return JA_OK;
}

// Sets *launched when this form took the job; leaves it false (and launches nothing) when the shape does not fit:
// blocks of different shapes, rows longer than 16 vectors per lane of a warp team, column blocks that are not whole 16-byte vectors,
// more than 256 column blocks, RoPE (its rotation needs the row's coordinates).
template <typename T>
ja_status_t row_tma_launch(RowOp op, const RowArgs& a, cudaStream_t st, bool* launched) {
    const ja_dtype_t dt = JaDtypeOf<T>::value;
    *launched = false;
    if (op == ROW_ROPE) return JA_OK;
    if (ja_config().row_tma == 0) return JA_OK;
    const int last = a.x.rank - 1;
    const int es = dt == JA_F32 ? 4 : 2, vec = 16 / es;
    const bool has_g = (op == ROW_RMS_SCALE || op == ROW_RMSNORM);
    const bool has_stat = (op == ROW_SUMSQ || op == ROW_MAX || op == ROW_EXPSUM || op == ROW_RMS_SCALE || op == ROW_EXP_SUB_DIV);
    const bool two_stats = (op == ROW_EXPSUM || op == ROW_EXP_SUB_DIV);
    const bool has_y = !(op == ROW_SUMSQ || op == ROW_MAX || op == ROW_EXPSUM);
    if (!a.x.blk_stride || a.x.bs[last] % vec != 0 || a.x.nblk[last] > 256) return JA_OK;
    if (has_y && a.y.blk_stride != a.x.blk_stride) return JA_OK;
    if (has_g && !a.g.blk_stride) return JA_OK;
    if (has_stat && !a.s0.blk_stride) return JA_OK;
    if (two_stats && a.s1.blk_stride != a.s0.blk_stride) return JA_OK;
    RowTmaGeom g;
    memset(&g, 0, sizeof g);
    const int64_t n = a.x.extent[last];
    g.n = (int)n;
    g.bsc = (int)a.x.bs[last];
    g.nbc = a.x.nblk[last];
    int64_t rows_per_blk = 1, n_lead = 1;
    for (int d = 0; d < last; ++d) { rows_per_blk *= a.x.bs[d]; n_lead *= a.x.nblk[d]; }
    if (rows_per_blk >= (1 << 30) || n >= (1 << 24) || n_lead >= ((int64_t)1 << 31)) return JA_OK;
    g.rows_per_blk = (int)rows_per_blk;
    g.blk_bytes = a.x.blk_stride;
    const int64_t row_bytes = n * es;
    if ((n + vec * 32 - 1) / (vec * 32) > 256) return JA_OK;
    // box width: the widest divisor of the column-block width that is a whole number of 128-byte lines and at most 256 cells
    g.bw = 0;
    for (int w = std::min(g.bsc, 256); w >= 128 / es; --w)
        if (g.bsc % w == 0 && (w * es) % 128 == 0) { g.bw = w; break; }
    if (!g.bw) return JA_OK;
    g.nh = g.bsc / g.bw;
    // rows per unit: the largest power of two (at most 32, at most a block holds) that keeps a stage within 32 KiB
    int R = 1;
    while (R < 32 && (int64_t)R * 2 * row_bytes <= 32 * 1024 && R * 2 <= rows_per_blk) R *= 2;
    g.R = R;
    // all eight consumer warps work: a stage of fewer than eight rows gives every row to a team of warps
    g.wpr = 1;
    while (g.wpr < CONSUMER_WARPS && R * g.wpr < CONSUMER_WARPS && n > (int64_t)g.wpr * vec * 32) g.wpr *= 2;
    const int vpl = (int)((n + (int64_t)vec * 32 * g.wpr - 1) / ((int64_t)vec * 32 * g.wpr));
    if (vpl > 16) return JA_OK;
    g.chunks_per_blk = (int)((rows_per_blk + R - 1) / R);
    g.n_units = n_lead * g.chunks_per_blk;
    g.seg_bytes = R * g.bw * es;
    g.half_bytes = g.nbc * g.seg_bytes;
    g.stage_bytes = g.nh * g.half_bytes;
    const int g_bytes = has_g ? (int)((row_bytes + 127) / 128 * 128) : 0;
    g.stat_blk_bytes = has_stat ? (int)a.s0.blk_stride : 0;
    g.g_blk_bytes = has_g ? (int)a.g.blk_stride : 0;
    g.eps = a.eps;
    g.wait_cap_us = (uint32_t)ja_config().wait_cap_us;
    int32_t* status = ja_device_status_word(st);
    if (!status) return ja_fail(JA_ERR_CUDA, "cannot resolve the device status word");
    RowMaps tm;
    ja_status_t s = encode_rows4(a.x, g, n_lead, dt, &tm.x);
    if (s != JA_OK) return s;
    tm.y = tm.x;
    if (has_y && (s = encode_rows4(a.y, g, n_lead, dt, &tm.y)) != JA_OK) return s;
    const int sms = ja_sm_count();
    s = launch_t<T>(op, tm, a, g, vpl, g_bytes, sms, status, st, launched);
    if (s != JA_OK || !*launched) return s;
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}

}  // namespace
