// Aggregating relayout (Sections 5.1 and 5.3): a producer that was executed through its join only leaves, for every
// output block, m unaggregated copies. The consumer needs every block of ITS tiling fully aggregated. The overlay of
// the two tilings gives atoms; each atom is cut into 2-D slabs exactly as in the plain relayout, and for every cell of
// a slab the m copies are read ("decompose"), (+)-combined in ascending copy order in f32 ("aggregate") and stored
// once, rounded once, at the cell's place in the consumer's block ("recompose"). One pass, no staging buffer.
// HBM-bound: m source cells read and one destination cell written per cell.
#include "ja_device.cuh"

namespace {

template <typename T> struct VecOf;
template <> struct VecOf<float> { static constexpr int N = 4; };            // 16 bytes
template <> struct VecOf<__nv_bfloat16> { static constexpr int N = 8; };    // 16 bytes
template <> struct VecOf<__half> { static constexpr int N = 8; };
template <typename T> struct IsF16 { static constexpr bool value = false; };
template <> struct IsF16<__half> { static constexpr bool value = true; };

// the cells of one 16-byte access that is already in registers
template <typename TS> __device__ __forceinline__ void unpack_cells(const uint4& v, float* f) {
    if (sizeof(TS) == 4) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    } else {
        const uint32_t h[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 t = ja_unpack16<IsF16<TS>::value>(h[e]);
            f[2 * e] = t.x;
            f[2 * e + 1] = t.y;
        }
    }
}
// p points into GLOBAL memory (the read-only path is used)
template <typename TS, int VEC> __device__ __forceinline__ void load_cells(const char* p, float* f) {
    if (VEC == 1) {
        f[0] = ja_to_float(*reinterpret_cast<const TS*>(p));
    } else {
        unpack_cells<TS>(__ldg(reinterpret_cast<const uint4*>(p)), f);
    }
}

template <typename TD, int VEC> __device__ __forceinline__ void store_cells(char* p, const float* f) {
    if (VEC == 1) {
        *reinterpret_cast<TD*>(p) = ja_from_float<TD>(f[0]);
    } else if (sizeof(TD) == 4) {
#pragma unroll
        for (int e = 0; e < VEC; e += 4) *reinterpret_cast<float4*>(p + e * 4) = make_float4(f[e], f[e + 1], f[e + 2], f[e + 3]);
    } else if (VEC == 8) {
        uint4 o;
        uint32_t* h = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
        for (int e = 0; e < 4; ++e) h[e] = ja_pack16<IsF16<TD>::value>(f[2 * e], f[2 * e + 1]);
        *reinterpret_cast<uint4*>(p) = o;
    } else {   // 4 cells of 16 bits
        uint2 o;
        o.x = ja_pack16<IsF16<TD>::value>(f[0], f[1]);
        o.y = ja_pack16<IsF16<TD>::value>(f[2], f[3]);
        *reinterpret_cast<uint2*>(p) = o;
    }
}

template <bool IS_MAX> __device__ __forceinline__ float combine(float a, float b) { return IS_MAX ? fmaxf(a, b) : a + b; }

// FEW: at most four copies (a form of its own: the two-at-a-time path costs registers that the many-copies loop pays for in
// resident warps -- eight copies ran in 288 us instead of 200 with both in one kernel)
template <typename TS, typename TD, int VEC, bool IS_MAX, bool FEW>
__global__ void __launch_bounds__(256) repartition_agg_kernel(const char* __restrict__ src, char* __restrict__ dst,
                                                              const CopySlab* __restrict__ slabs, int64_t n_slabs, int n_copies,
                                                              int64_t copy_stride) {
    for (int64_t s = blockIdx.x; s < n_slabs; s += gridDim.x) {
        const CopySlab sl = slabs[s];
        const int vpr = sl.row_bytes / (int)(VEC * sizeof(TS));  // accesses per row
        const int total = vpr * sl.rows;
        int i = threadIdx.x;
        if (FEW && VEC > 1) {
            // few copies: two accesses of a thread at a time, every load of both issued first and kept as it came (16 bytes
            // each) until it is combined, so that a thread has as many loads in flight as with many copies
            for (; i + 256 < total; i += 512) {
                const int r0 = i / vpr, c0 = i - r0 * vpr, r1 = (i + 256) / vpr, c1 = i + 256 - r1 * vpr;
                const char* sp0 = src + sl.src_off + (int64_t)r0 * sl.src_pitch + (int64_t)c0 * (VEC * sizeof(TS));
                const char* sp1 = src + sl.src_off + (int64_t)r1 * sl.src_pitch + (int64_t)c1 * (VEC * sizeof(TS));
                uint4 raw0[4], raw1[4];
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (c < n_copies) {
                        raw0[c] = __ldg(reinterpret_cast<const uint4*>(sp0 + (int64_t)c * copy_stride));
                        raw1[c] = __ldg(reinterpret_cast<const uint4*>(sp1 + (int64_t)c * copy_stride));
                    }
                float a0[VEC], a1[VEC];
                unpack_cells<TS>(raw0[0], a0);
                unpack_cells<TS>(raw1[0], a1);
#pragma unroll
                for (int c = 1; c < 4; ++c)
                    if (c < n_copies) {
                        float b0[VEC], b1[VEC];
                        unpack_cells<TS>(raw0[c], b0);
                        unpack_cells<TS>(raw1[c], b1);
#pragma unroll
                        for (int e = 0; e < VEC; ++e) {
                            a0[e] = combine<IS_MAX>(a0[e], b0[e]);
                            a1[e] = combine<IS_MAX>(a1[e], b1[e]);
                        }
                    }
                store_cells<TD, VEC>(dst + sl.dst_off + (int64_t)r0 * sl.dst_pitch + (int64_t)c0 * (VEC * sizeof(TD)), a0);
                store_cells<TD, VEC>(dst + sl.dst_off + (int64_t)r1 * sl.dst_pitch + (int64_t)c1 * (VEC * sizeof(TD)), a1);
            }
        }
        for (; i < total; i += 256) {
            const int r = i / vpr, c = i - r * vpr;
            const char* sp = src + sl.src_off + (int64_t)r * sl.src_pitch + (int64_t)c * (VEC * sizeof(TS));
            float acc[VEC];
            load_cells<TS, VEC>(sp, acc);
            int cc = 1;
            for (; cc + 3 < n_copies; cc += 4) {   // four copies in flight, combined in ascending order
                float t0[VEC], t1[VEC], t2[VEC], t3[VEC];
                load_cells<TS, VEC>(sp + (int64_t)cc * copy_stride, t0);
                load_cells<TS, VEC>(sp + (int64_t)(cc + 1) * copy_stride, t1);
                load_cells<TS, VEC>(sp + (int64_t)(cc + 2) * copy_stride, t2);
                load_cells<TS, VEC>(sp + (int64_t)(cc + 3) * copy_stride, t3);
#pragma unroll
                for (int e = 0; e < VEC; ++e)
                    acc[e] = combine<IS_MAX>(combine<IS_MAX>(combine<IS_MAX>(combine<IS_MAX>(acc[e], t0[e]), t1[e]), t2[e]), t3[e]);
            }
            for (; cc < n_copies; ++cc) {
                float t[VEC];
                load_cells<TS, VEC>(sp + (int64_t)cc * copy_stride, t);
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[e] = combine<IS_MAX>(acc[e], t[e]);
            }
            store_cells<TD, VEC>(dst + sl.dst_off + (int64_t)r * sl.dst_pitch + (int64_t)c * (VEC * sizeof(TD)), acc);
        }
    }
}

template <typename TS, typename TD>
void launch(const char* src, char* dst, const CopySlab* d_slabs, int64_t n_slabs, int n_copies, int64_t copy_stride, bool is_max,
            bool vec, unsigned grid, cudaStream_t st) {
    constexpr int V = VecOf<TS>::N;
#define JA_AGG_LAUNCH(VV, MAXF, FEWF) repartition_agg_kernel<TS, TD, VV, MAXF, FEWF><<<grid, 256, 0, st>>>(src, dst, d_slabs, n_slabs, n_copies, copy_stride)
    const bool few = vec && n_copies <= 4;
    if (vec) {
        if (few) {
            if (is_max) JA_AGG_LAUNCH(V, true, true);
            else JA_AGG_LAUNCH(V, false, true);
        } else {
            if (is_max) JA_AGG_LAUNCH(V, true, false);
            else JA_AGG_LAUNCH(V, false, false);
        }
    } else {
        if (is_max) JA_AGG_LAUNCH(1, true, false);
        else JA_AGG_LAUNCH(1, false, false);
    }
#undef JA_AGG_LAUNCH
}

}  // namespace

ja_status_t ja_launch_repartition_agg(const char* src, char* dst, const CopySlab* d_slabs, int64_t n_slabs, int n_copies,
                                      int64_t copy_stride, ja_dtype_t src_dt, ja_dtype_t dst_dt, ja_agg_t agg, int vec,
                                      cudaStream_t st) {
    if (n_slabs == 0) return JA_OK;
    const unsigned grid = (unsigned)(n_slabs < (int64_t)148 * 64 ? n_slabs : (int64_t)148 * 64);
    const bool is_max = agg == JA_AGG_MAX, v = vec > 1;
    // partial and destination relations: f32 or one 16-bit type (never bf16 on one side and f16 on the other)
    if (src_dt != JA_F32 && dst_dt != JA_F32 && src_dt != dst_dt)
        return ja_fail(JA_ERR_DTYPE, "aggregating relayout: partials and destination of different 16-bit types");
    const bool f16 = src_dt == JA_F16 || dst_dt == JA_F16;
#define JA_AGG_LAUNCH(TS, TD) launch<TS, TD>(src, dst, d_slabs, n_slabs, n_copies, copy_stride, is_max, v, grid, st)
    if (src_dt == JA_F32 && dst_dt == JA_F32) JA_AGG_LAUNCH(float, float);
    else if (src_dt == JA_F32 && f16) JA_AGG_LAUNCH(float, __half);
    else if (src_dt == JA_F32) JA_AGG_LAUNCH(float, __nv_bfloat16);
    else if (dst_dt == JA_F32 && f16) JA_AGG_LAUNCH(__half, float);
    else if (dst_dt == JA_F32) JA_AGG_LAUNCH(__nv_bfloat16, float);
    else if (f16) JA_AGG_LAUNCH(__half, __half);
    else JA_AGG_LAUNCH(__nv_bfloat16, __nv_bfloat16);
#undef JA_AGG_LAUNCH
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}
