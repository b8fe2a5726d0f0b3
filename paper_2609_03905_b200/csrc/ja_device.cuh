// Device-side helpers shared by the kernels: key-table lookups on a RelView and small numeric utilities.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ja_internal.h"

// block index of coordinate x along dimension d: arithmetic on uniform tilings, binary search otherwise
__device__ __forceinline__ int ja_find_blk(const RelView& v, int d, int64_t x) {
    if (v.bs[d]) return (int)(x / v.bs[d]);
    int lo = 0, hi = v.nblk[d] - 1;
    while (lo < hi) {
        int mid = (lo + hi + 1) >> 1;
        if (v.splits[d][mid] <= x) lo = mid;
        else hi = mid - 1;
    }
    return lo;
}

// byte offset in the payload of the cell with tensor coordinates x[0..rank)
__device__ __forceinline__ int64_t ja_elem_off(const RelView& v, const int64_t* x) {
    int64_t flat = 0, off = 0;
#pragma unroll
    for (int d = 0; d < JA_MAX_RANK; ++d) {
        if (d < v.rank) {
            int b = ja_find_blk(v, d, x[d]);
            int64_t lo = v.splits[d][b];
            int64_t w = v.splits[d][b + 1] - lo;
            flat = flat * v.nblk[d] + b;
            off = off * w + (x[d] - lo);
        }
    }
    return v.blk_off[flat] + off * v.esize;
}

__device__ __forceinline__ float ja_to_float(float x) { return x; }
__device__ __forceinline__ float ja_to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ float ja_to_float(__half x) { return __half2float(x); }
template <typename T> __device__ __forceinline__ T ja_from_float(float x);
template <> __device__ __forceinline__ float ja_from_float<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 ja_from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }
template <> __device__ __forceinline__ __half ja_from_float<__half>(float x) { return __float2half_rn(x); }

// cell type <-> ja_dtype_t, and the packed pair of a 16-bit type
template <typename T> struct JaDtypeOf;
template <> struct JaDtypeOf<float> { static constexpr ja_dtype_t value = JA_F32; };
template <> struct JaDtypeOf<__nv_bfloat16> { static constexpr ja_dtype_t value = JA_BF16; };
template <> struct JaDtypeOf<__half> { static constexpr ja_dtype_t value = JA_F16; };
// two f32 -> one packed pair of 16-bit cells (round to nearest even), and back; F16: false = bf16, true = f16
template <bool F16> __device__ __forceinline__ uint32_t ja_pack16(float lo, float hi) {
    if (F16) {
        const __half2 t = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<const uint32_t*>(&t);
    }
    const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&t);
}
template <bool F16> __device__ __forceinline__ float2 ja_unpack16(uint32_t w) {
    if (F16) return __half22float2(*reinterpret_cast<const __half2*>(&w));
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w));
}

// Launch order of the attention CTAs (CTAs are handed to SMs in order of blockIdx.x). One CTA = one query tile (or pair
// of tiles) of one (batch, head). (batch, head) pairs are taken in sections of `sect` consecutive pairs and inside a
// section all pairs run their heaviest tile first, then the next one, and so on. One section holding every pair is
// "longest work first" (short tail; used when tiles differ in weight); sections that fill the GPU once keep the CTAs
// that run together on few (batch, head) pairs, whose K / V tiles are then re-used through L2 (used for equal tiles).
// Returns the slot of the tile in heaviest-first order and the flat (batch, head) index.
__device__ __forceinline__ void ja_attn_decode_cta(int cta, int n_tiles, int n_bh, int sect, int* slot, int* bh) {
    const int per_section = sect * n_tiles;
    const int sec = cta / per_section;
    const int first_bh = sec * sect;
    const int g = min(sect, n_bh - first_bh);       // the last section may hold fewer pairs
    const int local = cta - sec * per_section;
    *slot = local / g;
    *bh = first_bh + local % g;
}

