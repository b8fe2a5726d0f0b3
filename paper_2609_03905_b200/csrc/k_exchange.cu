// Kernels of an exchange program executed on one GPU (Sections 5.2 - 5.3): decompose / recompose as batched box copies
// between relation blocks and dense atom buffers, and the local aggregation stage of an action -- the (+)-combination of
// the materialised parts of an aggregate, in the order given, in f32, rounded once. All three are plain HBM streams.
#include "ja_device.cuh"

namespace {

// 16-byte accesses when every offset, pitch and run of the launch allows, else one cell per access. Long runs: a CTA takes whole
// runs (the run's two offsets are computed once, the threads stride along it); short runs: the box is walked as one flat range.
template <typename V>
__global__ void __launch_bounds__(256) box_copy_kernel(const char* __restrict__ src, char* __restrict__ dst,
                                                        const JaBoxCopy* __restrict__ boxes) {
    const JaBoxCopy b = boxes[blockIdx.y];
    const int64_t per_row = b.run_bytes / (int64_t)sizeof(V), rows = b.n0 * b.n1;
    if (per_row >= 256) {
        for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
            const int64_t r0 = row / b.n1, r1 = row - r0 * b.n1;
            const V* s = reinterpret_cast<const V*>(src + b.src_off + r0 * b.src_pitch0 + r1 * b.src_pitch1);
            V* d = reinterpret_cast<V*>(dst + b.dst_off + r0 * b.dst_pitch0 + r1 * b.dst_pitch1);
            int64_t x = threadIdx.x;
            for (; x + 768 < per_row; x += 1024) {          // four independent accesses in flight per thread
                const V v0 = s[x], v1 = s[x + 256], v2 = s[x + 512], v3 = s[x + 768];
                d[x] = v0; d[x + 256] = v1; d[x + 512] = v2; d[x + 768] = v3;
            }
            for (; x < per_row; x += 256) d[x] = s[x];
        }
        return;
    }
    const int64_t total = rows * per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / per_row, x = i - row * per_row, r0 = row / b.n1, r1 = row - r0 * b.n1;
        const V v = *reinterpret_cast<const V*>(src + b.src_off + r0 * b.src_pitch0 + r1 * b.src_pitch1 + x * (int64_t)sizeof(V));
        *reinterpret_cast<V*>(dst + b.dst_off + r0 * b.dst_pitch0 + r1 * b.dst_pitch1 + x * (int64_t)sizeof(V)) = v;
    }
}

constexpr int MAX_PARTS = JA_EXCHANGE_MAX_PARTS;
struct CombineParams {
    const char* part[MAX_PARTS];
    char* out;
    int64_t n_vec;       // 16-byte vectors (the buffers are padded to whole vectors)
    int32_t n_parts, is_max;
};

template <typename T> struct Cells16 { static constexpr int N = 16 / (int)sizeof(T); };
template <typename T> __device__ __forceinline__ void unpack16(const uint4& v, float (&f)[Cells16<T>::N]);
template <> __device__ __forceinline__ void unpack16<float>(const uint4& v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
template <bool F16> __device__ __forceinline__ void unpack16_half(const uint4& v, float (&f)[8]) {
    const float2 a = ja_unpack16<F16>(v.x), b = ja_unpack16<F16>(v.y), c = ja_unpack16<F16>(v.z), d = ja_unpack16<F16>(v.w);
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
}
template <> __device__ __forceinline__ void unpack16<__nv_bfloat16>(const uint4& v, float (&f)[8]) { unpack16_half<false>(v, f); }
template <> __device__ __forceinline__ void unpack16<__half>(const uint4& v, float (&f)[8]) { unpack16_half<true>(v, f); }
template <typename T> __device__ __forceinline__ uint4 pack16(const float (&f)[Cells16<T>::N]);
template <> __device__ __forceinline__ uint4 pack16<float>(const float (&f)[4]) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
template <> __device__ __forceinline__ uint4 pack16<__nv_bfloat16>(const float (&f)[8]) {
    return make_uint4(ja_pack16<false>(f[0], f[1]), ja_pack16<false>(f[2], f[3]), ja_pack16<false>(f[4], f[5]), ja_pack16<false>(f[6], f[7]));
}
template <> __device__ __forceinline__ uint4 pack16<__half>(const float (&f)[8]) {
    return make_uint4(ja_pack16<true>(f[0], f[1]), ja_pack16<true>(f[2], f[3]), ja_pack16<true>(f[4], f[5]), ja_pack16<true>(f[6], f[7]));
}

// out = part[0] (+) part[1] (+) ... in that order; up to four parts' loads are in flight per thread
template <typename T>
__global__ void __launch_bounds__(256) combine_kernel(const CombineParams p) {
    constexpr int N = Cells16<T>::N;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p.n_parts == 2) {
        // two parts: two vectors of a thread at a time, so that four loads are in flight per thread as with more parts
        const uint4 *a = reinterpret_cast<const uint4*>(p.part[0]), *b = reinterpret_cast<const uint4*>(p.part[1]);
        for (; i + stride < p.n_vec; i += 2 * stride) {
            const uint4 a0 = a[i], a1 = a[i + stride], b0 = b[i], b1 = b[i + stride];
            float x0[N], x1[N], y0[N], y1[N];
            unpack16<T>(a0, x0);
            unpack16<T>(b0, y0);
            unpack16<T>(a1, x1);
            unpack16<T>(b1, y1);
#pragma unroll
            for (int e = 0; e < N; ++e) {
                x0[e] = p.is_max ? fmaxf(x0[e], y0[e]) : x0[e] + y0[e];
                x1[e] = p.is_max ? fmaxf(x1[e], y1[e]) : x1[e] + y1[e];
            }
            reinterpret_cast<uint4*>(p.out)[i] = pack16<T>(x0);
            reinterpret_cast<uint4*>(p.out)[i + stride] = pack16<T>(x1);
        }
    }
    for (; i < p.n_vec; i += stride) {
        float acc[N];
        unpack16<T>(reinterpret_cast<const uint4*>(p.part[0])[i], acc);
        for (int c0 = 1; c0 < p.n_parts; c0 += 4) {
            uint4 raw[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (c0 + k < p.n_parts) raw[k] = reinterpret_cast<const uint4*>(p.part[c0 + k])[i];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (c0 + k >= p.n_parts) break;
                float f[N];
                unpack16<T>(raw[k], f);
#pragma unroll
                for (int e = 0; e < N; ++e) acc[e] = p.is_max ? fmaxf(acc[e], f[e]) : acc[e] + f[e];
            }
        }
        reinterpret_cast<uint4*>(p.out)[i] = pack16<T>(acc);
    }
}

}  // namespace

ja_status_t ja_launch_box_copies(const char* src, char* dst, const JaBoxCopy* d_boxes, int n_boxes, int64_t max_box_bytes,
                                 bool vec16, int esize, cudaStream_t st) {
    if (n_boxes <= 0) return JA_OK;
    const int64_t per_box = (max_box_bytes / (vec16 ? 16 : esize) + 255) / 256;
    const int64_t cap = std::max<int64_t>(1, (int64_t)ja_sm_count() * 8 / n_boxes);
    dim3 grid((unsigned)std::max<int64_t>(1, std::min(per_box, cap)), (unsigned)n_boxes);
    if (vec16) box_copy_kernel<uint4><<<grid, 256, 0, st>>>(src, dst, d_boxes);
    else if (esize == 4) box_copy_kernel<uint32_t><<<grid, 256, 0, st>>>(src, dst, d_boxes);
    else box_copy_kernel<uint16_t><<<grid, 256, 0, st>>>(src, dst, d_boxes);
    JA_CUDA(cudaGetLastError());
    ja_count_launch();
    return JA_OK;
}

ja_status_t ja_launch_exchange_combine(const void* const* parts, int n_parts, void* out, int64_t bytes, ja_dtype_t dt,
                                       ja_agg_t agg, cudaStream_t st) {
    if (n_parts < 2 || n_parts > MAX_PARTS) return ja_fail(JA_ERR_UNSUPPORTED, "an aggregation of %d parts (2..%d)", n_parts, MAX_PARTS);
    CombineParams p;
    for (int i = 0; i < n_parts; ++i) p.part[i] = (const char*)parts[i];
    p.out = (char*)out;
    p.n_vec = (bytes + 15) / 16;
    p.n_parts = n_parts;
    p.is_max = agg == JA_AGG_MAX;
    const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((p.n_vec + 255) / 256, (int64_t)ja_sm_count() * 8));
    if (dt == JA_F32) combine_kernel<float><<<grid, 256, 0, st>>>(p);
    else if (dt == JA_F16) combine_kernel<__half><<<grid, 256, 0, st>>>(p);
    else combine_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(p);
    JA_CUDA(cudaGetLastError());
    ja_count_launch();
    return JA_OK;
}
