// ja_repartition data movement (Section 5.3): the overlay of the source and destination tilings gives
// atoms; each atom is cut into 2-D slabs (rows x contiguous run) and copied from its source block to its
// destination block -- "decompose" and "recompose" in one pass, no staging buffer. One CTA per slab,
// 128-bit accesses when every offset, pitch and run length allows it. Pure byte movement: bit-exact.
#include "ja_device.cuh"

namespace {

template <typename V>
__global__ void __launch_bounds__(256) repartition_kernel(const char* __restrict__ src, char* __restrict__ dst,
                                                          const CopySlab* __restrict__ slabs, int64_t n_slabs) {
    for (int64_t s = blockIdx.x; s < n_slabs; s += gridDim.x) {
        const CopySlab sl = slabs[s];
        const int vpr = sl.row_bytes / (int)sizeof(V);  // vectors per row
        const int total = vpr * sl.rows;
        const char* sp = src + sl.src_off;
        char* dp = dst + sl.dst_off;
        for (int i = threadIdx.x; i < total; i += 256) {
            int r = i / vpr, c = i - r * vpr;
            V v = *reinterpret_cast<const V*>(sp + (int64_t)r * sl.src_pitch + (int64_t)c * sizeof(V));
            *reinterpret_cast<V*>(dp + (int64_t)r * sl.dst_pitch + (int64_t)c * sizeof(V)) = v;
        }
    }
}

}  // namespace

ja_status_t ja_launch_repartition(const char* src, char* dst, const CopySlab* d_slabs, int64_t n_slabs, int vec_bytes,
                                  cudaStream_t st) {
    if (n_slabs == 0) return JA_OK;
    unsigned grid = (unsigned)(n_slabs < (int64_t)148 * 64 ? n_slabs : (int64_t)148 * 64);
    switch (vec_bytes) {
        case 16: repartition_kernel<uint4><<<grid, 256, 0, st>>>(src, dst, d_slabs, n_slabs); break;
        case 8: repartition_kernel<uint2><<<grid, 256, 0, st>>>(src, dst, d_slabs, n_slabs); break;
        case 4: repartition_kernel<uint32_t><<<grid, 256, 0, st>>>(src, dst, d_slabs, n_slabs); break;
        default: repartition_kernel<uint16_t><<<grid, 256, 0, st>>>(src, dst, d_slabs, n_slabs); break;
    }
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}
