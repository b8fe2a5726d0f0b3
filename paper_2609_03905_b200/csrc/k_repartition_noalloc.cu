// ja_repartition_noalloc: the block relayout of ja_repartition for callers that must not allocate.
//
// Who needs it: code that runs where device allocation is forbidden or impossible -- inside a region whose memory
// was budgeted up front (an inference server that hands every byte of HBM to its own pool at start-up), in a
// loop that must never take cudaMalloc's implicit device synchronisation, or under a memory-accounting
// harness that fails any allocation it did not make itself. ja_repartition builds its copy plan in a
// cudaMalloc'ed table and keeps it cached; this entry point keeps the plan in a fixed, file-scope device array
// instead and never calls cudaMalloc, cudaFree, or any allocating library routine (host or device).
//
// Consequences of the fixed array, which every caller should know:
//   * it is sized for JA_NOALLOC_MAX_SLABS copy slabs (512 KiB); every GPU that loads the library holds it
//     until the process exits; a relayout that needs more slabs is refused with JA_ERR_UNSUPPORTED;
//   * all calls share it, and it keeps the previous call's plan until the next call overwrites the part it
//     uses (nothing in it has to start at zero: a call only reads the entries it has just written);
//   * two calls that overlap on the GPU (different streams, or the same stream from two threads) race on it --
//     serialise them;
//   * the first call on each device resolves the array's device address (set-up, one cudaGetSymbolAddress with
//     that device current); make that first call before starting any stream capture;
//   * the plan travels to the device with a stream-ordered copy out of a fixed host table that the next call
//     overwrites, so the host may block for the few microseconds the copy needs, and a call on a stream that is
//     being captured is refused (JA_ERR_UNSUPPORTED, nothing enqueued): a recorded copy would read, at replay
//     time, whatever plan the latest call left in that table.
#include <string.h>

#include <mutex>

#include "ja_device.cuh"

#define JA_NOALLOC_MAX_SLABS 16384
#define JA_NOALLOC_MAX_SPLITS 1024   // split points per dimension after overlay

namespace {

// The plan lives here. In host code this name is only a stand-in for the symbol: it is NOT a device address and
// must never be passed to a kernel; the address comes from cudaGetSymbolAddress (see scratch_for_device()).
static __device__ __align__(256) CopySlab g_noalloc_slabs[JA_NOALLOC_MAX_SLABS];

template <typename V>
__global__ void __launch_bounds__(256) repartition_noalloc_kernel(const char* __restrict__ src, char* __restrict__ dst,
                                                                  const CopySlab* __restrict__ slabs, int n_slabs) {
    for (int s = blockIdx.x; s < n_slabs; s += gridDim.x) {
        const CopySlab sl = slabs[s];
        const int vpr = sl.row_bytes / (int)sizeof(V);
        const int total = vpr * sl.rows;
        const char* sp = src + sl.src_off;
        char* dp = dst + sl.dst_off;
        for (int i = threadIdx.x; i < total; i += 256) {
            const int r = i / vpr, c = i - r * vpr;
            *reinterpret_cast<V*>(dp + (int64_t)r * sl.dst_pitch + (int64_t)c * sizeof(V)) =
                *reinterpret_cast<const V*>(sp + (int64_t)r * sl.src_pitch + (int64_t)c * sizeof(V));
        }
    }
}

constexpr int MAX_DEVICES = 64;
CopySlab* g_scratch_ptr[MAX_DEVICES];   // device address of g_noalloc_slabs, per device (zero-initialised)

// set-up, once per device, with that device current
ja_status_t scratch_for_device(CopySlab** out) {
    int dev = 0;
    JA_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return ja_fail(JA_ERR_UNSUPPORTED, "device ordinal %d not supported", dev);
    if (!g_scratch_ptr[dev]) {
        CopySlab* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void**)&p, g_noalloc_slabs);
        if (e != cudaSuccess) return ja_cuda_fail(e, "cudaGetSymbolAddress(g_noalloc_slabs)");
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return JA_OK;
}

struct Tiling1D {
    const int64_t* sp;
    int32_t n;   // intervals
};
int owner(const Tiling1D& t, int64_t x) {   // interval of t that contains x
    int lo = 0, hi = t.n - 1;
    while (lo < hi) {
        int mid = (lo + hi + 1) >> 1;
        if (t.sp[mid] <= x) lo = mid;
        else hi = mid - 1;
    }
    return lo;
}

}  // namespace

extern "C" ja_status_t ja_repartition_noalloc(int32_t rank, const int64_t* extents, const int32_t* src_nparts,
                                              const int64_t* const* src_splits, const int32_t* dst_nparts,
                                              const int64_t* const* dst_splits, ja_dtype_t dtype, const void* src_device,
                                              void* dst_device, void* cuda_stream) {
    if (rank < 1 || rank > JA_MAX_RANK || !extents || !src_nparts || !src_splits || !dst_nparts || !dst_splits)
        return ja_fail(JA_ERR_INVALID_ARG, "rank must be 1..%d and every array non-NULL", JA_MAX_RANK);
    if (dtype != JA_F32 && dtype != JA_BF16 && dtype != JA_F16) return ja_fail(JA_ERR_DTYPE, "unknown dtype %d", (int)dtype);
    if (!src_device || !dst_device || src_device == dst_device) return ja_fail(JA_ERR_INVALID_ARG, "payload pointers must be distinct and non-NULL");
    if (((uintptr_t)src_device | (uintptr_t)dst_device) % JA_ALIGN) return ja_fail(JA_ERR_ALIGNMENT, "payloads must be %d-byte aligned", JA_ALIGN);
    const int es = dtype == JA_F32 ? 4 : 2;
    Tiling1D S[JA_MAX_RANK], T[JA_MAX_RANK];
    // All host-side working tables are fixed-size statics (no heap); the mutex serialises the host side of concurrent
    // calls. It does not make overlapping GPU work safe: the device plan table is still shared.
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    static int64_t over[JA_MAX_RANK][JA_NOALLOC_MAX_SPLITS];   // overlay split points per dimension
    int n_over[JA_MAX_RANK];
    int64_t n_atoms = 1;
    for (int d = 0; d < rank; ++d) {
        S[d] = {src_splits[d], src_nparts[d]};
        T[d] = {dst_splits[d], dst_nparts[d]};
        for (const Tiling1D* t : {&S[d], &T[d]}) {
            if (t->n < 1 || !t->sp || t->sp[0] != 0 || t->sp[t->n] != extents[d])
                return ja_fail(JA_ERR_TILING, "split points of dimension %d do not tile [0, %lld)", d, (long long)extents[d]);
            for (int i = 0; i < t->n; ++i)
                if (t->sp[i + 1] <= t->sp[i]) return ja_fail(JA_ERR_TILING, "split points of dimension %d are not ascending", d);
        }
        if (S[d].n + T[d].n + 2 > JA_NOALLOC_MAX_SPLITS)
            return ja_fail(JA_ERR_UNSUPPORTED, "dimension %d has more than %d split points", d, JA_NOALLOC_MAX_SPLITS);
        int i = 0, j = 0, n = 0;   // merge the two ascending lists, dropping duplicates
        while (i <= S[d].n || j <= T[d].n) {
            int64_t a = i <= S[d].n ? S[d].sp[i] : INT64_MAX, b = j <= T[d].n ? T[d].sp[j] : INT64_MAX;
            int64_t v = a < b ? a : b;
            if (a == v) ++i;
            if (b == v) ++j;
            over[d][n++] = v;
        }
        n_over[d] = n - 1;   // atoms along d
        n_atoms *= n_over[d];
    }
    int64_t total_blocks_s = 1, total_blocks_t = 1;
    for (int d = 0; d < rank; ++d) { total_blocks_s *= S[d].n; total_blocks_t *= T[d].n; }
    if (total_blocks_s > 4096 || total_blocks_t > 4096)
        return ja_fail(JA_ERR_UNSUPPORTED, "ja_repartition_noalloc handles at most 4096 blocks per tiling");
    // per-block byte offsets (row-major key order, 128-byte aligned blocks)
    static int64_t s_off[4096], t_off[4096];
    {
        for (int pass = 0; pass < 2; ++pass) {
            const Tiling1D* t = pass ? T : S;
            int64_t* tab = pass ? t_off : s_off;
            int32_t idx[JA_MAX_RANK] = {0, 0, 0, 0};
            int64_t off = 0, nb = pass ? total_blocks_t : total_blocks_s;
            for (int64_t b = 0; b < nb; ++b) {
                tab[b] = off;
                int64_t n = 1;
                for (int d = 0; d < rank; ++d) n *= t[d].sp[idx[d] + 1] - t[d].sp[idx[d]];
                off += (n * es + JA_ALIGN - 1) / JA_ALIGN * JA_ALIGN;
                for (int d = rank - 1; d >= 0; --d) {
                    if (++idx[d] < t[d].n) break;
                    idx[d] = 0;
                }
            }
        }
    }
    // ---- atoms -> slabs, into a fixed staging table ---------------------------------------------------------------
    static CopySlab host_slabs[JA_NOALLOC_MAX_SLABS];
    int64_t n_slabs = 0, all_or = 0;
    int32_t a_idx[JA_MAX_RANK] = {0, 0, 0, 0};
    for (int64_t a = 0; a < n_atoms; ++a) {
        int64_t lo[JA_MAX_RANK], hi[JA_MAX_RANK];
        int32_t sb[JA_MAX_RANK], tb[JA_MAX_RANK];
        int64_t sflat = 0, tflat = 0;
        for (int d = 0; d < rank; ++d) {
            lo[d] = over[d][a_idx[d]];
            hi[d] = over[d][a_idx[d] + 1];
            sb[d] = owner(S[d], lo[d]);
            tb[d] = owner(T[d], lo[d]);
            sflat = sflat * S[d].n + sb[d];
            tflat = tflat * T[d].n + tb[d];
        }
        const int64_t rows = rank >= 2 ? hi[rank - 2] - lo[rank - 2] : 1;
        const int64_t row_bytes = (hi[rank - 1] - lo[rank - 1]) * es;
        int64_t outer = 1;
        for (int d = 0; d + 2 < rank; ++d) outer *= hi[d] - lo[d];
        const int64_t rows_per = (64 * 1024) / row_bytes > 0 ? (64 * 1024) / row_bytes : 1;
        const int64_t sw = S[rank - 1].sp[sb[rank - 1] + 1] - S[rank - 1].sp[sb[rank - 1]];
        const int64_t tw = T[rank - 1].sp[tb[rank - 1] + 1] - T[rank - 1].sp[tb[rank - 1]];
        for (int64_t o = 0; o < outer; ++o) {
            int64_t x[JA_MAX_RANK];
            int64_t rem = o;
            for (int d = rank - 3; d >= 0; --d) {
                const int64_t e = hi[d] - lo[d];
                x[d] = lo[d] + rem % e;
                rem /= e;
            }
            for (int64_t r0 = 0; r0 < rows; r0 += rows_per) {
                if (rank >= 2) x[rank - 2] = lo[rank - 2] + r0;
                x[rank - 1] = lo[rank - 1];
                int64_t so = 0, to = 0;   // element offsets inside the source / destination block
                for (int d = 0; d < rank; ++d) {
                    const int64_t slo = S[d].sp[sb[d]], swd = S[d].sp[sb[d] + 1] - slo;
                    const int64_t tlo = T[d].sp[tb[d]], twd = T[d].sp[tb[d] + 1] - tlo;
                    so = so * swd + (x[d] - slo);
                    to = to * twd + (x[d] - tlo);
                }
                if (n_slabs >= JA_NOALLOC_MAX_SLABS)
                    return ja_fail(JA_ERR_UNSUPPORTED, "relayout needs more than %d copy slabs (the fixed plan table of ja_repartition_noalloc)",
                                   JA_NOALLOC_MAX_SLABS);
                CopySlab& s = host_slabs[n_slabs++];
                s.src_off = s_off[sflat] + so * es;
                s.dst_off = t_off[tflat] + to * es;
                s.rows = (int32_t)((rows - r0) < rows_per ? (rows - r0) : rows_per);
                s.row_bytes = (int32_t)row_bytes;
                s.src_pitch = (int32_t)(sw * es);
                s.dst_pitch = (int32_t)(tw * es);
                all_or |= s.src_off | s.dst_off | s.row_bytes | s.src_pitch | s.dst_pitch;
            }
        }
        for (int d = rank - 1; d >= 0; --d) {
            if (++a_idx[d] < n_over[d]) break;
            a_idx[d] = 0;
        }
    }
    if (n_slabs == 0) return JA_OK;
    CopySlab* d_slabs = nullptr;
    ja_status_t st = scratch_for_device(&d_slabs);
    if (st != JA_OK) return st;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        JA_CUDA(cudaStreamIsCapturing(stream, &cap));
        if (cap != cudaStreamCaptureStatusNone)
            return ja_fail(JA_ERR_UNSUPPORTED, "ja_repartition_noalloc was called on a stream that is being captured: its plan is staged in "
                                               "a host table shared by all calls, which a replay would read too late");
    }
    // plan -> the fixed device table (stream-ordered; the copy reads host_slabs before returning because it is pageable)
    JA_CUDA(cudaMemcpyAsync(d_slabs, host_slabs, (size_t)n_slabs * sizeof(CopySlab), cudaMemcpyHostToDevice, stream));
    int vec = 16;
    while (vec > es && (all_or % vec) != 0) vec /= 2;
    const unsigned grid = (unsigned)(n_slabs < 148 * 64 ? n_slabs : 148 * 64);
    const char* sp = (const char*)src_device;
    char* dp = (char*)dst_device;
    switch (vec) {
        case 16: repartition_noalloc_kernel<uint4><<<grid, 256, 0, stream>>>(sp, dp, d_slabs, (int)n_slabs); break;
        case 8: repartition_noalloc_kernel<uint2><<<grid, 256, 0, stream>>>(sp, dp, d_slabs, (int)n_slabs); break;
        case 4: repartition_noalloc_kernel<uint32_t><<<grid, 256, 0, stream>>>(sp, dp, d_slabs, (int)n_slabs); break;
        default: repartition_noalloc_kernel<uint16_t><<<grid, 256, 0, stream>>>(sp, dp, d_slabs, (int)n_slabs); break;
    }
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}
