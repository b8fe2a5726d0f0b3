// Tensor-core matmul join-agg "ij,jk->ik" (MUL / SUM) for bf16 relations under ANY tiling: the form for decompositions
// whose blocks the TMA-fed kernel (k_gemm_tc.cu) cannot address -- block rows that are not multiples of 16 bytes (a
// contracted index cut 64 ways leaves 172-cell rows), blocks of different shapes, blocks narrower than a TMA box. The paper's
// premise is that whatever interval decomposition the optimizer picks is executed at kernel speed; without this kernel such
// decompositions fell to the plain-ALU kernel, forty times slower.
//
// Same contraction engine as the TMA form -- tcgen05.mma, kind::f16, M = 128, N = 256, K = 16, A K-major and B MN-major
// under the 128-byte swizzle, fp32 accumulator in tensor memory, two accumulator stages -- but the operands reach shared
// memory through plain global loads: eight loader warps copy 16-byte pieces into the swizzled layout the matrix
// descriptors expect. Where every block row starts on a 4-byte boundary (even block widths) the pieces travel as
// asynchronous copies (cp.async of 16, 8 or 4 bytes, whatever the source address allows, zero-filled past a block's edge)
// that complete on the stage's barrier, so four stages -- 192 KiB -- are in flight per SM without passing through
// registers; with odd block widths the pieces are assembled from 2-byte loads in registers and stored.
//
// One persistent CTA per SM. A work item is one 128 x 256 tile of ONE output key (tiles never span blocks; blocks smaller
// than a tile leave part of it idle). For its tile a CTA walks the function specs that share the output key, the
// contracted blocks j ascending, 64 contracted cells per pipeline stage: that walk into one accumulator is the SUM
// aggregation of Definition 3.7; the aggregated tile is rounded once and stored at its place in the output block.
//   warps 0..7   loaders        warp 8   tcgen05.mma issuer (converged warp, one elected lane)        warps 9..12  epilogue
// Every mbarrier wait is bounded; on expiry the CTA records JA_ERR_TIMEOUT and leaves through the normal exit.
#include <algorithm>

#include "ja_device.cuh"
#include "ja_ptx.cuh"

namespace {

using namespace ja_ptx;

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int LOADERS = 256, NUM_THREADS = LOADERS + 32 + 128;
constexpr int A_STAGE_BYTES = BM * BK * 2;                  // 16 KiB: 128 rows of 128 bytes
constexpr int B_GROUP_BYTES = BK * 64 * 2;                  // 8 KiB: 64 contracted rows x 64 columns
constexpr int B_STAGE_BYTES = B_GROUP_BYTES * (BN / 64);    // 32 KiB
constexpr int SMEM_BYTES = STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + 1024 + 256;

struct LdParams {
    RelView A, B, C;
    int32_t* status;
    uint32_t wait_cap_us;
    int32_t tiles_i, tiles_k;   // tiles per output block along i and k (of the LARGEST block)
    int32_t total_tiles;        // nblk_i * tiles_i * nblk_k * tiles_k
    int32_t f16;                // cell type of all three relations: 0 = bf16, 1 = f16
};

__device__ __forceinline__ int64_t interval_width(const RelView& v, int d, int idx) {
    if (v.bs[d]) return min(v.bs[d], v.extent[d] - (int64_t)idx * v.bs[d]);
    return v.splits[d][idx + 1] - v.splits[d][idx];
}
__device__ __forceinline__ int64_t block_offset(const RelView& v, int64_t flat) {
    return v.blk_stride ? flat * v.blk_stride : v.blk_off[flat];
}

// Eight consecutive bf16 cells starting at p, of which the first `valid` (0..8) exist; the rest read as zero. The widest
// loads the address allows.
__device__ __forceinline__ uint4 load8(const char* p, int valid) {
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (valid <= 0) return v;
    const uintptr_t a = reinterpret_cast<uintptr_t>(p);
    if (valid >= 8) {
        if ((a & 15) == 0) return *reinterpret_cast<const uint4*>(p);
        if ((a & 7) == 0) {
            const uint2 lo = *reinterpret_cast<const uint2*>(p), hi = *reinterpret_cast<const uint2*>(p + 8);
            return make_uint4(lo.x, lo.y, hi.x, hi.y);
        }
        if ((a & 3) == 0) {
            const uint32_t* q = reinterpret_cast<const uint32_t*>(p);
            return make_uint4(q[0], q[1], q[2], q[3]);
        }
    }
    const uint16_t* h = reinterpret_cast<const uint16_t*>(p);
    uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int e = 0; e < 8; ++e)
        if (e < valid) w[e >> 1] |= (uint32_t)h[e] << ((e & 1) * 16);
    return make_uint4(w[0], w[1], w[2], w[3]);
}
// the mirror image for the output: eight bf16 cells (packed in four words), the first `valid` of them stored
__device__ __forceinline__ void store8(char* p, const uint32_t (&w)[4], int valid) {
    if (valid <= 0) return;
    const uintptr_t a = reinterpret_cast<uintptr_t>(p);
    if (valid >= 8) {
        if ((a & 15) == 0) { *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]); return; }
        if ((a & 3) == 0) {
            uint32_t* q = reinterpret_cast<uint32_t*>(p);
            q[0] = w[0]; q[1] = w[1]; q[2] = w[2]; q[3] = w[3];
            return;
        }
    }
    uint16_t* h = reinterpret_cast<uint16_t*>(p);
#pragma unroll
    for (int e = 0; e < 8; ++e)
        if (e < valid) h[e] = (uint16_t)(w[e >> 1] >> ((e & 1) * 16));
}

// The same eight cells as an asynchronous global -> shared copy (needs a 4-byte aligned source): the widest cp.async the
// address allows; bytes past `valid` cells are zero-filled by the copy itself.
__device__ __forceinline__ void cp_async(uint32_t dst, const char* src, int bytes, int src_bytes) {
    if (bytes == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
    else if (bytes == 8)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void copy8_async(uint32_t dst, const char* p, int valid) {
    const int vb = max(0, min(8, valid)) * 2;
    const uintptr_t a = reinterpret_cast<uintptr_t>(p);
    if ((a & 15) == 0) {
        cp_async(dst, p, 16, vb);
    } else if ((a & 7) == 0) {
        cp_async(dst, p, 8, min(8, vb));
        cp_async(dst + 8, p + 8, 8, max(0, vb - 8));
    } else {
#pragma unroll
        for (int w = 0; w < 4; ++w) cp_async(dst + 4 * w, p + 4 * w, 4, max(0, min(4, vb - 4 * w)));
    }
}

struct Tile {
    int ib, kb;            // output key
    int64_t r0, c0;        // tile origin inside the output block
    int64_t bm, bn;        // extents of the output block
    bool live;             // false: past the end of a block smaller than the largest one
};
__device__ __forceinline__ Tile tile_of(const LdParams& p, int t) {
    Tile tl;
    const int per_kb = p.tiles_k, per_row = p.B.nblk[1] * per_kb;
    const int row = t / per_row, col = t - row * per_row;
    tl.ib = row / p.tiles_i;
    tl.kb = col / per_kb;
    tl.r0 = (int64_t)(row - tl.ib * p.tiles_i) * BM;
    tl.c0 = (int64_t)(col - tl.kb * per_kb) * BN;
    tl.bm = interval_width(p.A, 0, tl.ib);
    tl.bn = interval_width(p.B, 1, tl.kb);
    tl.live = tl.r0 < tl.bm && tl.c0 < tl.bn;
    return tl;
}

// ASYNC: every block row of A and B starts on a 4-byte boundary
template <bool ASYNC, bool F16>   // F16: cells are f16 instead of bf16
__global__ void __launch_bounds__(NUM_THREADS, 1) gemm_ld_kernel(const LdParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;   // swizzle atoms need 1024-byte alignment
    uint8_t* smem = smem_raw + (base - raw);
    uint8_t* pA = smem;
    uint8_t* pB = smem + STAGES * A_STAGE_BYTES;
    const uint32_t sA = base, sB = base + STAGES * A_STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * (A_STAGE_BYTES + B_STAGE_BYTES));
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };                       // loaders (one arrival per warp) -> MMA
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };           // MMA commit -> loaders
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };       // MMA commit -> epilogue
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };  // epilogue (one arrival per warp) -> MMA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
    volatile int* ctl = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0), lane = threadIdx.x % 32;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), ASYNC ? LOADERS : LOADERS / 32);   // one arrival per loader thread's copies / per loader warp
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), 4);
        }
        wait_ctl_init(ctl, p.wait_cap_us);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);
    const RelView &A = p.A, &B = p.B, &C = p.C;
    const int nbj = A.nblk[1], nbk = B.nblk[1];

    if (warp < 8) {
        // ================= loaders =================
        const int tid = threadIdx.x;   // 0..255
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.total_tiles && ok; t += gridDim.x) {
            const Tile tl = tile_of(p, t);
            if (!tl.live) continue;
            for (int jb = 0; jb < nbj && ok; ++jb) {   // the tuples of this output key, ascending j
                const int64_t wj = interval_width(A, 1, jb);
                const char* a_blk = A.base + block_offset(A, (int64_t)tl.ib * nbj + jb);   // bm rows of wj cells
                const char* b_blk = B.base + block_offset(B, (int64_t)jb * nbk + tl.kb);   // wj rows of bn cells
                for (int64_t j0 = 0; j0 < wj; j0 += BK) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1, ctl, p.status)) { ok = false; break; }
                    // A: 128 rows x 8 pieces of 8 contracted cells; piece (r, c) lives at r * 128 + ((c ^ (r & 7)) * 16)
                    // B: 64 contracted rows x 32 pieces of 8 columns; piece (k, c) lives in column group c / 8 at
                    //    k * 128 + (((c & 7) ^ (k & 7)) * 16)
                    if (ASYNC) {
                        const uint32_t dA = sA + stage * A_STAGE_BYTES, dB = sB + stage * B_STAGE_BYTES;
#pragma unroll
                        for (int n = 0; n < BM * 8 / LOADERS; ++n) {
                            const int e = tid + n * LOADERS, r = e >> 3, c = e & 7;
                            const int64_t row = tl.r0 + r, k = j0 + c * 8;
                            const bool in = row < tl.bm && k < wj;
                            copy8_async(dA + r * 128 + ((c ^ (r & 7)) << 4), in ? a_blk + (row * wj + k) * 2 : a_blk, in ? (int)min((int64_t)8, wj - k) : 0);
                        }
#pragma unroll
                        for (int n = 0; n < BK * 32 / LOADERS; ++n) {
                            const int e = tid + n * LOADERS, kr = e >> 5, c = e & 31;
                            const int64_t k = j0 + kr, col = tl.c0 + c * 8;
                            const bool in = k < wj && col < tl.bn;
                            copy8_async(dB + (c >> 3) * B_GROUP_BYTES + kr * 128 + (((c & 7) ^ (kr & 7)) << 4), in ? b_blk + (k * tl.bn + col) * 2 : b_blk,
                                        in ? (int)min((int64_t)8, tl.bn - col) : 0);
                        }
                        // this thread's arrival on the stage's barrier happens when all its copies above have landed
                        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(full_bar(stage)) : "memory");
                    } else {
                        uint8_t* dA = pA + stage * A_STAGE_BYTES;
                        uint8_t* dB = pB + stage * B_STAGE_BYTES;
                        uint4 va[BM * 8 / LOADERS];
#pragma unroll
                        for (int n = 0; n < BM * 8 / LOADERS; ++n) {
                            const int e = tid + n * LOADERS, r = e >> 3, c = e & 7;
                            const int64_t row = tl.r0 + r, k = j0 + c * 8;
                            va[n] = load8(a_blk + (row * wj + k) * 2, row < tl.bm ? (int)min((int64_t)8, wj - k) : 0);
                        }
                        uint4 vb[BK * 32 / LOADERS];
#pragma unroll
                        for (int n = 0; n < BK * 32 / LOADERS; ++n) {
                            const int e = tid + n * LOADERS, kr = e >> 5, c = e & 31;
                            const int64_t k = j0 + kr, col = tl.c0 + c * 8;
                            vb[n] = load8(b_blk + (k * tl.bn + col) * 2, k < wj ? (int)min((int64_t)8, tl.bn - col) : 0);
                        }
#pragma unroll
                        for (int n = 0; n < BM * 8 / LOADERS; ++n) {
                            const int e = tid + n * LOADERS, r = e >> 3, c = e & 7;
                            *reinterpret_cast<uint4*>(dA + r * 128 + ((c ^ (r & 7)) << 4)) = va[n];
                        }
#pragma unroll
                        for (int n = 0; n < BK * 32 / LOADERS; ++n) {
                            const int e = tid + n * LOADERS, kr = e >> 5, c = e & 31;
                            *reinterpret_cast<uint4*>(dB + (c >> 3) * B_GROUP_BYTES + kr * 128 + (((c & 7) ^ (kr & 7)) << 4)) = vb[n];
                        }
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads through the async proxy
                        __syncwarp();
                        if (lane == 0) mbar_arrive(full_bar(stage));
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 8) {
        // ================= MMA issuer =================
        const uint32_t leader = elect_one();
        constexpr uint32_t fmt = F16 ? 0u : 1u;   // A and B: bf16 (format 1) or f16 (format 0); D f32; B MN-major
        const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | (1u << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
        int stage = 0, it = 0;
        uint32_t phase = 0, acc_phase[2] = {0, 0};
        bool ok = true;
        for (int t = blockIdx.x; t < p.total_tiles && ok; t += gridDim.x) {
            const Tile tl = tile_of(p, t);
            if (!tl.live) continue;
            const int acc = it & 1;
            ++it;
            if (!mbar_wait(tempty_bar(acc), acc_phase[acc] ^ 1, ctl, p.status)) { ok = false; break; }
            acc_phase[acc] ^= 1;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * BN;
            uint32_t accumulate = 0;
            for (int jb = 0; jb < nbj && ok; ++jb) {
                const int64_t wj = interval_width(A, 1, jb);
                for (int64_t j0 = 0; j0 < wj; j0 += BK) {
                    if (!mbar_wait(full_bar(stage), phase, ctl, p.status)) { ok = false; break; }
                    if (ASYNC) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the copies wrote through the generic proxy
                    tc_fence_after();
                    const uint32_t a_addr = sA + stage * A_STAGE_BYTES, b_addr = sB + stage * B_STAGE_BYTES;
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk)   // zero-filled tails make every stage a full one
                        umma_bf16_w<1>(d_tmem, desc_sw128(a_addr + kk * 32, 16), desc_sw128(b_addr + kk * 2048, B_GROUP_BYTES), idesc,
                                       kk > 0 ? 1u : accumulate, leader);
                    accumulate = 1;
                    umma_commit_w<1>(empty_bar(stage), leader);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (ok) umma_commit_w<1>(tfull_bar(acc), leader);
        }
    } else {
        // ================= epilogue =================
        const int q = warp & 3;   // TMEM lane quarter this warp may access
        uint32_t acc_phase[2] = {0, 0};
        int it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < p.total_tiles && ok; t += gridDim.x) {
            const Tile tl = tile_of(p, t);
            if (!tl.live) continue;
            const int acc = it & 1;
            ++it;
            if (!mbar_wait(tfull_bar(acc), acc_phase[acc], ctl, p.status)) { ok = false; break; }
            acc_phase[acc] ^= 1;
            tc_fence_after();
            const int64_t r = tl.r0 + q * 32 + lane;
            char* c_row = C.base + block_offset(C, (int64_t)tl.ib * nbk + tl.kb) + (r * tl.bn + tl.c0) * 2;
            const int64_t cols = min((int64_t)BN, tl.bn - tl.c0);
#pragma unroll 1
            for (int ch = 0; ch * 32 < cols; ++ch) {
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + ch * 32, v);
                tmem_ld_wait();
                if (r < tl.bm) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float lo = __uint_as_float(v[g * 8 + 2 * e]), hi = __uint_as_float(v[g * 8 + 2 * e + 1]);
                            w[e] = ja_pack16<F16>(lo, hi);
                        }
                        store8(c_row + (ch * 32 + g * 8) * 2, w, (int)min((int64_t)8, cols - ch * 32 - g * 8));
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

}  // namespace

// *launched stays false when the relations are too small for 128 x 256 tiles to pay (the plain-ALU kernel takes them)
ja_status_t ja_launch_gemm_ld(const ja_relation* Ar, const ja_relation* Br, const ja_relation* Cr, cudaStream_t st, bool* launched) {
    *launched = false;
    if (Ar->dtype == JA_F32 || Br->dtype != Ar->dtype || Cr->dtype != Ar->dtype) return JA_OK;
    int64_t max_bm = 0, max_bn = 0;
    for (int i = 0; i < Ar->nblk[0]; ++i) max_bm = std::max(max_bm, Ar->splits[0][i + 1] - Ar->splits[0][i]);
    for (int i = 0; i < Br->nblk[1]; ++i) max_bn = std::max(max_bn, Br->splits[1][i + 1] - Br->splits[1][i]);
    if (max_bm < 64 || max_bn < 64 || Ar->extent[1] < 64) return JA_OK;
    LdParams p;
    p.A = ja_view(Ar);
    p.B = ja_view(Br);
    p.C = ja_view(Cr);
    p.f16 = Ar->dtype == JA_F16;
    p.status = ja_device_status_word(st);
    if (!p.status) return ja_fail(JA_ERR_CUDA, "cannot resolve the device status word");
    p.wait_cap_us = (uint32_t)ja_config().wait_cap_us;
    p.tiles_i = (int)((max_bm + BM - 1) / BM);
    p.tiles_k = (int)((max_bn + BN - 1) / BN);
    const int64_t total = (int64_t)Ar->nblk[0] * p.tiles_i * Br->nblk[1] * p.tiles_k;
    if (total >= (1ll << 31)) return JA_OK;
    p.total_tiles = (int)total;
    bool even = true;   // every block row starts on a 4-byte boundary when every block width of A's j and B's k is even
    for (int i = 0; i < Ar->nblk[1]; ++i) even = even && (Ar->splits[1][i + 1] - Ar->splits[1][i]) % 2 == 0;
    for (int i = 0; i < Br->nblk[1]; ++i) even = even && (Br->splits[1][i + 1] - Br->splits[1][i]) % 2 == 0;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!configured[dev & 63]) {
        JA_CUDA(cudaFuncSetAttribute(gemm_ld_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
        JA_CUDA(cudaFuncSetAttribute(gemm_ld_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
        JA_CUDA(cudaFuncSetAttribute(gemm_ld_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
        JA_CUDA(cudaFuncSetAttribute(gemm_ld_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
        configured[dev & 63] = true;
    }
    const int grid = (int)std::min<int64_t>(total, ja_sm_count());
    if (p.f16) {
        if (even) gemm_ld_kernel<true, true><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(p);
        else gemm_ld_kernel<false, true><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(p);
    } else {
        if (even) gemm_ld_kernel<true, false><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(p);
        else gemm_ld_kernel<false, false><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(p);
    }
    JA_CUDA(cudaGetLastError());
    ja_count_launch();
    *launched = true;
    return JA_OK;
}
