// Tensor-core matmul join-agg "ij,jk->ik" (MUL / SUM) for bf16 relations with uniform blocks.
//
// One persistent CTA per SM. For every output tile (128 rows x up to 256 columns of ONE output key, or of
// several adjacent output keys when blocks are narrow) the CTA walks the function specs that share that
// output key in ascending order of the contracted block index j -- the SUM aggregation of Definition 3.7 is
// the accumulation of all those tuples into one fp32 accumulator in tensor memory; only the aggregated block
// is written (Recompose = the store at the key's offset).
//
//   warp 0      TMA producer: cp.async.bulk.tensor straight from the block-key layout. A relation with
//               uniform blocks is a rank-4 tensor (col in block, row in block, col-block, row-block), so one
//               tensor map per operand addresses every block; ragged tiles rely on zero fill inside a block.
//   warp 1      tcgen05.mma issuer (one elected lane), kind::f16, M=128, N<=256, K=16, A K-major and
//               B MN-major (weights are [in, out] row-major), both under the 128-byte swizzle.
//   warps 2..5  epilogue: tcgen05.ld of the fp32 accumulator, one RNE rounding to bf16, 16-byte stores.
//
// Two accumulator stages (2 x 256 TMEM columns) let the epilogue of tile t overlap the mainloop of tile t+1.
// Every mbarrier wait is bounded; on expiry the CTA records JA_ERR_TIMEOUT, drains its copies and exits.
//
// The kernel exists in two forms (template parameter CG):
//   CG = 1  one CTA per 128 x 256 tile, tcgen05.mma.cta_group::1.
//   CG = 2  a cluster of two CTAs (two SMs) per 256 x 256 tile, tcgen05.mma.cta_group::2 issued by the leader
//           CTA: each CTA stages its own 128 rows of A and its own half of the tile's B columns (plain TMA
//           loads, no multicast), so every SM pulls a third less operand data per flop through L2 and can
//           keep six stages in flight; each CTA holds the accumulator rows of its own half in its own TMEM.
#include <cuda.h>
#include <stdlib.h>
#include <string.h>

#include "ja_device.cuh"
#include "ja_ptx.cuh"

namespace {

using namespace ja_ptx;

constexpr int BM = 128, BN = 256;
constexpr int NUM_THREADS = 192;
// BK = contraction depth of one pipeline stage. The two-CTA form stages 128-deep chunks so that every box it issues
// (A: 128 rows x 64 k, B: 128 k x 64 columns) is 16 KiB: fewer, larger TMA copies per flop than 64-deep stages.
// What bounds this kernel is operand delivery, not the tensor pipe: timing-only ablations on [16384, 4096] x [4096, 4096]
// with half of the B boxes not loaded ran at 1617 TFLOP/s against 1391, with half of A as well at 1821. A form that cuts
// the bytes per flop by a quarter -- tiles of 256 x 512 on both accumulators, A fetched once per 512 columns -- was built,
// passed the parity tests and measured SLOWER, because the shared memory left holds either four 64-deep stages of 8 KiB
// B boxes (1196 TFLOP/s on the same product) or two 128-deep stages (1339; 1205 against 1330-1418 on the up-projections):
// more, smaller copies or too shallow a pipeline cost more than the saved bytes bring.
template <int CG> struct Cfg {
    static constexpr int BK = CG == 1 ? 64 : 128;
    static constexpr int STAGES = CG == 1 ? 4 : 3;
    static constexpr int A_HALF_BYTES = BM * 64 * 2;                 // 128 rows x 64 k under the 128-byte swizzle
    static constexpr int A_STAGE_BYTES = A_HALF_BYTES * (BK / 64);
    static constexpr int B_CHUNK_BYTES = BK * 64 * 2;                // one box: BK k-rows x 64 columns
    static constexpr int B_STAGE_BYTES = B_CHUNK_BYTES * (BN / CG / 64);
    static constexpr int SMEM_BYTES = STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + 1024 /*align*/ + 256 /*barriers*/;
};

struct GemmParams {
    char* c_base;
    const int64_t* c_blk_off;  // device: byte offsets of the output blocks
    int32_t* status;           // status word of the launching stream (set at launch)
    uint32_t wait_cap_us;      // limit of every bounded wait (set at launch)
    int32_t bm, bk, bn;        // block extents along i, j, k
    int32_t nbm, nbk, nbn;     // blocks along i, j, k
    int32_t M, N;              // tensor extents along i, k
    int32_t a_box_rows;        // rows per A box (= min(bm, 128))
    int32_t m_tiles, n_tiles;  // tile grid (tiles are 128*CG rows x up to 256 columns)
    int32_t tiles_per_mblk;    // >= 1 when row tiles never leave a block, 0 when tiles are cut from global rows
    int32_t tiles_per_nblk;    // >= 1 when tiles stay inside one column block, 0 when tiles span blocks
    int32_t group_m;           // row tiles per rasterisation band
    int32_t heavy_first;       // 1: full-width tiles are scheduled before the narrow last tile of every column block (see tile_of_iter)
    // fused epilogue (a join-agg chain executed in one pass, the intermediate never stored)
    int32_t epi;               // EPI_*
    int32_t bn_tile;           // output columns per tile: 256, or 128 for EPI_SWIGLU (two 128-column products per tile)
    int32_t n_copies;          // 1: SUM over all contracted blocks (aggregated output). nbk: join only -- tile (c, ., .) covers the
                               // single contracted block c and is stored to copy c of a partial relation [c, i, k]
    int32_t c_esize;           // bytes per output cell: 2 (bf16 / f16) or 4 (f32, partial relations only)
    int32_t f16;               // cell type of the operands (and of a 2-byte output): 0 = bf16, 1 = f16
    const char* r_base;        // EPI_ADD: payload of the relation added to the product (tiled exactly like the output)
    const float2* rope_table;  // EPI_ROPE: (cos, sin)[position][pair]
    int32_t rope_S, rope_D;    // EPI_ROPE: positions per sequence (row % rope_S), rotated extent (column % rope_D)
};
enum { EPI_NONE = 0, EPI_ADD = 1, EPI_ROPE = 2, EPI_SWIGLU = 3 };

// What one CTA does for one tile: its own 128 rows, and (CG 2) its own half of the tile's columns as B operand.
struct TileCoord {
    int mb, r0;          // row block and first row inside it of THIS CTA's 128 rows
    int row_g0;          // first global row of this CTA's rows
    int rows;            // valid rows (0..128)
    int n_g0, nb, c0;    // first global column of the tile / its column block / first column inside it
    int width;           // valid columns of the tile (multiple of 8)
    int jb0, jb1;        // contracted blocks [jb0, jb1) accumulated into this tile
    int copy;            // copy index of a partial relation (0 for an aggregated output)
};

template <int CG>
__device__ __forceinline__ TileCoord tile_coord(const GemmParams& p, int t, int cta_rank) {
    TileCoord tc;
    // join-only form: copies are the slowest tile coordinate, so tiles in flight share one contracted block
    const int per_copy = p.m_tiles * p.n_tiles;
    tc.copy = t / per_copy;
    t -= tc.copy * per_copy;
    tc.jb0 = p.n_copies > 1 ? tc.copy : 0;
    tc.jb1 = p.n_copies > 1 ? tc.copy + 1 : p.nbk;
    // heavy-first schedule: t counts the full-width tiles of all column blocks first, then the narrow last tiles
    int n_tiles_v = p.n_tiles;
    bool narrow = false;
    if (p.heavy_first) {
        const int full_tiles = p.m_tiles * p.nbn * (p.tiles_per_nblk - 1);
        narrow = t >= full_tiles;
        if (narrow) t -= full_tiles;
        n_tiles_v = narrow ? p.nbn : p.nbn * (p.tiles_per_nblk - 1);
    }
    // banded rasterisation: tiles that run at the same time cover group_m row tiles x several column tiles, so the
    // operand strips they stream fit in L2 together. (A second level -- super-columns of column tiles whose B strip would
    // stay in L2 while every row band passes over it -- was built and measured on the block's projections: launch times
    // within 1 % of this order for strips of 16 to 48 tiles, and MORE DRAM traffic, 1.9-2.5 GB against 1.7 GB per
    // up-projection launch, so it is not here.)
    const int band_sz = p.group_m * n_tiles_v;
    const int band = t / band_sz, tin = t - band * band_sz;
    const int rows_in_band = min(p.group_m, p.m_tiles - band * p.group_m);
    const int mt = band * p.group_m + tin % rows_in_band;
    int nt = tin / rows_in_band;
    if (p.heavy_first) nt = narrow ? nt * p.tiles_per_nblk + p.tiles_per_nblk - 1 : (nt / (p.tiles_per_nblk - 1)) * p.tiles_per_nblk + nt % (p.tiles_per_nblk - 1);
    if (p.tiles_per_mblk > 0) {   // CG == 1 only: row tiles stay inside a block
        tc.mb = mt / p.tiles_per_mblk;
        tc.r0 = (mt % p.tiles_per_mblk) * BM;
        tc.rows = min(BM, p.bm - tc.r0);
        tc.row_g0 = tc.mb * p.bm + tc.r0;
    } else {                      // tiles cut from global rows (block height divides 128, or is a multiple of 128)
        tc.row_g0 = mt * (BM * CG) + cta_rank * BM;
        tc.mb = tc.row_g0 / p.bm;
        tc.r0 = tc.row_g0 % p.bm;
        tc.rows = max(0, min(BM, p.M - tc.row_g0));
    }
    if (p.tiles_per_nblk > 0) {
        tc.nb = nt / p.tiles_per_nblk;
        tc.c0 = (nt % p.tiles_per_nblk) * p.bn_tile;
        tc.width = min(p.bn_tile, p.bn - tc.c0);
        tc.n_g0 = tc.nb * p.bn + tc.c0;
    } else {
        tc.n_g0 = nt * p.bn_tile;
        tc.nb = tc.n_g0 / p.bn;
        tc.c0 = tc.n_g0 % p.bn;
        tc.width = min(p.bn_tile, p.N - tc.n_g0);
    }
    return tc;
}

// Which tile a CTA group works on in its i-th round, or -1 when it has none left. Plain round-robin, or -- with the heavy-first
// order, where tiles come sorted by weight -- round-robin that reverses direction every round, so that the groups that got an
// extra full tile in the last full-width round are the last to be handed narrow ones.
__device__ __forceinline__ int tile_of_iter(const GemmParams& p, int i, int first, int step, int total) {
    const int t = i * step + ((p.heavy_first && (i & 1)) ? step - 1 - first : first);
    return t < total ? t : -1;
}

// F16: cell type of the operands and of a 2-byte output -- bf16 or f16 (a compile-time choice: a select between the two
// conversions in the epilogue cost the plain contraction a tenth of its rate)
template <int CG, bool F16>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmB2, const GemmParams p) {
    constexpr int STAGES = Cfg<CG>::STAGES, BK = Cfg<CG>::BK;
    constexpr int A_STAGE_BYTES = Cfg<CG>::A_STAGE_BYTES, A_HALF_BYTES = Cfg<CG>::A_HALF_BYTES;
    constexpr int B_STAGE_BYTES = Cfg<CG>::B_STAGE_BYTES, B_CHUNK_BYTES = Cfg<CG>::B_CHUNK_BYTES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // swizzle atoms need 1024-byte alignment
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t sA = base, sB = base + STAGES * A_STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * (A_STAGE_BYTES + B_STAGE_BYTES));
    // bars[0..S) full, [S..2S) empty, [2S..2S+2) tmem_full, [2S+2..2S+4) tmem_empty
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x / 32, 0), lane = threadIdx.x % 32;   // warp-uniform by construction
    const int cta_rank = CG == 2 ? (int)cluster_ctarank() : 0;   // 0 = leader of the pair
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);    // CG 2: only the leader's is used; both CTAs' copies complete_tx on it
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), 4 * CG);  // one arrival per epilogue warp of every CTA of the group
        }
        wait_ctl_init(abort_flag, p.wait_cap_us);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // all 512 TMEM columns: two 128 x 256 fp32 accumulators (in each CTA of a pair)
        if (CG == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();   // the peer's barriers exist before anything remote touches them
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);

    const int total_tiles = p.m_tiles * p.n_tiles * p.n_copies;
    const int kchunks = (p.bk + Cfg<CG>::BK - 1) / Cfg<CG>::BK;
    const int first_tile = blockIdx.x / CG, tile_step = gridDim.x / CG;

    if (warp == 0) {
        // ================= TMA producer (one per CTA) =================
        if (lane == 0) {
            uint32_t last_parity[STAGES];
            bool issued[STAGES];
            for (int s = 0; s < STAGES; ++s) { last_parity[s] = 0; issued[s] = false; }
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int it = 0; ok; ++it) {
                const int t = tile_of_iter(p, it, first_tile, tile_step, total_tiles);
                if (t < 0) break;
                const TileCoord tc = tile_coord<CG>(p, t, cta_rank);
                // EPI_SWIGLU: the MMA tile is [128 columns of x W1 | the same 128 columns of x W3]
                const int n_mma = p.epi == EPI_SWIGLU ? 2 * tc.width : (tc.width + 15) / 16 * 16;
                const int my_cols = n_mma / CG;                    // B columns this CTA stages
                const int my_c0 = cta_rank * my_cols;              // their offset inside the tile
                const int nchunks = (my_cols + 63) / 64;
                const uint32_t tx = (uint32_t)CG * (A_STAGE_BYTES + nchunks * B_CHUNK_BYTES);
                for (int jb = tc.jb0; jb < tc.jb1 && ok; ++jb) {    // the tuples of this output key, ascending j
                    for (int kc = 0; kc < kchunks; ++kc) {
                        if (!mbar_wait(empty_bar(stage), phase ^ 1, abort_flag, p.status)) { ok = false; break; }
                        uint32_t fb = full_bar(stage);
                        if (CG == 2) fb = mapa_cluster(fb, 0);      // completion is counted on the leader's barrier
                        if (cta_rank == 0) mbar_expect_tx(full_bar(stage), tx);
                        issued[stage] = true;
                        last_parity[stage] = phase;
                        // A: boxes of a_box_rows rows x 64 k, one set per 64-deep half of the stage
                        const int nboxes = BM / p.a_box_rows;
                        for (int kh = 0; kh < BK / 64; ++kh)
                            for (int bx = 0; bx < nboxes; ++bx)
                                tma_load_4d<CG>(sA + stage * A_STAGE_BYTES + kh * A_HALF_BYTES + bx * p.a_box_rows * 128, &tmA, fb,
                                                kc * BK + kh * 64, tc.r0, jb, tc.mb + bx);
                        // B: one box of BK k-rows x 64 columns per 64-column chunk
                        for (int c = 0; c < nchunks; ++c) {
                            int mc = my_c0 + 64 * c;               // column of the MMA tile this box starts at
                            const CUtensorMap* tb = &tmB;
                            if (p.epi == EPI_SWIGLU && mc >= p.bn_tile) { tb = &tmB2; mc -= p.bn_tile; }
                            int nb, cin;
                            if (p.tiles_per_nblk > 0) { nb = tc.nb; cin = tc.c0 + mc; }
                            else { int g = tc.n_g0 + mc; nb = g / p.bn; cin = g % p.bn; }
                            tma_load_4d<CG>(sB + stage * B_STAGE_BYTES + c * B_CHUNK_BYTES, tb, fb, cin, kc * BK, nb, jb);
                        }
                        if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    }
                }
            }
            // drain: wait (bounded) for copies already in flight before the CTA may exit. In a pair both CTAs' copies
            // complete on the leader's barriers, and the peer cannot leave before the leader reaches the cluster barrier.
            if (!ok && cta_rank == 0) {
                for (int s = 0; s < STAGES; ++s) {
                    if (!issued[s]) continue;
                    const uint64_t t0 = global_ns();
                    while (!mbar_try_wait(full_bar(s), last_parity[s]) && global_ns() - t0 < 200000000ull) {}
                }
            }
            (void)issued; (void)last_parity;
        }
    } else if (warp == 1) {
        // ================= MMA issuer (leader CTA only): the whole warp runs the loop, one elected lane issues =================
        if (cta_rank == 0) {
            const uint32_t leader = elect_one();
            int stage = 0;
            uint32_t phase = 0;
            uint32_t acc_phase[2] = {0, 0};
            bool ok = true;
            for (int it = 0; ok; ++it) {
                const int t = tile_of_iter(p, it, first_tile, tile_step, total_tiles);
                if (t < 0) break;
                const TileCoord tc = tile_coord<CG>(p, t, 0);
                const int acc = it & 1;
                const uint32_t n_mma = p.epi == EPI_SWIGLU ? (uint32_t)(2 * tc.width) : (uint32_t)((tc.width + 15) / 16 * 16);
                // D f32; A and B both bf16 (format 1) or both f16 (format 0); B MN-major
                constexpr uint32_t fmt = F16 ? 0u : 1u;
                const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | (1u << 16) | ((n_mma >> 3) << 17) |
                                       ((uint32_t)((BM * CG) >> 4) << 24);
                if (!mbar_wait(tempty_bar(acc), acc_phase[acc] ^ 1, abort_flag, p.status)) { ok = false; break; }
                acc_phase[acc] ^= 1;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                uint32_t accumulate = 0;
                for (int jb = tc.jb0; jb < tc.jb1 && ok; ++jb) {
                    for (int kc = 0; kc < kchunks; ++kc) {
                        if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status)) { ok = false; break; }
                        tc_fence_after();
                        const int kvalid = min(BK, p.bk - kc * BK);
                        const int k16 = (kvalid + 15) / 16;
                        const uint32_t a_addr = sA + stage * A_STAGE_BYTES;
                        const uint32_t b_addr = sB + stage * B_STAGE_BYTES;
                        // A: K-major, 16 k = 32 bytes inside the swizzle atom, 64 k per half; B: MN-major, 16 k-rows =
                        // 2048 bytes, 64-column groups BK*128 bytes apart
                        if (k16 == BK / 16) {   // a full stage: straight-line code, no branch between two tcgen05.mma
#pragma unroll
                            for (int kk = 0; kk < BK / 16; ++kk) {
                                const uint64_t da = desc_sw128(a_addr + (kk >> 2) * A_HALF_BYTES + (kk & 3) * 32, 16);
                                const uint64_t db = desc_sw128(b_addr + kk * 2048, BK * 128);
                                umma_bf16_w<CG>(d_tmem, da, db, idesc, kk > 0 ? 1u : accumulate, leader);
                            }
                        } else {
                            for (int kk = 0; kk < k16; ++kk) {
                                const uint64_t da = desc_sw128(a_addr + (kk >> 2) * A_HALF_BYTES + (kk & 3) * 32, 16);
                                const uint64_t db = desc_sw128(b_addr + kk * 2048, BK * 128);
                                umma_bf16_w<CG>(d_tmem, da, db, idesc, kk > 0 ? 1u : accumulate, leader);
                            }
                        }
                        accumulate = 1;
                        umma_commit_w<CG>(empty_bar(stage), leader);  // frees the smem stage (in both CTAs) once these MMAs have read it
                        if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    }
                }
                if (ok) umma_commit_w<CG>(tfull_bar(acc), leader);    // accumulator complete -> epilogue(s)
            }
        }
    } else {
        // ================= epilogue (warps 2..5 of every CTA) =================
        const int q = warp & 3;  // TMEM lane group this warp may access
        uint32_t acc_phase[2] = {0, 0};
        bool ok = true;
        const uint32_t tempty0 = CG == 2 ? mapa_cluster(tempty_bar(0), 0) : tempty_bar(0);
        const uint32_t tempty1 = CG == 2 ? mapa_cluster(tempty_bar(1), 0) : tempty_bar(1);
        for (int it = 0; ok; ++it) {
            const int t = tile_of_iter(p, it, first_tile, tile_step, total_tiles);
            if (t < 0) break;
            const TileCoord tc = tile_coord<CG>(p, t, cta_rank);
            const int acc = it & 1;
            if (!mbar_wait(tfull_bar(acc), acc_phase[acc], abort_flag, p.status)) { ok = false; break; }
            acc_phase[acc] ^= 1;
            tc_fence_after();
            const int r = q * 32 + lane;                     // row of this CTA's 128 rows held by this thread
            const int grow = tc.row_g0 + r;                  // global row
            const bool row_ok = r < tc.rows;
            int ib = 0, iin = 0;
            if (row_ok) { ib = grow / p.bm; iin = grow % p.bm; }
            for (int ch = 0; ch * 32 < tc.width; ++ch) {
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + ch * 32, v);
                if (p.epi == EPI_SWIGLU) {   // silu(x W1) * (x W3): the W3 product sits 128 columns to the right
                    uint32_t w[32];
                    tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN + p.bn_tile + ch * 32, w);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float a = __uint_as_float(v[i]);
                        v[i] = __float_as_uint(a / (1.f + __expf(-a)) * __uint_as_float(w[i]));
                    }
                } else {
                    tmem_ld_wait();
                }
                if (row_ok) {
                    const int gcol = tc.n_g0 + ch * 32;
                    const int kb = gcol / p.bn, cin = gcol % p.bn;
                    const int64_t off = p.c_blk_off[((int64_t)tc.copy * p.nbm + ib) * p.nbn + kb] + ((int64_t)iin * p.bn + cin) * p.c_esize;
                    char* dst = p.c_base + off;
                    const int valid = min(32, tc.width - ch * 32);  // multiple of 8
                    if (p.c_esize == 4) {   // partial relation kept in f32: the accumulator is stored as it is
#pragma unroll
                        for (int g = 0; g < 8; ++g)
                            if (g * 4 < valid)
                                *reinterpret_cast<uint4*>(dst + g * 16) = make_uint4(v[g * 4], v[g * 4 + 1], v[g * 4 + 2], v[g * 4 + 3]);
                        continue;
                    }
                    if (p.epi == EPI_ROPE) {
                        // rotate pairs (2p, 2p+1) by the angle of (position, pair): position = row inside its sequence
                        const float2* tab = p.rope_table + ((int64_t)(grow % p.rope_S) * p.rope_D + gcol % p.rope_D) / 2;
#pragma unroll
                        for (int i = 0; i < 32; i += 2) {
                            const float2 cs = tab[i / 2];
                            const float x0 = __uint_as_float(v[i]), x1 = __uint_as_float(v[i + 1]);
                            v[i] = __float_as_uint(x0 * cs.x - x1 * cs.y);
                            v[i + 1] = __float_as_uint(x0 * cs.y + x1 * cs.x);
                        }
                    }
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        if (g * 8 < valid) {
                            float f[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[g * 8 + e]);
                            if (p.epi == EPI_ADD) {   // key-aligned join with the addend relation: same block, same cell
                                const uint4 rv = *reinterpret_cast<const uint4*>(p.r_base + off + g * 16);
                                const uint32_t* pr = reinterpret_cast<const uint32_t*>(&rv);
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float2 rf = ja_unpack16<F16>(pr[e]);
                                    f[2 * e] += rf.x;
                                    f[2 * e + 1] += rf.y;
                                }
                            }
                            uint4 o;
                            uint32_t* po = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                            for (int e = 0; e < 4; ++e) po[e] = ja_pack16<F16>(f[2 * e], f[2 * e + 1]);
                            *reinterpret_cast<uint4*>(dst + g * 16) = o;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (CG == 1) mbar_arrive(acc ? tempty1 : tempty0);
                else mbar_arrive_cluster(acc ? tempty1 : tempty0);   // the leader's MMA thread owns the accumulators of both CTAs
            }
        }
    }
    // ---- teardown ---------------------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();   // nobody leaves while the peer may still signal its barriers or read its smem
    if (warp == 1) {
        tc_fence_after();
        if (CG == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

// ---- host: tensor maps -------------------------------------------------------------------------------------
// A relation [R, C] with equal blocks br x bc is the rank-4 tensor (c in block, r in block, col-block, row-block).
ja_status_t encode_blocked_2d(const ja_relation* r, int box_inner, int box_rows, CUtensorMap* tm) {
    if (box_rows > 256) return ja_fail(JA_ERR_INVALID_ARG, "TMA box too tall");
    EncodeTiledFn enc = get_encode();
    if (!enc) return ja_fail(JA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const int64_t br = r->bs[0], bc = r->bs[1];
    const int64_t blk_stride = r->nblocks > 1 ? r->blk_off[1] - r->blk_off[0] : (int64_t)r->bytes;
    cuuint64_t dims[4] = {(cuuint64_t)bc, (cuuint64_t)br, (cuuint64_t)r->nblk[1], (cuuint64_t)r->nblk[0]};
    cuuint64_t strides[3] = {(cuuint64_t)(bc * 2), (cuuint64_t)blk_stride, (cuuint64_t)(blk_stride * r->nblk[1])};
    cuuint32_t box[4] = {(cuuint32_t)box_inner, (cuuint32_t)box_rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUtensorMapDataType cell = r->dtype == JA_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    CUresult res = enc(tm, cell, 4, r->base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                       CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (res != CUDA_SUCCESS) return ja_fail(JA_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)res);
    return JA_OK;
}

}  // namespace

struct GemmTcPlan {
    CUtensorMap tmA, tmB, tmB2;
    GemmParams p;
    int grid;
    int cg;   // CTAs per tile: 1 or 2
};

ja_status_t ja_gemm_tc_plan(const ja_relation* A, const ja_relation* B, const ja_relation* C, const GemmEpilogue* ep,
                            std::shared_ptr<GemmTcPlan>* out, bool* eligible) {
    *eligible = false;
    if (!A->equal_blocks || !B->equal_blocks || !C->equal_blocks) return JA_OK;
    if (A->dtype == JA_F32 || B->dtype != A->dtype || (C->esize == 2 && C->dtype != A->dtype)) return JA_OK;
    const int epi = ep ? ep->epi : 0;
    const int bn_tile = epi == EPI_SWIGLU ? 128 : BN;
    if (epi == EPI_SWIGLU && (B->bs[1] % 128 != 0 || !ep->B2 || !ep->B2->equal_blocks)) return JA_OK;
    if (epi == EPI_ROPE && (ep->rope_D % 32 != 0 || B->bs[1] % 32 != 0)) return JA_OK;
    const int64_t bm = A->bs[0], bk = A->bs[1], bn = B->bs[1];
    // TMA needs 16-byte row pitches; boxes are 64 elements wide; A boxes hold min(bm,128) rows
    if (bk % 8 || bn % 8 || bk < 64 || bn < 64) return JA_OK;
    if (bm < 128 && (128 % bm != 0 || bm % 8 != 0)) return JA_OK;
    if (A->extent[0] >= (1ll << 31) || B->extent[1] >= (1ll << 31)) return JA_OK;
    std::shared_ptr<GemmTcPlan> plan(new GemmTcPlan());
    GemmParams& p = plan->p;
    p.c_base = (char*)C->base;
    p.c_blk_off = ja_view(C).blk_off;
    p.status = nullptr;
    p.bm = (int)bm; p.bk = (int)bk; p.bn = (int)bn;
    p.nbm = A->nblk[0]; p.nbk = A->nblk[1]; p.nbn = B->nblk[1];
    p.M = (int)A->extent[0]; p.N = (int)B->extent[1];
    p.a_box_rows = (int)std::min<int64_t>(bm, 128);
    p.epi = epi;
    p.bn_tile = bn_tile;
    p.n_copies = (ep && ep->partials) ? p.nbk : 1;
    p.c_esize = C->esize;
    p.f16 = A->dtype == JA_F16;
    if (p.c_esize == 4 && !(ep && ep->partials)) return JA_OK;
    p.r_base = (epi == EPI_ADD) ? (const char*)ep->addend->base : nullptr;
    p.rope_table = (epi == EPI_ROPE) ? ep->rope_table : nullptr;
    p.rope_S = ep ? ep->rope_S : 1;
    p.rope_D = ep ? ep->rope_D : 2;
    if (bn % 64 == 0 && bn < bn_tile && p.nbn > 1) { p.tiles_per_nblk = 0; p.n_tiles = (p.N + bn_tile - 1) / bn_tile; }
    else { p.tiles_per_nblk = (int)((bn + bn_tile - 1) / bn_tile); p.n_tiles = p.tiles_per_nblk * p.nbn; }
    // Two-CTA form: 256-row tiles cut from global rows; needs 128-row halves that never straddle a block and, when
    // tiles span column blocks, column tails whose halves still start on a 64-column box boundary.
    // narrow last tile in every column block (block width not a multiple of the tile width): schedule it after the full tiles
    const JaConfig& cfg = ja_config();
    p.heavy_first = (p.n_copies == 1 && p.tiles_per_nblk > 1 && bn % bn_tile != 0 && cfg.gemm_heavy_first != 0) ? 1 : 0;
    p.group_m = cfg.gemm_group_m >= 1 ? cfg.gemm_group_m : 8;
    bool two = (bm % 128 == 0 || 128 % bm == 0) && p.M >= 256 && bk >= Cfg<2>::BK;
    if (p.tiles_per_nblk == 0 && (p.N % bn_tile) % (bn_tile / 2) != 0) two = false;
    if (cfg.gemm_cta_group == 1) two = false;
    plan->cg = two ? 2 : 1;
    if (two || bm < 128) { p.tiles_per_mblk = 0; p.m_tiles = (p.M + BM * plan->cg - 1) / (BM * plan->cg); }
    else { p.tiles_per_mblk = (int)((bm + BM - 1) / BM); p.m_tiles = p.tiles_per_mblk * p.nbm; }
    ja_status_t st;
    if ((st = encode_blocked_2d(A, 64, p.a_box_rows, &plan->tmA)) != JA_OK) return st;
    if ((st = encode_blocked_2d(B, 64, two ? Cfg<2>::BK : Cfg<1>::BK, &plan->tmB)) != JA_OK) return st;
    plan->tmB2 = plan->tmB;
    if (epi == EPI_SWIGLU && (st = encode_blocked_2d(ep->B2, 64, two ? Cfg<2>::BK : Cfg<1>::BK, &plan->tmB2)) != JA_OK) return st;
    const int sms = ja_sm_count();
    const int tiles = p.m_tiles * p.n_tiles * p.n_copies;
    plan->grid = two ? 2 * std::min(sms / 2, tiles) : std::min(sms, tiles);
    cudaError_t e;
    if (p.f16)
        e = two ? cudaFuncSetAttribute(gemm_tc_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<2>::SMEM_BYTES)
                : cudaFuncSetAttribute(gemm_tc_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<1>::SMEM_BYTES);
    else
        e = two ? cudaFuncSetAttribute(gemm_tc_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<2>::SMEM_BYTES)
                : cudaFuncSetAttribute(gemm_tc_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<1>::SMEM_BYTES);
    if (e != cudaSuccess) return ja_cuda_fail(e, "cudaFuncSetAttribute(gemm_tc_kernel)");
    *out = plan;
    *eligible = true;
    return JA_OK;
}

ja_status_t ja_launch_gemm_tc(const GemmTcPlan& plan, cudaStream_t st) {
    GemmParams p = plan.p;
    p.status = ja_device_status_word(st);
    if (!p.status) return ja_fail(JA_ERR_CUDA, "cannot resolve the device status word");
    p.wait_cap_us = (uint32_t)ja_config().wait_cap_us;
    if (plan.cg == 2) {
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3((unsigned)plan.grid, 1, 1);
        cfg.blockDim = dim3(NUM_THREADS, 1, 1);
        cfg.dynamicSmemBytes = Cfg<2>::SMEM_BYTES;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (p.f16) JA_CUDA(cudaLaunchKernelEx(&cfg, gemm_tc_kernel<2, true>, plan.tmA, plan.tmB, plan.tmB2, p));
        else JA_CUDA(cudaLaunchKernelEx(&cfg, gemm_tc_kernel<2, false>, plan.tmA, plan.tmB, plan.tmB2, p));
    } else {
        if (p.f16) gemm_tc_kernel<1, true><<<plan.grid, NUM_THREADS, Cfg<1>::SMEM_BYTES, st>>>(plan.tmA, plan.tmB, plan.tmB2, p);
        else gemm_tc_kernel<1, false><<<plan.grid, NUM_THREADS, Cfg<1>::SMEM_BYTES, st>>>(plan.tmA, plan.tmB, plan.tmB2, p);
        JA_CUDA(cudaGetLastError());
    }
    ja_count_launch();
    return JA_OK;
}
