// Internal declarations of libja (host bookkeeping + kernel launchers). Not part of the C ABI.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <map>
#include <memory>
#include <mutex>
#include <string>
#include <vector>

#include "ja.h"

#define JA_MAX_RANK 4
#define JA_MAX_IN 4
#define JA_ALIGN 128
#define JA_MAX_SEQ 16      // packed sequences per attention spec

// ---- device-side view of a tensor relation (passed to kernels by value) -------------------------
// Key table on the device: per-dimension split points and per-block byte offsets. A kernel turns a
// tensor coordinate into (block key, offset inside the block) with these and nothing else.
struct RelView {
    char* base;                          // payload
    const int64_t* splits[JA_MAX_RANK];  // device; splits[d][0..nblk[d]]
    const int64_t* blk_off;              // device; byte offset of every block, row-major key order
    int64_t extent[JA_MAX_RANK];
    int64_t bs[JA_MAX_RANK];             // uniform block size of dimension d, or 0 if irregular
    int64_t blk_stride;                  // bytes between consecutive blocks when all blocks have one shape, else 0
    int32_t nblk[JA_MAX_RANK];
    int32_t rank;
    int32_t esize;
};

struct ja_relation {
    int32_t rank = 0;
    int64_t extent[JA_MAX_RANK] = {0, 0, 0, 0};
    int32_t nblk[JA_MAX_RANK] = {1, 1, 1, 1};
    std::vector<int64_t> splits[JA_MAX_RANK];
    int64_t bs[JA_MAX_RANK] = {0, 0, 0, 0};
    ja_dtype_t dtype = JA_BF16;
    int32_t esize = 2;
    void* base = nullptr;
    size_t bytes = 0;         // payload size implied by the tiling
    int64_t nblocks = 0;
    std::vector<int64_t> blk_off;  // bytes
    bool equal_blocks = false;     // every block has the same shape (constant block stride)
    uint64_t id = 0;
    // lazily created device copies of the key table
    mutable int64_t* d_tables = nullptr;
    mutable bool on_device = false;
};

struct ExecPlan;  // per (spec, relations) cached launch state

struct ja_spec {
    std::string einsum;
    std::vector<std::string> ins;
    std::string out;
    std::string letters;  // order of first appearance
    std::vector<std::vector<int64_t>> parts;  // per letter: split points
    ja_fn_t fn = JA_FN_MUL;
    ja_agg_t agg = JA_AGG_SUM;
    std::vector<double> params;
    int64_t p = 0;
    std::vector<int32_t> in_keys;   // [p][n_in]
    std::vector<int32_t> out_keys;  // [p]
    // launch state cached per tuple of relation ids; guarded by plans_mu (ja_execute may be called from several threads
    // on one spec); entries that name a destroyed relation are dropped by ja_relation_destroy
    mutable std::mutex plans_mu;
    mutable std::map<std::vector<uint64_t>, std::shared_ptr<ExecPlan>> plans;
};

// ---- helpers implemented in ja_host.cu ------------------------------------------------------------
ja_status_t ja_fail(ja_status_t st, const char* fmt, ...);
ja_status_t ja_cuda_fail(cudaError_t e, const char* what);
ja_status_t ja_relation_to_device(const ja_relation* r);
RelView ja_view(const ja_relation* r);
// The status word of (current device, stream): a fixed table of words per device, one per stream seen so far (the 64th and
// later streams of a device share the last word). nullptr when the table's address cannot be resolved.
int* ja_device_status_word(cudaStream_t st);
void ja_count_launch(int n = 1);
int ja_sm_count();   // multiprocessors of the current device (cached per device)

// Switches that force a kernel form or a schedule. Read ONCE from the environment (JA_* variables) when the library is
// first used; afterwards only ja_debug_set changes them (tests, A/B measurements). -1 = not forced.
struct JaConfig {
    int attn_mma_sync = -1;     // JA_ATTN_MMA_SYNC     1: the mma.sync attention kernel
    int attn_one_tile = -1;     // JA_ATTN_ONE_TILE     1: one query tile per CTA
    int attn_persistent = -1;   // JA_ATTN_PERSISTENT   0 / 1: work items drawn from a counter by one CTA per SM
    int attn_section = -1;      // JA_ATTN_SECTION      n: launch-order sections of n (batch, head) pairs
    int attn_variant = -1;      // JA_ATTN_VARIANT      row-thread variant of the two-tile kernel (see k_attention_tc.cu)
    int gemm_cta_group = -1;    // JA_GEMM_CTA_GROUP    1: no two-CTA pairs
    int gemm_group_m = -1;      // JA_GEMM_GROUP_M      n: row tiles per rasterisation band
    int gemm_heavy_first = -1;  // JA_GEMM_HEAVY_FIRST  0: plain tile order
    int gemm_split = -1;        // JA_GEMM_SPLIT        0: the last partial wave is not split along the contracted index
    int gemm_loader = -1;       // JA_GEMM_LOADER       1: operands staged by plain loads even where TMA could take them; 0: never
    int row_tma = -1;           // JA_ROW_TMA           0: row join-aggs without the TMA-staged kernel
    int row_team = -1;          // JA_ROW_TEAM          n: threads per row of the plain row kernel
    int row_reduce = -1;        // JA_ROW_REDUCE        0: statistics-only row forms never take the plain read-stream kernel, 1: whenever the tiling fits
    int64_t wait_cap_us = 2000000;   // JA_WAIT_CAP (nanoseconds in the environment): limit of every device-side wait
};
JaConfig& ja_config();

#define JA_CUDA(call)                                              \
    do {                                                           \
        cudaError_t e_ = (call);                                   \
        if (e_ != cudaSuccess) return ja_cuda_fail(e_, #call);     \
    } while (0)

// ---- kernel launchers (one per .cu file) ------------------------------------------------------------
// Plain-ALU tiled matmul join-agg over arbitrary tilings (f32 or bf16 operands, f32 accumulate). The key tables of the
// three relations must be on the device (ja_relation_to_device).
// the definition in its relational form, one thread per output cell: any spec whose operator is a scalar function of the
// joined cells (*launched stays false otherwise)
ja_status_t ja_launch_generic(const ja_spec* spec, const ja_relation* const* inputs, const ja_relation* out, cudaStream_t st, bool* launched);
ja_status_t ja_launch_matmul_simt(const ja_relation* A, const ja_relation* B, const ja_relation* C, cudaStream_t st,
                                  bool partials = false);

// tcgen05 matmul join-agg for bf16 relations under any tiling, operands staged by plain loads (k_gemm_ld.cu); *launched
// stays false when the blocks are too small for its tiles. Key tables must be on the device.
ja_status_t ja_launch_gemm_ld(const ja_relation* A, const ja_relation* B, const ja_relation* C, cudaStream_t st, bool* launched);

// Memory-bound join-aggs: flat key-aligned maps and row-structured maps / reductions.
enum RowOp {
    ROW_SUMSQ = 0, ROW_MAX, ROW_EXPSUM, ROW_RMS_SCALE, ROW_EXP_SUB_DIV, ROW_RMSNORM, ROW_SOFTMAX, ROW_ROPE
};
struct RowArgs {
    RelView x;     // [R..., j] input
    RelView s0;    // statistics relation keyed by R (ss or m) -- input or output depending on op
    RelView s1;    // second statistics relation (l)
    RelView g;     // [j] gain vector
    RelView y;     // [R..., j] output
    float eps;     // RMS_SCALE / RMSNORM
    float theta;   // ROPE
    const float2* rope_table;  // device [extent(s)][d/2] (cos, sin)
    int rope_d;                // extent of the rotated index d (rows may hold several heads of d cells each)
};
ja_status_t ja_launch_row(RowOp op, const RowArgs& a, ja_dtype_t dt, cudaStream_t st);
// bulk-copy pipelined form for uniform tilings; *launched stays false when the shape does not fit it
ja_status_t ja_launch_row_tma(RowOp op, const RowArgs& a, ja_dtype_t dt, cudaStream_t st, bool* launched);
// statistics-only forms (sum of squares, row maximum, sum of exponentials) as a plain read stream; *launched as above
ja_status_t ja_launch_row_reduce(RowOp op, const RowArgs& a, ja_dtype_t dt, cudaStream_t st, bool* launched);
ja_status_t ja_launch_flat(ja_fn_t fn, const void* a, const void* b, void* out, int64_t n_elems, ja_dtype_t dt,
                           cudaStream_t st);

// Repartition: list of 2-D slab copies.
struct CopySlab {
    int64_t src_off, dst_off;        // bytes
    int32_t rows, row_bytes;         // slab shape
    int32_t src_pitch, dst_pitch;    // bytes between consecutive rows
};
ja_status_t ja_launch_repartition(const char* src, char* dst, const CopySlab* d_slabs, int64_t n_slabs, int vec_bytes,
                                  cudaStream_t st);
// Aggregating relayout: every slab is read from n_copies copies of the source, copy_stride bytes apart, (+)-combined
// in ascending copy order in f32 and stored once. Slab sizes are in SOURCE bytes; destination offsets / pitches in
// destination bytes. vec = cells per access (8 / 4 for 16-byte accesses of bf16 / f32 sources, or 1).
ja_status_t ja_launch_repartition_agg(const char* src, char* dst, const CopySlab* d_slabs, int64_t n_slabs, int n_copies,
                                      int64_t copy_stride, ja_dtype_t src_dt, ja_dtype_t dst_dt, ja_agg_t agg, int vec,
                                      cudaStream_t st);

// tcgen05 / TMEM / TMA matmul join-agg for bf16 relations with uniform blocks.
struct GemmTcPlan;
// Fused epilogue of the matmul join-agg: the next join-agg of a chain applied to the accumulator before its single store.
//   epi 0 none; 1 ADD with `addend` (tiled like the output); 2 ROPE (rotation table, position = row % rope_S, rotated
//   extent rope_D); 3 SWIGLU: silu(A B) * (A B2), B2 tiled like B.
struct GemmEpilogue {
    int epi;
    const ja_relation* addend;
    const ja_relation* B2;
    const float2* rope_table;
    int rope_S, rope_D;
    int partials;   // join only: C is a partial relation [c, i, k] holding one copy per contracted block, nothing is summed across blocks
};
ja_status_t ja_gemm_tc_plan(const ja_relation* A, const ja_relation* B, const ja_relation* C, const GemmEpilogue* ep,
                            std::shared_ptr<GemmTcPlan>* out, bool* eligible);
ja_status_t ja_launch_gemm_tc(const GemmTcPlan& plan, cudaStream_t st);

// Attention join-agg (QK^T join, online-softmax aggregation, PV).
// the four tensor maps (Q, K, V, O) of the tensor-memory kernels, encoded once per (spec, relations) tuple
struct AttnTcCache {
    alignas(64) unsigned char maps[4][128];
    bool valid = false;
};
struct AttnArgs {
    AttnTcCache* cache;    // where the tensor maps are kept between launches, or nullptr
    RelView q, k, v, o;
    RelView lse;           // optional second output [b, q, h] f32: log of the softmax denominator; base == nullptr if absent
    bool lse_rows_layout;  // lse blocks follow the closed-form order of q's (b, s, h) blocks (tensor-memory kernels)
    float scale;
    int causal;
    int32_t B, S, H, D;    // H = query heads
    int32_t group;         // query heads per key/value head (grouped-query attention); 1 otherwise
    int32_t align;         // greatest common divisor of every q / k split point and sequence end
    int32_t n_ends;        // packed sequences: ends[0..n_ends) ascending, ends[n_ends-1] == S; 0 = one sequence
    int32_t ends[JA_MAX_SEQ];
    int32_t sect;          // (batch, head) pairs per launch-order section (set by the launcher)
    // host copies of the sequence split points of q (= o) and k (= v), nblk[1] + 1 entries each, and whether all four
    // payloads follow the closed-form block order the tensor-memory kernel addresses by (uniform b and h blocks)
    const int32_t* q_split;
    const int32_t* k_split;
    bool rows_layout;
    bool f16;              // cell type of Q, K, V, O: false = bf16, true = f16
};
ja_status_t ja_launch_attention(const AttnArgs& a, cudaStream_t st);
// tcgen05 / TMEM form; *launched stays false when the tiling does not fit it
ja_status_t ja_launch_attention_tc(const AttnArgs& a, cudaStream_t st, bool* launched);
// the online-softmax aggregation of m partial attention results (O_c, lse_c) into (O, lse); l may be nullptr
ja_status_t ja_launch_attention_combine(const ja_relation* const* op, const ja_relation* const* lp, int m, const ja_relation* o,
                                        const ja_relation* l, cudaStream_t st);
// an exchange program on one GPU: batched copies of boxes between relation blocks and dense atom buffers (decompose / recompose),
// and the local aggregation of an action -- out = parts[0] (+) parts[1] (+) ... in that order, f32, one rounding
struct JaBoxCopy {
    int64_t src_off, dst_off;                // bytes from the two base pointers
    int64_t n0, n1, run_bytes;               // n0 x n1 runs of run_bytes contiguous bytes
    int64_t src_pitch0, src_pitch1, dst_pitch0, dst_pitch1;   // bytes between consecutive indices of the two outer dimensions
};
#define JA_EXCHANGE_MAX_PARTS 16
ja_status_t ja_launch_box_copies(const char* src, char* dst, const JaBoxCopy* d_boxes, int n_boxes, int64_t max_box_bytes,
                                 bool vec16, int esize, cudaStream_t st);
ja_status_t ja_launch_exchange_combine(const void* const* parts, int n_parts, void* out, int64_t bytes, ja_dtype_t dt,
                                       ja_agg_t agg, cudaStream_t st);
void ja_attention_reset_queues();   // zeroes the work counters of the persistent attention kernel (after a device-side failure)
