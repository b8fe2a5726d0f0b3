// Memory-bound join-aggs, bf16 instantiations of the row-structured forms (register-resident rows: the form for tilings
// the bulk-copy pipeline does not take, and RoPE), the flat key-aligned maps, and the dispatch of ja_launch_row.
#include "k_membound_impl.cuh"

ja_status_t ja_launch_row_f32(RowOp op, const RowArgs& a, cudaStream_t st);
ja_status_t ja_launch_row_f16(RowOp op, const RowArgs& a, cudaStream_t st);

ja_status_t ja_launch_flat(ja_fn_t fn, const void* a, const void* b, void* out, int64_t n_elems, ja_dtype_t dt,
                           cudaStream_t st) {
    // payload sizes are multiples of 128 bytes, so whole 16-byte vectors cover them exactly
    const int64_t n_vec = n_elems * (dt == JA_F32 ? 4 : 2) / 16;
    int64_t want = (n_vec + 255) / 256;
    unsigned grid = (unsigned)(want < (int64_t)148 * 32 ? (want > 0 ? want : 1) : (int64_t)148 * 32);
    if (dt == JA_BF16) {
        if (fn == JA_FN_ADD) flat_16bit_kernel<JA_FN_ADD, false><<<grid, 256, 0, st>>>((const uint4*)a, (const uint4*)b, (uint4*)out, n_vec);
        else flat_16bit_kernel<JA_FN_SILU_MUL, false><<<grid, 256, 0, st>>>((const uint4*)a, (const uint4*)b, (uint4*)out, n_vec);
    } else if (dt == JA_F16) {
        if (fn == JA_FN_ADD) flat_16bit_kernel<JA_FN_ADD, true><<<grid, 256, 0, st>>>((const uint4*)a, (const uint4*)b, (uint4*)out, n_vec);
        else flat_16bit_kernel<JA_FN_SILU_MUL, true><<<grid, 256, 0, st>>>((const uint4*)a, (const uint4*)b, (uint4*)out, n_vec);
    } else {
        if (fn == JA_FN_ADD) flat_f32_kernel<JA_FN_ADD><<<grid, 256, 0, st>>>((const float4*)a, (const float4*)b, (float4*)out, n_vec);
        else flat_f32_kernel<JA_FN_SILU_MUL><<<grid, 256, 0, st>>>((const float4*)a, (const float4*)b, (float4*)out, n_vec);
    }
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}

ja_status_t ja_launch_row(RowOp op, const RowArgs& a, ja_dtype_t dt, cudaStream_t st) {
    bool launched = false;
    // statistics-only forms on uniform tilings: a plain read stream
    ja_status_t s = ja_launch_row_reduce(op, a, dt, st, &launched);
    if (s != JA_OK || launched) return s;
    // uniform tilings: bulk-copy pipeline through shared memory
    s = ja_launch_row_tma(op, a, dt, st, &launched);
    if (s != JA_OK || launched) return s;
    if (dt == JA_F32) return ja_launch_row_f32(op, a, st);
    if (dt == JA_F16) return ja_launch_row_f16(op, a, st);
    return launch_row_typed<__nv_bfloat16>(op, a, st);
}
