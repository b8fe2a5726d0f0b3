// f32 instantiations of the bulk-copy pipelined row-structured join-aggs, and the dispatch on the cell type.
#include "k_row_tma_impl.cuh"

ja_status_t ja_launch_row_tma_bf16(RowOp op, const RowArgs& a, cudaStream_t st, bool* launched);
ja_status_t ja_launch_row_tma_f16(RowOp op, const RowArgs& a, cudaStream_t st, bool* launched);

ja_status_t ja_launch_row_tma(RowOp op, const RowArgs& a, ja_dtype_t dt, cudaStream_t st, bool* launched) {
    if (dt == JA_F32) return row_tma_launch<float>(op, a, st, launched);
    return dt == JA_F16 ? ja_launch_row_tma_f16(op, a, st, launched) : ja_launch_row_tma_bf16(op, a, st, launched);
}
