// f16 instantiations of the bulk-copy pipelined row-structured join-aggs (one translation unit per cell type keeps
// the build parallel). f16 rows take the plain per-cell arithmetic of the f32 rows on eight cells per 16-byte vector.
#include "k_row_tma_impl.cuh"

ja_status_t ja_launch_row_tma_f16(RowOp op, const RowArgs& a, cudaStream_t st, bool* launched) {
    return row_tma_launch<__half>(op, a, st, launched);
}
