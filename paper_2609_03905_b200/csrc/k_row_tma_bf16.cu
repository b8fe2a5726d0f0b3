// bf16 instantiations of the bulk-copy pipelined row-structured join-aggs (one translation unit per cell type keeps
// the build parallel).
#include "k_row_tma_impl.cuh"

ja_status_t ja_launch_row_tma_bf16(RowOp op, const RowArgs& a, cudaStream_t st, bool* launched) {
    return row_tma_launch<__nv_bfloat16>(op, a, st, launched);
}
