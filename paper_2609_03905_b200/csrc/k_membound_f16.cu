// f16 instantiations of the register-resident row-structured join-aggs (one translation unit per cell type keeps the
// build parallel).
#include "k_membound_impl.cuh"

ja_status_t ja_launch_row_f16(RowOp op, const RowArgs& a, cudaStream_t st) { return launch_row_typed<__half>(op, a, st); }
