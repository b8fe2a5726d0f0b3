// Plain-ALU matmul join-agg "ij,jk->ik" (MUL / SUM) over ARBITRARY tilings, f32 or bf16 operands with
// f32 accumulation. Every operand cell is located through the relation's key table, so any tiling
// works; the contracted index is walked block by block in ascending key order, which is the SUM
// aggregation over the function specs that share an output type (Definition 3.7, Example 3.8).
// Used for f32 relations (tf32 tensor-core math cannot meet a 1e-5 bound) and as the fallback for
// bf16 relations whose blocks the tensor-core path cannot address.
// Join-only form (partials != 0): grid.z enumerates the contracted blocks; CTA (., ., c) multiplies block c alone and
// stores copy c of the partial relation C[c, i, k] -- nothing is summed across function specs.
#include "ja_device.cuh"

namespace {

constexpr int TM = 64, TN = 64, TK = 16;

template <typename T>
__global__ void __launch_bounds__(256) matmul_simt_kernel(RelView A, RelView B, RelView C, int partials) {
    __shared__ float As[TK][TM + 4];
    __shared__ float Bs[TK][TN + 4];
    const int tid = threadIdx.x;
    const int64_t i0 = (int64_t)blockIdx.y * TM, k0 = (int64_t)blockIdx.x * TN;
    const int64_t M = A.extent[0], J = A.extent[1], N = B.extent[1];
    const int tr = tid / 16, tc = tid % 16;  // this thread owns rows tr*4.., cols tc*4..
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

    const int jb_lo = partials ? (int)blockIdx.z : 0, jb_hi = partials ? (int)blockIdx.z + 1 : A.nblk[1];
    for (int jb = jb_lo; jb < jb_hi; ++jb) {  // the tuples of this output key, ascending
        const int64_t jlo = A.splits[1][jb], jhi = A.splits[1][jb + 1];
        for (int64_t j0 = jlo; j0 < jhi; j0 += TK) {
            for (int e = tid; e < TM * TK; e += 256) {
                int r = e / TK, c = e % TK;
                int64_t x[2] = {i0 + r, j0 + c};
                float v = 0.f;
                if (x[0] < M && x[1] < jhi) v = ja_to_float(*(const T*)(A.base + ja_elem_off(A, x)));
                As[c][r] = v;
            }
            for (int e = tid; e < TK * TN; e += 256) {
                int r = e / TN, c = e % TN;
                int64_t x[2] = {j0 + r, k0 + c};
                float v = 0.f;
                if (x[0] < jhi && x[1] < N) v = ja_to_float(*(const T*)(B.base + ja_elem_off(B, x)));
                Bs[r][c] = v;
            }
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < TK; ++kk) {
                float a[4], b[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) a[u] = As[kk][tr * 4 + u];
#pragma unroll
                for (int u = 0; u < 4; ++u) b[u] = Bs[kk][tc * 4 + u];
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int w = 0; w < 4; ++w) acc[u][w] = fmaf(a[u], b[w], acc[u][w]);
            }
            __syncthreads();
        }
    }
    (void)J;
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            int64_t x[3] = {i0 + tr * 4 + u, k0 + tc * 4 + w, 0};
            if (x[0] < M && x[1] < N) {
                if (partials) { x[2] = x[1]; x[1] = x[0]; x[0] = blockIdx.z; }
                *(T*)(C.base + ja_elem_off(C, x)) = ja_from_float<T>(acc[u][w]);
            }
        }
}

}  // namespace

ja_status_t ja_launch_matmul_simt(const RelView& A, const RelView& B, const RelView& C, ja_dtype_t dt, cudaStream_t st,
                                  bool partials) {
    dim3 grid((unsigned)((B.extent[1] + TN - 1) / TN), (unsigned)((A.extent[0] + TM - 1) / TM), partials ? (unsigned)A.nblk[1] : 1u);
    if (dt == JA_F32) matmul_simt_kernel<float><<<grid, 256, 0, st>>>(A, B, C, partials ? 1 : 0);
    else matmul_simt_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(A, B, C, partials ? 1 : 0);
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}
