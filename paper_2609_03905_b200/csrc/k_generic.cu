// The general join-agg of Definition 3.7 for specs no specialised kernel takes: any einsum over up to four operands
// whose concrete operator is a scalar function of the joined cells (product, identity, square, sum, silu(a) b, exp(a - b))
// with SUM, MAX or no aggregation over the indices that do not reach the output. This is the definition executed in its
// relational form on the GPU: one thread per output cell walks the joined tuples of that cell -- the coordinates of the
// summed indices in ascending order -- applies the operator in f32 and aggregates in f32; every operand cell is located
// through its relation's key table (binary search per index), so any tiling of any operand works. It exists so that
// every spec ja_spec_create accepts executes; it is not a fast path (batched or transposed contractions of real size
// belong on the tensor-core kernels through a relayout).
#include <stdlib.h>
#include <string.h>

#include "ja_device.cuh"

namespace {

constexpr int MAX_OPERANDS = 4, MAX_SUMMED = 4;

struct GenericParams {
    RelView in[MAX_OPERANDS];
    RelView out;
    int32_t n_in, n_out, n_sum;                     // operands, output indices, summed indices
    int32_t in_dtype[MAX_OPERANDS], out_dtype;
    int32_t in_pos[MAX_OPERANDS][JA_MAX_RANK];      // position of every operand index in the coordinate vector (output indices first)
    int64_t out_ext[JA_MAX_RANK], sum_ext[MAX_SUMMED];
    int64_t n_out_cells, n_sum_cells;
    int32_t fn, agg;
};

__device__ __forceinline__ float load_cell(const RelView& v, int dtype, const int64_t* x) {
    const char* p = v.base + ja_elem_off(v, x);
    if (dtype == JA_F32) return *reinterpret_cast<const float*>(p);
    if (dtype == JA_F16) return __half2float(*reinterpret_cast<const __half*>(p));
    return __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(p));
}

__global__ void __launch_bounds__(256) generic_join_agg_kernel(const GenericParams p) {
    for (int64_t cell = (int64_t)blockIdx.x * 256 + threadIdx.x; cell < p.n_out_cells; cell += (int64_t)gridDim.x * 256) {
        int64_t coord[JA_MAX_RANK + MAX_SUMMED];
        int64_t rem = cell;
        for (int d = p.n_out - 1; d >= 0; --d) {
            coord[d] = rem % p.out_ext[d];
            rem /= p.out_ext[d];
        }
        float acc = p.agg == JA_AGG_MAX ? -INFINITY : 0.f;
        for (int64_t s = 0; s < p.n_sum_cells; ++s) {      // the tuples joined into this output cell, ascending
            int64_t r2 = s;
            for (int d = p.n_sum - 1; d >= 0; --d) {
                coord[p.n_out + d] = r2 % p.sum_ext[d];
                r2 /= p.sum_ext[d];
            }
            float v[MAX_OPERANDS];
            for (int k = 0; k < p.n_in; ++k) {
                int64_t x[JA_MAX_RANK];
                for (int d = 0; d < p.in[k].rank; ++d) x[d] = coord[p.in_pos[k][d]];
                v[k] = load_cell(p.in[k], p.in_dtype[k], x);
            }
            float g;
            switch (p.fn) {
                case JA_FN_MUL: g = v[0]; for (int k = 1; k < p.n_in; ++k) g *= v[k]; break;
                case JA_FN_ADD: g = v[0]; for (int k = 1; k < p.n_in; ++k) g += v[k]; break;
                case JA_FN_SQUARE: g = v[0] * v[0]; break;
                case JA_FN_SILU_MUL: g = v[0] / (1.f + __expf(-v[0])) * v[1]; break;
                case JA_FN_EXP_SUB: g = __expf(v[0] - v[1]); break;
                default: g = v[0]; break;   // JA_FN_IDENT
            }
            acc = p.agg == JA_AGG_MAX ? fmaxf(acc, g) : acc + g;
        }
        char* o = p.out.base + ja_elem_off(p.out, coord);
        if (p.out_dtype == JA_F32) *reinterpret_cast<float*>(o) = acc;
        else if (p.out_dtype == JA_F16) *reinterpret_cast<__half*>(o) = __float2half_rn(acc);
        else *reinterpret_cast<__nv_bfloat16*>(o) = __float2bfloat16_rn(acc);
    }
}

}  // namespace

// *launched stays false when the spec is outside this kernel's reach (more than four operands or summed indices, an
// operator that is not a scalar function of the joined cells, NONE aggregation with summed indices).
ja_status_t ja_launch_generic(const ja_spec* spec, const ja_relation* const* inputs, const ja_relation* out, cudaStream_t st, bool* launched) {
    *launched = false;
    const int n_in = (int)spec->ins.size();
    if (n_in < 1 || n_in > MAX_OPERANDS) return JA_OK;
    switch (spec->fn) {
        case JA_FN_MUL: case JA_FN_ADD: break;
        case JA_FN_IDENT: case JA_FN_SQUARE: if (n_in != 1) return JA_OK; break;
        case JA_FN_SILU_MUL: case JA_FN_EXP_SUB: if (n_in != 2) return JA_OK; break;
        default: return JA_OK;
    }
    GenericParams p;
    memset(&p, 0, sizeof p);
    std::string coords = spec->out;             // output indices first, then the summed ones in order of first appearance
    for (char c : spec->letters)
        if (coords.find(c) == std::string::npos) coords.push_back(c);
    p.n_in = n_in;
    p.n_out = (int)spec->out.size();
    p.n_sum = (int)coords.size() - p.n_out;
    if (p.n_out < 1 || p.n_out > JA_MAX_RANK || p.n_sum > MAX_SUMMED) return JA_OK;
    if (spec->agg != JA_AGG_SUM && spec->agg != JA_AGG_MAX && !(spec->agg == JA_AGG_NONE && p.n_sum == 0)) return JA_OK;
    auto extent_of = [&](char c) { return spec->parts[spec->letters.find(c)].back(); };
    p.n_out_cells = 1;
    p.n_sum_cells = 1;
    for (int d = 0; d < p.n_out; ++d) { p.out_ext[d] = extent_of(coords[d]); p.n_out_cells *= p.out_ext[d]; }
    for (int d = 0; d < p.n_sum; ++d) { p.sum_ext[d] = extent_of(coords[p.n_out + d]); p.n_sum_cells *= p.sum_ext[d]; }
    for (int k = 0; k < n_in; ++k) {
        p.in[k] = ja_view(inputs[k]);
        p.in_dtype[k] = (int)inputs[k]->dtype;
        for (size_t d = 0; d < spec->ins[k].size(); ++d) p.in_pos[k][d] = (int)coords.find(spec->ins[k][d]);
    }
    p.out = ja_view(out);
    p.out_dtype = (int)out->dtype;
    p.fn = (int)spec->fn;
    p.agg = (int)spec->agg;
    const int64_t want = (p.n_out_cells + 255) / 256, cap = (int64_t)ja_sm_count() * 32;
    generic_join_agg_kernel<<<(unsigned)(want < cap ? (want > 0 ? want : 1) : cap), 256, 0, st>>>(p);
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    *launched = true;
    return JA_OK;
}
