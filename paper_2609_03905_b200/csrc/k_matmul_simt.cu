// Plain-ALU matmul join-agg "ij,jk->ik" (MUL / SUM) over ARBITRARY tilings, f32 or bf16 operands with f32 accumulation.
// Used for f32 relations (tf32 tensor-core math cannot meet a 1e-5 bound) and for bf16 relations whose blocks neither
// tensor-core loader can take.
//
// One CTA owns one tile of ONE output key (an output block is cut into TM x TN tiles; tiles never span blocks), and walks
// the function specs that share that output key -- the contracted blocks j -- in ascending order: that walk is the SUM
// aggregation of Definition 3.7 (Example 3.8). The key tables are consulted once per (tile, contracted block): two block
// offsets and two widths; inside a block every cell is base + (row * width + column). Operand chunks of TK contracted
// cells go global -> registers -> shared memory with the next chunk's loads in flight while the current one is
// multiplied, 16 bytes per load where every split point of the inner indices is a multiple of the vector width
// (block starts are 128-byte aligned by the layout), one cell per load otherwise.
// Tile size: 64 x 64 (4 x 4 outputs per thread), or 32 x 32 (2 x 2) when 64 x 64 tiles would not give every SM a CTA --
// an output key's walk is never split between CTAs, so small problems get their parallelism from smaller tiles.
// Join-only form (partials != 0): grid.z enumerates the contracted blocks; CTA (., ., c) multiplies block c alone and
// stores copy c of the partial relation C[c, i, k] -- nothing is summed across function specs.
#include <algorithm>

#include "ja_device.cuh"

namespace {

constexpr int NT = 256;

struct SimtParams {
    RelView A, B, C;
    int32_t partials;
    int32_t tiles_i, tiles_k;   // tiles per output block along i and k (of the LARGEST block; CTAs past a smaller block's end leave)
};

// Width of interval `idx` of dimension d and byte offset of block `flat`: arithmetic on uniform tilings (nothing is read
// from memory -- on a small problem a key-table read is a cold DRAM access in front of every operand load), the key table
// otherwise.
__device__ __forceinline__ int64_t interval_width(const RelView& v, int d, int idx) {
    if (v.bs[d]) return min(v.bs[d], v.extent[d] - (int64_t)idx * v.bs[d]);
    return v.splits[d][idx + 1] - v.splits[d][idx];
}
__device__ __forceinline__ int64_t block_offset(const RelView& v, int64_t flat) {
    return v.blk_stride ? flat * v.blk_stride : v.blk_off[flat];
}

template <typename T> struct VecOf;
template <> struct VecOf<float> { typedef float4 type; static constexpr int W = 4; };
template <> struct VecOf<__nv_bfloat16> { typedef uint4 type; static constexpr int W = 8; };
template <> struct VecOf<__half> { typedef uint4 type; static constexpr int W = 8; };

template <typename T, int W> __device__ __forceinline__ void unpack_vec(const typename VecOf<T>::type& v, float (&f)[W]);
template <> __device__ __forceinline__ void unpack_vec<float, 4>(const float4& v, float (&f)[4]) { f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
template <bool F16> __device__ __forceinline__ void unpack_16bit(const uint4& v, float (&f)[8]) {
    const uint32_t* p = reinterpret_cast<const uint32_t*>(&v);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float2 t = ja_unpack16<F16>(p[e]);
        f[2 * e] = t.x;
        f[2 * e + 1] = t.y;
    }
}
template <> __device__ __forceinline__ void unpack_vec<__nv_bfloat16, 8>(const uint4& v, float (&f)[8]) { unpack_16bit<false>(v, f); }
template <> __device__ __forceinline__ void unpack_vec<__half, 8>(const uint4& v, float (&f)[8]) { unpack_16bit<true>(v, f); }

// TM x TN output tile, 256 threads, (TM/16) x (TN/16) outputs per thread. VECTOR: 16-byte operand loads.
// TK: contracted cells per chunk (64 with the small tiles: a small problem is bound by the latency of its chunk loads)
template <typename T, int TM, int TN, bool VECTOR>
__global__ void __launch_bounds__(NT) matmul_simt_kernel(const SimtParams p) {
    constexpr int TK = TM == 32 ? 64 : 32;
    constexpr int W = VecOf<T>::W;
    typedef typename VecOf<T>::type V;
    constexpr int UM = TM / 16, UN = TN / 16;
    // per-thread loads of one chunk: A is TM x TK (vectors run along j), B is TK x TN (vectors run along k)
    constexpr int NA = VECTOR ? (TM * TK / W + NT - 1) / NT : TM * TK / NT;
    constexpr int NB = VECTOR ? (TK * TN / W + NT - 1) / NT : TK * TN / NT;
    __shared__ __align__(16) float As[TK][TM + 4];
    __shared__ __align__(16) float Bs[TK][TN + 4];
    const RelView &A = p.A, &B = p.B, &C = p.C;
    const int tid = threadIdx.x;
    const int kb = blockIdx.x / p.tiles_k, tk = blockIdx.x % p.tiles_k;
    const int ib = blockIdx.y / p.tiles_i, ti = blockIdx.y % p.tiles_i;
    const int64_t bm = interval_width(A, 0, ib), bn = interval_width(B, 1, kb);
    const int64_t r0 = (int64_t)ti * TM, c0 = (int64_t)tk * TN;      // tile origin inside the output block
    if (r0 >= bm || c0 >= bn) return;                                // this block is smaller than the largest one
    const int tr = tid / 16, tc = tid % 16;
    float acc[UM][UN];
#pragma unroll
    for (int a = 0; a < UM; ++a)
#pragma unroll
        for (int b = 0; b < UN; ++b) acc[a][b] = 0.f;

    V va[VECTOR ? NA : 1], vb[VECTOR ? NB : 1];
    T sa[VECTOR ? 1 : NA], sb[VECTOR ? 1 : NB];
    const int nbj = A.nblk[1], nbk = B.nblk[1];
    const int jb_lo = p.partials ? (int)blockIdx.z : 0, jb_hi = p.partials ? (int)blockIdx.z + 1 : nbj;

    // one chunk = TK contracted cells starting at j0 inside contracted block jb
    const char *a_blk = nullptr, *b_blk = nullptr;
    int64_t wj = 0;
    auto set_block = [&](int jb) {
        wj = interval_width(A, 1, jb);
        a_blk = A.base + block_offset(A, (int64_t)ib * nbj + jb);    // block (ib, jb): bm rows of wj cells
        b_blk = B.base + block_offset(B, (int64_t)jb * nbk + kb);    // block (jb, kb): wj rows of bn cells
    };
    auto load_chunk = [&](int64_t j0) {
        if (VECTOR) {
#pragma unroll
            for (int n = 0; n < NA; ++n) {
                const int e = tid + n * NT, r = e / (TK / W), c = (e % (TK / W)) * W;
                V v = {};
                if (e < TM * TK / W && r0 + r < bm && j0 + c < wj) v = *reinterpret_cast<const V*>(a_blk + ((r0 + r) * wj + j0 + c) * (int64_t)sizeof(T));
                va[n] = v;
            }
#pragma unroll
            for (int n = 0; n < NB; ++n) {
                const int e = tid + n * NT, r = e / (TN / W), c = (e % (TN / W)) * W;
                V v = {};
                if (e < TK * TN / W && j0 + r < wj && c0 + c < bn) v = *reinterpret_cast<const V*>(b_blk + ((j0 + r) * bn + c0 + c) * (int64_t)sizeof(T));
                vb[n] = v;
            }
        } else {
#pragma unroll
            for (int n = 0; n < NA; ++n) {
                const int e = tid + n * NT, r = e / TK, c = e % TK;
                sa[n] = (r0 + r < bm && j0 + c < wj) ? *reinterpret_cast<const T*>(a_blk + ((r0 + r) * wj + j0 + c) * (int64_t)sizeof(T)) : ja_from_float<T>(0.f);
            }
#pragma unroll
            for (int n = 0; n < NB; ++n) {
                const int e = tid + n * NT, r = e / TN, c = e % TN;
                sb[n] = (j0 + r < wj && c0 + c < bn) ? *reinterpret_cast<const T*>(b_blk + ((j0 + r) * bn + c0 + c) * (int64_t)sizeof(T)) : ja_from_float<T>(0.f);
            }
        }
    };
    auto store_chunk = [&]() {
        if (VECTOR) {
#pragma unroll
            for (int n = 0; n < NA; ++n) {
                const int e = tid + n * NT, r = e / (TK / W), c = (e % (TK / W)) * W;
                if (e < TM * TK / W) {
                    float f[W];
                    unpack_vec<T, W>(va[n], f);
#pragma unroll
                    for (int u = 0; u < W; ++u) As[c + u][r] = f[u];
                }
            }
#pragma unroll
            for (int n = 0; n < NB; ++n) {
                const int e = tid + n * NT, r = e / (TN / W), c = (e % (TN / W)) * W;
                if (e < TK * TN / W) {
                    float f[W];
                    unpack_vec<T, W>(vb[n], f);
#pragma unroll
                    for (int u = 0; u < W; u += 4) *reinterpret_cast<float4*>(&Bs[r][c + u]) = make_float4(f[u], f[u + 1], f[u + 2], f[u + 3]);
                }
            }
        } else {
#pragma unroll
            for (int n = 0; n < NA; ++n) {
                const int e = tid + n * NT;
                As[e % TK][e / TK] = ja_to_float(sa[n]);
            }
#pragma unroll
            for (int n = 0; n < NB; ++n) {
                const int e = tid + n * NT;
                Bs[e / TN][e % TN] = ja_to_float(sb[n]);
            }
        }
    };

    // the walk: contracted blocks ascending, chunks ascending inside a block; the next chunk's loads are issued before the
    // current chunk is multiplied
    int jb = jb_lo;
    int64_t j0 = 0;
    set_block(jb);
    load_chunk(0);
    while (true) {
        store_chunk();
        __syncthreads();
        // advance to the next chunk (possibly the first one of the next contracted block) and start its loads
        int64_t nj0 = j0 + TK;
        int njb = jb;
        if (nj0 >= wj) { nj0 = 0; ++njb; }
        const bool more = njb < jb_hi;
        if (more) {
            if (njb != jb) set_block(njb);
            load_chunk(nj0);
        }
#pragma unroll 8
        for (int kk = 0; kk < TK; ++kk) {
            float a[UM], b[UN];
#pragma unroll
            for (int u = 0; u < UM; ++u) a[u] = As[kk][tr * UM + u];
#pragma unroll
            for (int u = 0; u < UN; ++u) b[u] = Bs[kk][tc * UN + u];
#pragma unroll
            for (int u = 0; u < UM; ++u)
#pragma unroll
                for (int w = 0; w < UN; ++w) acc[u][w] = fmaf(a[u], b[w], acc[u][w]);
        }
        if (!more) break;
        __syncthreads();
        jb = njb;
        j0 = nj0;
    }

    // Recompose: the aggregated tile goes to its place in the output block (copy c of a partial relation in join-only form)
    const int64_t c_flat = p.partials ? ((int64_t)blockIdx.z * A.nblk[0] + ib) * nbk + kb : (int64_t)ib * nbk + kb;
    char* c_blk = C.base + block_offset(C, c_flat);
#pragma unroll
    for (int u = 0; u < UM; ++u) {
        const int64_t r = r0 + tr * UM + u;
        if (r >= bm) continue;
        const int64_t c = c0 + tc * UN;
        T* dst = reinterpret_cast<T*>(c_blk) + r * bn + c;
        if (VECTOR && UN == 4 && c + 3 < bn) {
            if (sizeof(T) == 4) {
                *reinterpret_cast<float4*>(dst) = make_float4(acc[u][0], acc[u][1], acc[u][2], acc[u][3]);
            } else {
                constexpr bool F16 = JaDtypeOf<T>::value == JA_F16;
                *reinterpret_cast<uint2*>(dst) = make_uint2(ja_pack16<F16>(acc[u][0], acc[u][1]), ja_pack16<F16>(acc[u][2], acc[u][3]));
            }
        } else {
#pragma unroll
            for (int w = 0; w < UN; ++w)
                if (c + w < bn) dst[w] = ja_from_float<T>(acc[u][w]);
        }
    }
}

template <typename T, int TM, int TN>
void launch(const SimtParams& p, dim3 grid, bool vec, cudaStream_t st) {
    if (vec) matmul_simt_kernel<T, TM, TN, true><<<grid, NT, 0, st>>>(p);
    else matmul_simt_kernel<T, TM, TN, false><<<grid, NT, 0, st>>>(p);
}

}  // namespace

// host_* : the relations' split points along the inner indices (A's j, B's k) and the block extents, for the choice of
// tile size and load width
ja_status_t ja_launch_matmul_simt(const ja_relation* Ar, const ja_relation* Br, const ja_relation* Cr, cudaStream_t st, bool partials) {
    SimtParams p;
    p.A = ja_view(Ar);
    p.B = ja_view(Br);
    p.C = ja_view(Cr);
    p.partials = partials ? 1 : 0;
    const ja_dtype_t dt = Ar->dtype;
    const int W = dt == JA_F32 ? 4 : 8;
    int64_t max_bm = 0, max_bn = 0;
    for (int i = 0; i < Ar->nblk[0]; ++i) max_bm = std::max(max_bm, Ar->splits[0][i + 1] - Ar->splits[0][i]);
    for (int i = 0; i < Br->nblk[1]; ++i) max_bn = std::max(max_bn, Br->splits[1][i + 1] - Br->splits[1][i]);
    bool vec = true;   // every vector must lie inside one block row: split points of j and k multiples of the vector width
    for (int64_t s : Ar->splits[1]) vec = vec && s % W == 0;
    for (int64_t s : Br->splits[1]) vec = vec && s % W == 0;
    const int copies = partials ? Ar->nblk[1] : 1;
    auto tiles = [&](int t) { return (int64_t)Ar->nblk[0] * ((max_bm + t - 1) / t) * Br->nblk[1] * ((max_bn + t - 1) / t) * copies; };
    const bool small = tiles(64) < ja_sm_count();
    const int t = small ? 32 : 64;
    p.tiles_i = (int)((max_bm + t - 1) / t);
    p.tiles_k = (int)((max_bn + t - 1) / t);
    const int64_t gx = (int64_t)Br->nblk[1] * p.tiles_k, gy = (int64_t)Ar->nblk[0] * p.tiles_i;
    if (gx > 0x7fffffff || gy > 65535 || copies > 65535) return ja_fail(JA_ERR_UNSUPPORTED, "matmul tiling too fine for the plain-ALU kernel's grid");
    dim3 grid((unsigned)gx, (unsigned)gy, (unsigned)copies);
    if (dt == JA_F32) {
        if (small) launch<float, 32, 32>(p, grid, vec, st);
        else launch<float, 64, 64>(p, grid, vec, st);
    } else if (dt == JA_F16) {
        if (small) launch<__half, 32, 32>(p, grid, vec, st);
        else launch<__half, 64, 64>(p, grid, vec, st);
    } else {
        if (small) launch<__nv_bfloat16, 32, 32>(p, grid, vec, st);
        else launch<__nv_bfloat16, 64, 64>(p, grid, vec, st);
    }
    ja_count_launch();
    JA_CUDA(cudaGetLastError());
    return JA_OK;
}
