/*
 * ja_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow CPU oracle for join-agg execution over tensor relations in the
 * degenerate, purely relational form: every key identifies ONE cell and every
 * sub-tensor is ONE scalar (paper Section 1, "tensor relation"; Definition 3.7
 * "Implementation").  All arithmetic is IEEE fp64.  Only the tests, the smoke
 * check and the CPU-baseline leg of the benchmark may call into this file; the
 * GPU library shares no code, header, table or constant with it.
 *
 * Engine "T1" (orc_join_agg): pipelined index-nested-loop evaluation of
 *
 *     V[o] = (+) over all assignments a of the aggregated indices of
 *            g( U_1[pi_1(o,a)], ..., U_n[pi_n(o,a)] )
 *
 * i.e.  SELECT L_o, AGG(g(v_1..v_n)) FROM R_1 NATURAL JOIN ... R_n GROUP BY L_o.
 * Because the index set of a tensor type is a full box (Definition 3.1), the
 * "index" on each relation is direct addressing.  The aggregated indices are
 * enumerated in ascending order, last-listed fastest, so the fold order per
 * output key is fixed.
 *
 * The remaining entry points are plain definitions of two operators whose
 * full-size evaluation through the generic engine would take hours (matrix
 * multiply, Example 3.4; causal dot-product attention, Example 3.10 restricted
 * to one KV head per query head), each checked against the generic engine and
 * against library routines by the CPU tests.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC -o libja_oracle.so ja_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_MAX_IDX 12
#define ORC_MAX_IN 4

/* scalar functions g applied to one joined tuple of scalars */
enum {
    ORC_FN_MUL = 0,         /* product of all inputs (einsum)                      */
    ORC_FN_IDENT = 1,       /* v0                                                  */
    ORC_FN_SQUARE = 2,      /* v0^2                                                */
    ORC_FN_ADD = 3,         /* sum of all inputs                                   */
    ORC_FN_SILU_MUL = 4,    /* v0/(1+exp(-v0)) * v1                                */
    ORC_FN_RMS_SCALE = 5,   /* v0 * (v1/n + eps)^(-1/2) * v2 ; p[0]=eps, p[1]=n    */
    ORC_FN_EXP_SUB = 6,     /* exp(v0 - v1)                                        */
    ORC_FN_EXP_SUB_DIV = 7  /* exp(v0 - v1) / v2                                   */
};

/* aggregation operators (+): binary, associative, commutative (Definition 3.7) */
enum { ORC_AGG_NONE = 0, ORC_AGG_SUM = 1, ORC_AGG_MAX = 2 };

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Round an fp64 value to the nearest bfloat16 (8 significant bits, exponent
 * range of fp32), ties to even, and return it as fp64. */
double orc_round_bf16(double x) {
    if (isnan(x) || isinf(x) || x == 0.0) return x;
    int e;
    (void)frexp(x, &e);            /* |x| = f * 2^e, f in [0.5, 1) => leading bit at 2^(e-1) */
    int lead = e - 1;
    if (lead < -126) lead = -126;  /* subnormal range shares the quantum of the lowest binade */
    int qexp = lead - 7;           /* quantum = 2^(lead-7): 7 explicit mantissa bits            */
    double scaled = ldexp(x, -qexp);          /* exact */
    double r = ldexp(nearbyint(scaled), qexp); /* nearbyint: round-half-even in the default mode */
    if (fabs(r) >= ldexp(1.0, 128)) return x > 0 ? INFINITY : -INFINITY;
    return r;
}

double orc_round_f32(double x) { return (double)(float)x; }

/* IEEE binary16 (the precision of the paper's experiments, Section 6): 10 explicit mantissa bits, lowest binade 2^-14,
 * largest finite value 65504; one rounding from fp64, ties to even. */
double orc_round_f16(double x) {
    if (isnan(x) || isinf(x) || x == 0.0) return x;
    int e;
    (void)frexp(x, &e);
    int lead = e - 1;
    if (lead < -14) lead = -14;    /* subnormals share the quantum of the lowest binade */
    int qexp = lead - 10;
    double r = ldexp(nearbyint(ldexp(x, -qexp)), qexp);
    if (fabs(r) >= ldexp(1.0, 16)) return x > 0 ? INFINITY : -INFINITY;
    return r;
}

void orc_round_array(double* a, int64_t n, int dtype /* 0 = f32, 1 = bf16, 2 = f16 */) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) a[i] = dtype == 2 ? orc_round_f16(a[i]) : dtype ? orc_round_bf16(a[i]) : orc_round_f32(a[i]);
}

static double apply_g(int fn, const double* v, int n, const double* p) {
    switch (fn) {
        case ORC_FN_MUL: {
            double r = v[0];
            for (int k = 1; k < n; ++k) r *= v[k];
            return r;
        }
        case ORC_FN_IDENT: return v[0];
        case ORC_FN_SQUARE: return v[0] * v[0];
        case ORC_FN_ADD: {
            double r = v[0];
            for (int k = 1; k < n; ++k) r += v[k];
            return r;
        }
        case ORC_FN_SILU_MUL: return v[0] / (1.0 + exp(-v[0])) * v[1];
        case ORC_FN_RMS_SCALE: return v[0] * (1.0 / sqrt(v[1] / p[1] + p[0])) * v[2];
        case ORC_FN_EXP_SUB: return exp(v[0] - v[1]);
        case ORC_FN_EXP_SUB_DIV: return exp(v[0] - v[1]) / v[2];
        default: return NAN;
    }
}

/*
 * Generic scalar-keyed join-agg (engine T1).
 *
 *   n_idx, extent[n_idx]      the named indices and their upper bounds (zero-bounded types)
 *   n_in, in_rank[k], in_idx  operand k is keyed by indices in_idx[k*ORC_MAX_IDX + 0..rank), dense row-major
 *   out_rank, out_idx         output key columns (GROUP BY list)
 *   pred_lo, pred_hi          selection predicate: keep a joined tuple only if
 *                             value(index pred_lo) <= value(index pred_hi); -1/-1 = no predicate.
 *                             (The causal band of attention is such a selection.)
 *   An output key with no surviving tuple receives the identity of (+): 0 for SUM, -inf for MAX.
 * Returns 0 on success, nonzero on a malformed request.
 */
int orc_join_agg(int n_idx, const int64_t* extent, int n_in, const int* in_rank, const int* in_idx,
                 const double* const* in_data, int out_rank, const int* out_idx, double* out, int fn,
                 const double* fn_params, int agg, int pred_lo, int pred_hi) {
    if (n_idx < 1 || n_idx > ORC_MAX_IDX || n_in < 1 || n_in > ORC_MAX_IN) return 1;
    int is_out[ORC_MAX_IDX] = {0};
    for (int d = 0; d < out_rank; ++d) {
        if (out_idx[d] < 0 || out_idx[d] >= n_idx) return 2;
        is_out[out_idx[d]] = 1;
    }
    int agg_idx[ORC_MAX_IDX], n_agg = 0;
    for (int x = 0; x < n_idx; ++x)
        if (!is_out[x]) agg_idx[n_agg++] = x;
    if (agg == ORC_AGG_NONE && n_agg != 0) return 3;

    /* row-major strides of every operand, expressed per named index */
    int64_t in_stride[ORC_MAX_IN][ORC_MAX_IDX];
    memset(in_stride, 0, sizeof in_stride);
    for (int k = 0; k < n_in; ++k) {
        int64_t s = 1;
        for (int d = in_rank[k] - 1; d >= 0; --d) {
            int x = in_idx[k * ORC_MAX_IDX + d];
            if (x < 0 || x >= n_idx) return 4;
            in_stride[k][x] += s; /* a repeated letter addresses a diagonal */
            s *= extent[x];
        }
    }
    int64_t n_out = 1;
    for (int d = 0; d < out_rank; ++d) n_out *= extent[out_idx[d]];
    int64_t n_aggr = 1;
    for (int a = 0; a < n_agg; ++a) n_aggr *= extent[agg_idx[a]];

#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < n_out; ++o) {
        int64_t val[ORC_MAX_IDX];
        /* decode the output key (row-major over out_idx) */
        int64_t rem = o;
        for (int d = out_rank - 1; d >= 0; --d) {
            int x = out_idx[d];
            val[x] = rem % extent[x];
            rem /= extent[x];
        }
        double acc = (agg == ORC_AGG_MAX) ? -INFINITY : 0.0;
        for (int64_t t = 0; t < n_aggr; ++t) {
            /* decode the aggregated-index assignment: last-listed index fastest, ascending */
            int64_t r2 = t;
            for (int a = n_agg - 1; a >= 0; --a) {
                int x = agg_idx[a];
                val[x] = r2 % extent[x];
                r2 /= extent[x];
            }
            if (pred_lo >= 0 && !(val[pred_lo] <= val[pred_hi])) continue; /* selection */
            double v[ORC_MAX_IN];
            for (int k = 0; k < n_in; ++k) {
                int64_t off = 0;
                for (int x = 0; x < n_idx; ++x) off += in_stride[k][x] * val[x];
                v[k] = in_data[k][off];
            }
            double g = apply_g(fn, v, n_in, fn_params);
            if (agg == ORC_AGG_SUM) acc = acc + g;
            else if (agg == ORC_AGG_MAX) acc = (g > acc) ? g : acc;
            else acc = g;
        }
        out[o] = acc;
    }
    return 0;
}

/*
 * Matrix multiply C[i,k] = SUM_j A[i,j] * B[j,k]  (Example 3.4; "a join on the
 * shared inner index followed by a SUM aggregation").  Row-major dense operands.
 * For every output key (i,k) the products are added in ascending j, exactly as
 * orc_join_agg does; only the loop nest is arranged so that k runs innermost.
 */
void orc_matmul(const double* A, const double* B, double* C, int64_t M, int64_t J, int64_t N) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        double* c = C + i * N;
        for (int64_t k = 0; k < N; ++k) c[k] = 0.0;
        for (int64_t j = 0; j < J; ++j) {
            const double a = A[i * J + j];
            const double* b = B + j * N;
            for (int64_t k = 0; k < N; ++k) c[k] += a * b[k];
        }
    }
}

/*
 * Dot-product attention, plain definition, operands laid out [b, s, h, d]:
 *   S[b,h,q,k] = scale * SUM_d Q[b,q,h,d] K[b,k,h,d]
 *   selection  k <= pos(q)  when causal, pos(q) = qpos[q] (the position of query row q in its
 *              sequence; qpos == NULL means pos(q) = q, i.e. Q holds every row of the sequence)
 *   P          = exp(S - max_k S) / SUM_k exp(S - max_k S)   over the selected k
 *   O[b,q,h,d] = SUM_k P[b,h,q,k] V[b,k,h,d]
 * Q and O have Sq rows per sequence, K and V have Sk.  Nothing inside is rounded.
 */
void orc_attention(const double* Q, const double* K, const double* V, double* O, int64_t B, int64_t Sq,
                   int64_t Sk, int64_t H, int64_t D, double scale, int causal, const int64_t* qpos) {
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
    for (int64_t bh = 0; bh < B * H; ++bh) {
        for (int64_t q = 0; q < Sq; ++q) {
            const int64_t b = bh / H, h = bh % H;
            const int64_t pos = qpos ? qpos[q] : q;
            const int64_t nk = causal ? pos + 1 : Sk;
            double* s = (double*)malloc(sizeof(double) * (size_t)nk);
            const double* qv = Q + ((b * Sq + q) * H + h) * D;
            double m = -INFINITY;
            for (int64_t k = 0; k < nk; ++k) {
                const double* kv = K + ((b * Sk + k) * H + h) * D;
                double dot = 0.0;
                for (int64_t d = 0; d < D; ++d) dot += qv[d] * kv[d];
                s[k] = scale * dot;
                if (s[k] > m) m = s[k];
            }
            double l = 0.0;
            for (int64_t k = 0; k < nk; ++k) {
                s[k] = exp(s[k] - m);
                l += s[k];
            }
            double* o = O + ((b * Sq + q) * H + h) * D;
            for (int64_t d = 0; d < D; ++d) o[d] = 0.0;
            for (int64_t k = 0; k < nk; ++k) {
                const double p = s[k] / l;
                const double* vv = V + ((b * Sk + k) * H + h) * D;
                for (int64_t d = 0; d < D; ++d) o[d] += p * vv[d];
            }
            free(s);
        }
    }
}
