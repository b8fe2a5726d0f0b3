/*
 * ja.h -- C ABI of libja: execution of join-agg specs over tensor relations on one B200.
 *
 * Vocabulary follows the paper ("Every Kernel Is a Join"):
 *   tensor type      rank + lower/upper bound vectors (Definition 3.1)
 *   tiling           a set of tensor types that cover a type disjointly (Definition 3.2)
 *   tensor relation  a tensor stored as (sub_tensor_key, sub_tensor) pairs, the key being the tensor
 *                    type of the sub-tensor (Section 1; Section 3.2)
 *   function spec F  one joined tuple of input sub-tensor types -> output sub-tensor types (Definition 3.5)
 *   join-agg spec J  the set {F_1..F_p} obtained from one interval decomposition of the named indices
 *                    (Definition 3.6; Section 3.3: exactly prod_s intervals[s] function specs)
 *   implementation   Join (run f on every F) -> Aggregate ((+) over the F sharing an output type)
 *                    -> Recompose (Definition 3.7)
 *
 * Conventions
 *   - Every call returns ja_status_t; JA_OK == 0.  ja_last_error() gives a thread-local message.
 *   - Argument errors are reported synchronously, before anything is enqueued; nothing is ever
 *     partially enqueued.
 *   - Handles (ja_spec_t, ja_relation_t) are opaque, owned by the library, freed by *_destroy.
 *   - "host" / "device" in a parameter comment says where the pointed-to memory lives.
 *   - Relation payloads are DEVICE memory owned by the caller (borrowed, never freed here), 128-byte
 *     aligned, and must outlive every enqueued use.
 *   - Canonical orders: index letters in order of first appearance in the einsum string (inputs left
 *     to right, then the output); function specs row-major over the interval grid in that letter order
 *     (last letter fastest); blocks of a relation row-major over the relation's own index order;
 *     atoms row-major over the overlay grid.
 *
 * Payload layout of a relation ("block-key layout"): blocks in row-major key order, each block a dense
 * row-major array of its own extents, blocks back to back, each starting on a 128-byte boundary.
 *
 * Exchange programs (Section 5: the ExProg language, validity, the simulator, synthesis, placement, preamble
 * generation, and a program's execution on one GPU) are declared in ja_exprog.h, which includes this header.
 */
#ifndef JA_H_
#define JA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    JA_OK = 0,
    JA_ERR_INVALID_ARG = 1,
    JA_ERR_PARSE = 2,              /* malformed einsum string */
    JA_ERR_SHAPE = 3,              /* extents / ranks disagree */
    JA_ERR_TILING = 4,             /* split points do not tile the index range (Definition 3.2 / 3.6) */
    JA_ERR_PARTITION_MISMATCH = 5, /* a relation's tiling differs from in_k(J) / out(J): repartition first (Section 4.3, sub-cost 1) */
    JA_ERR_DTYPE = 6,
    JA_ERR_UNSUPPORTED = 7,        /* no kernel for this (einsum, fn, agg, dtype) combination */
    JA_ERR_ALIGNMENT = 8,
    JA_ERR_OOM = 9,
    JA_ERR_CUDA = 10,
    JA_ERR_TIMEOUT = 11            /* a bounded device-side wait ran out (reported through ja_stream_status) */
} ja_status_t;

/* cell type of a relation. The two 16-bit types run through the same kernels (tensor cores for the contractions, f32
 * accumulation and f32 row arithmetic, one rounding to nearest even at each store); JA_F16 is the precision of the
 * paper's experiments (Section 6), JA_BF16 the one the benchmark configurations of this library are stated in. */
typedef enum { JA_F32 = 0, JA_BF16 = 1, JA_F16 = 2 } ja_dtype_t;

/* aggregation operator (+) of Definition 3.7 */
typedef enum {
    JA_AGG_NONE = 0,           /* every output type is produced by exactly one function spec */
    JA_AGG_SUM = 1,
    JA_AGG_MAX = 2,
    JA_AGG_ONLINE_SOFTMAX = 3  /* (O~,m,l) (+) (O~',m',l'): m*=max(m,m'), O~ e^(m-m*) + O~' e^(m'-m*), same for l */
} ja_agg_t;

/* concrete operator f applied to one joined tuple (Definition 3.5).  fn_params in brackets. */
typedef enum {
    JA_FN_MUL = 0,         /* product of the operands: einsum contraction                               */
    JA_FN_IDENT = 1,       /* x                                                                           */
    JA_FN_SQUARE = 2,      /* x^2                                                                         */
    JA_FN_ADD = 3,         /* x + y                                                                       */
    JA_FN_SILU_MUL = 4,    /* a / (1 + exp(-a)) * b                                                       */
    JA_FN_RMS_SCALE = 5,   /* x * (ss/n + eps)^(-1/2) * g, n = extent of the last index        [eps]     */
    JA_FN_EXP_SUB = 6,     /* exp(x - m)                                                                  */
    JA_FN_EXP_SUB_DIV = 7, /* exp(x - m) / l                                                              */
    JA_FN_ROPE = 8,        /* rotate pairs (2p,2p+1) of the last index by t*theta^(-2p/d), t = value of the
                              second index of "bshd"                                             [theta]  */
    JA_FN_ATTENTION = 9,   /* per (q-block,k-block) tuple: scale*Q K^T, causal band, partial (O~,m,l);
                              with JA_AGG_ONLINE_SOFTMAX, then O = O~/l.   [scale, causal, end_1 .. end_n]
                              Example 3.10: "bqhd,bkgd,bkgd->bqhd" is grouped-query attention, query head h joins
                              key/value head h / (extent(h)/extent(g)) and the split of h must be the split of g
                              scaled by that factor (else JA_ERR_TILING); end_1 < .. < end_n = extent(q), n <= 16,
                              are the ends of sequences packed along q and k: every end must be a split point of
                              q and of k (else JA_ERR_TILING) and only blocks of one sequence are joined          */
    JA_FN_RMSNORM = 10,    /* fused chain SQUARE/SUM -> RMS_SCALE over the last index              [eps]  */
    JA_FN_SOFTMAX = 11,    /* fused chain IDENT/MAX -> EXP_SUB/SUM -> EXP_SUB_DIV over the last index     */
    JA_FN_MATMUL_ADD = 12, /* fused chain MUL/SUM -> ADD:        "ij,jk,ik->ik"   C = A B + R                   */
    JA_FN_MATMUL_ROPE = 13,/* fused chain MUL/SUM -> ROPE:       "ij,jk->ik"      rows are tokens of sequences of
                              seq_len rows, columns are heads of head_dim cells  [theta, seq_len, head_dim]     */
    JA_FN_SWIGLU_UP = 14   /* fused chain 2 x MUL/SUM -> SILU_MUL: "ij,jk,jk->ik" silu(A B) * (A B')            */
} ja_fn_t;

typedef struct ja_spec ja_spec_t;
typedef struct ja_relation ja_relation_t;

/* Interval decomposition of one named index (Section 3.3): nparts+1 ascending split points (host),
 * splits[0] == 0, splits[nparts] == extent. */
typedef struct {
    char name;
    int64_t extent;
    int32_t nparts;
    const int64_t* splits; /* host, copied */
} ja_index_part_t;

/* ---- join-agg spec (Definition 3.6, Section 3.3) ------------------------------------------------
 * Builds J for `einsum` (lower-case letters, ',' between operands, "->" before the output, at most 4
 * operands of rank <= 4) from one ja_index_part_t per distinct letter (host array, any order).
 * fn_params: host array of n_fn_params doubles, meaning per ja_fn_t above.  accum_dtype must be JA_F32.
 * Errors: JA_ERR_PARSE, JA_ERR_SHAPE (letter without a partition / duplicate), JA_ERR_TILING,
 * JA_ERR_INVALID_ARG.  Allocates no device memory and makes no CUDA call. */
ja_status_t ja_spec_create(const char* einsum, const ja_index_part_t* parts, int32_t n_parts, ja_fn_t fn,
                           const double* fn_params, int32_t n_fn_params, ja_agg_t agg, ja_dtype_t accum_dtype,
                           ja_spec_t** out);
ja_status_t ja_spec_destroy(ja_spec_t* spec);

/* Introspection (host outputs, caller-allocated) -- the bit-exact bookkeeping surface.
 * p = number of function specs = prod_s intervals[s]. */
ja_status_t ja_spec_num_tuples(const ja_spec_t* spec, int64_t* p, int32_t* n_inputs);
/* in_keys[p][n_inputs], out_keys[p]: flat block keys of every function spec, canonical order. */
ja_status_t ja_spec_get_tuples(const ja_spec_t* spec, int32_t* in_keys, int32_t* out_keys);
/* Tiling in_k(J) (operand >= 0) or out(J) (operand == -1): rank, blocks per dimension [rank], and the
 * split points of every dimension concatenated (sum_d (nblocks[d]+1) values). */
ja_status_t ja_spec_operand_tiling(const ja_spec_t* spec, int32_t operand, int32_t* rank, int32_t* nblocks,
                                   int64_t* splits_flat);
/* Cost-model counts of Section 4.3: join_elems = sum_F sum_k |I(T^(i_k))|; agg_elems = sum over distinct
 * output types of (m-1) |I(T^(o))|.  For an a x b x c matmul grid these are (a+c)N^2 and (b-1)N^2 (Section 4.4). */
ja_status_t ja_spec_cost_terms(const ja_spec_t* spec, int64_t* join_elems, int64_t* agg_elems);

/* ---- tensor relation (Section 1, Section 3.2) -----------------------------------------------------
 * extents[rank], nparts[rank], splits[rank] (host; splits[d] has nparts[d]+1 entries). */
ja_status_t ja_relation_bytes(int32_t rank, const int64_t* extents, const int32_t* nparts,
                              const int64_t* const* splits, ja_dtype_t dtype, size_t* bytes);
/* device_ptr: DEVICE payload of at least `bytes` bytes as reported by ja_relation_bytes, 128-byte aligned,
 * borrowed.  Errors: JA_ERR_TILING, JA_ERR_ALIGNMENT, JA_ERR_INVALID_ARG (buffer too small).  No CUDA call. */
ja_status_t ja_relation_create(int32_t rank, const int64_t* extents, const int32_t* nparts,
                               const int64_t* const* splits, ja_dtype_t dtype, void* device_ptr, size_t bytes,
                               ja_relation_t** out);
/* Frees the key tables and every cached launch state or copy plan that names this relation; never the payload. */
ja_status_t ja_relation_destroy(ja_relation_t* rel);
ja_status_t ja_relation_num_blocks(const ja_relation_t* rel, int64_t* nblocks, int32_t* rank);
/* Key table (host outputs): per block, in key order, coords[rank] (int32), lower[rank], upper[rank]
 * (the tensor type = the key of the paper) and the byte offset of the block in the payload. */
ja_status_t ja_relation_get_keys(const ja_relation_t* rel, int32_t* coords, int64_t* lower, int64_t* upper,
                                 int64_t* offsets);

/* ---- execution (Definition 3.7) -------------------------------------------------------------------
 * Runs Join -> Aggregate -> Recompose of `spec` in ONE kernel launch sequence on `cuda_stream`
 * (a cudaStream_t passed as void*; NULL = the legacy default stream), asynchronously.
 * inputs[k] must be tiled exactly as in_k(J), outputs[0] as out(J) (else JA_ERR_PARTITION_MISMATCH).
 * Supported forms (letters are free; shapes of the signature matter):
 *   "ij,jk->ik"            MUL / SUM        bf16, f16 or f32 operands (one dtype for all three relations), f32 accumulate.
 *                                            bf16 / f16: tensor cores under every tiling
 *                                            (operands fetched by TMA on uniform blocks with 16-byte rows, by plain
 *                                            asynchronous loads otherwise; plain ALUs only where blocks are smaller than
 *                                            64 cells a side); f32: plain ALUs
 *   "ij,jk,ik->ik"         MATMUL_ADD / SUM   } fused chains: the accumulator of the contraction goes through the
 *   "ij,jk->ik"            MATMUL_ROPE / SUM  } next join-agg before its single rounding and store; bf16 or f16 relations
 *   "ij,jk,jk->ik"         SWIGLU_UP / SUM    } on uniform blocks only (JA_ERR_UNSUPPORTED otherwise: run the chain)
 *   "X,X->X", X any rank   ADD | SILU_MUL / NONE          key-aligned join
 *   "Rj->R"                SQUARE/SUM, IDENT/MAX          R = leading letters; f32 statistics output
 *   "Rj,R->R"              EXP_SUB / SUM
 *   "Rj,R,j->Rj"           RMS_SCALE / NONE               (R of rank 1)
 *   "Rj,R,R->Rj"           EXP_SUB_DIV / NONE
 *   "Rj,j->Rj"             RMSNORM / NONE   (fused)       "Rj->Rj"  SOFTMAX / NONE (fused)
 *   "bshd->bshd"           ROPE / NONE
 *   "bqhd,bkhd,bkhd->bqhd" ATTENTION / ONLINE_SOFTMAX     d unsplit, extent 128; any length, split points and sequence
 *   "bqhd,bkgd,bkgd->bqhd"   (grouped-query form)         ends (tensor-memory kernels where all are multiples of 128 rows,
 *                                                          mma.sync tiles for multiples of 64, a per-row form otherwise);
 *                                                          Q, K, V, O of one 16-bit dtype (bf16 or f16; the probabilities
 *                                                          enter the second product rounded to that dtype)
 *   any other einsum       MUL | ADD | IDENT | SQUARE | SILU_MUL | EXP_SUB with SUM | MAX | NONE: up to four operands
 *                          and four summed indices, any tilings and dtypes -- Definition 3.7 executed cell by cell (one
 *                          thread per output cell walks its joined tuples in ascending order): complete, not fast
 * n_outputs is 1, except for ATTENTION where it may be 2: outputs[1] then receives lse[b, q, h] = log of the softmax
 * denominator of every query row (f32, tiled like the first three indices of outputs[0]) -- with it two results over
 * disjoint key ranges combine by the online-softmax aggregation: O = w1 O1 + w2 O2, w_i = exp(lse_i - lse).
 * The first call for a given (spec, relations) tuple builds and caches tables on the device (a few
 * synchronous cudaMalloc / cudaMemcpy); later calls only launch. */
ja_status_t ja_execute(const ja_spec_t* spec, const ja_relation_t* const* inputs, int32_t n_inputs,
                       ja_relation_t* const* outputs, int32_t n_outputs, void* cuda_stream);

/* ---- repartition (Section 5.3: overlay -> atoms, decompose + recompose) ---------------------------
 * Copies the tensor held by `src` into the tiling of `dst` (same rank, extents, dtype): every atom of the
 * overlay of the two tilings moves from its source block to its destination block.  Bit-exact, no
 * aggregation.  Asynchronous on `cuda_stream`. */
ja_status_t ja_repartition(const ja_relation_t* src, ja_relation_t* dst, void* cuda_stream);
/* Overlay introspection (host, no CUDA): number of atoms, then per atom lower[rank], upper[rank],
 * flat source block, flat destination block.  Pass NULL arrays to query the count only. */
ja_status_t ja_overlay_atoms(const ja_relation_t* src, const ja_relation_t* dst, int64_t* n_atoms, int64_t* lower,
                             int64_t* upper, int32_t* src_block, int32_t* dst_block);

/* ---- a producer executed through its join, and the aggregating relayout that consumes it (Sections 5.1, 5.3) ----
 * ja_execute_join runs step (1) of Definition 3.7 alone: the concrete operator of every function spec, nothing
 * aggregated across specs. `partials` receives the unaggregated blocks as a PARTIAL RELATION: a relation of rank
 * rank(out)+1 whose leading index is the copy index c, extent m = the number of function specs per output type
 * (it must be the same for all of them), cut into its m unit intervals; the other indices are those of the output,
 * tiled as out(J). Block (c, key) holds the output of the c-th function spec (ascending F) with output type `key`.
 * Supported: "ij,jk->ik" MUL/SUM -- copy c is A[:, block c] B[block c, :]. bf16 / f16 operands on uniform blocks: tensor
 * cores, partial relation of the operands' dtype (one rounding per copy) or f32 (the accumulator as it is); otherwise plain ALUs and a
 * partial relation of the operands' dtype. Errors as ja_execute; JA_ERR_UNSUPPORTED for other forms.
 *
 * ja_repartition_agg is the one-processor image of an exchange program: every atom of the overlay of the partial
 * relation's tiling (copy index dropped) and dst's tiling has m copies; they are (+)-combined in ascending copy
 * order in f32 (agg = JA_AGG_SUM or JA_AGG_MAX; JA_AGG_NONE only when m == 1, a plain relayout) and stored once,
 * rounded once, in dst's block. partials and dst may each be f32 or a 16-bit type (the same one when both are 16-bit:
 * JA_ERR_DTYPE otherwise). partials is borrowed and
 * unchanged. Asynchronous on `cuda_stream`; the first call per (partials, dst) pair builds and caches the copy plan
 * (one synchronous cudaMalloc + cudaMemcpy). Errors: JA_ERR_SHAPE, JA_ERR_TILING (copy index not cut into unit
 * intervals), JA_ERR_INVALID_ARG (aggregation missing; dst aliases partials). */
ja_status_t ja_execute_join(const ja_spec_t* spec, const ja_relation_t* const* inputs, int32_t n_inputs,
                            ja_relation_t* partials, void* cuda_stream);
ja_status_t ja_repartition_agg(const ja_relation_t* partials, ja_agg_t agg, ja_relation_t* dst, void* cuda_stream);

/* ---- the online-softmax aggregation as a step of its own (Definition 3.7 step 2 for ATTENTION; Section 5.1) ------
 * When the function specs of an attention output key are executed apart -- m calls of ja_execute with n_outputs = 2,
 * each over its own range of the key index -- every call leaves a partial result O_c (already divided by its own
 * denominator) and lse_c. Their (+)-combination is  lse = log sum_c exp(lse_c),  O = sum_c exp(lse_c - lse) O_c,
 * the (O~, m, l) aggregation of JA_AGG_ONLINE_SOFTMAX written for normalised partials; copies are combined in
 * ascending order in f32 and O is rounded once. A partial whose lse is -inf for a row (no key of its range joined with
 * it) contributes nothing to that row; a row with no key at all gets O = 0 and lse = -inf.
 *   o_parts, lse_parts  host arrays of m (1..8) relations: O_c [b, s, h, 128] and lse_c [b, s, h] (f32); borrowed, unchanged
 *   o, lse              outputs: o of the dtype of the partials; lse f32 or NULL. Every relation may have its own tiling
 *                       (the last index unsplit).
 * Asynchronous on `cuda_stream`. Errors: JA_ERR_INVALID_ARG (NULL, aliasing), JA_ERR_SHAPE, JA_ERR_DTYPE,
 * JA_ERR_UNSUPPORTED (m outside 1..8). */
ja_status_t ja_attention_combine(const ja_relation_t* const* o_parts, const ja_relation_t* const* lse_parts, int32_t m,
                                 ja_relation_t* o, ja_relation_t* lse, void* cuda_stream);

/* ---- logical optimization (Section 4.2, Algorithm 1; cost proxy of Section 4.3) -------------------------------
 * Chooses one join-agg spec per abstract operator of a computation TREE (every node but the last is consumed by
 * exactly one later node; the last node produces the result) for p processors = p function specs per operator.
 * A spec is the vector of interval counts of the operator's letters, in order of first appearance (near-equal
 * intervals, Section 3.3); specs(Op) are all count vectors whose product is p (fixed letters keep one interval).
 * Cost(J, T_1..T_n) = repartition (the cells of operand k when its producer's output tiling differs from in_k(J);
 * nothing for inputs of the computation) + join (the cells of every input block of every function spec) +
 * aggregation ((m-1) x the cells of every distinct output type). The dynamic program keeps, per operator and per
 * output tiling, the cheapest spec and the producers' tilings that achieved it, and walks back from the root.
 * All arrays are HOST memory; no CUDA call is made.
 *   counts   out, [n_nodes][JA_PLAN_MAX_LETTERS]: interval count per letter of the chosen spec (0 beyond the letters)
 *   total_cost  out (may be NULL): the minimum of the summed Cost
 * ja_plan_cost evaluates the summed Cost of a given assignment (same layout of `counts`).
 * Errors: JA_ERR_PARSE, JA_ERR_SHAPE (operand / producer mismatch), JA_ERR_INVALID_ARG (not a tree in topological
 * order), JA_ERR_UNSUPPORTED (a node consumed twice: ja_plan_optimize_graph handles that, Section 4.5; more than 8 letters),
 * JA_ERR_TILING (no decomposition into p function specs). */
#define JA_PLAN_MAX_LETTERS 8
typedef struct {
    const char* einsum;       /* signature of the abstract operator, as for ja_spec_create */
    const int64_t* extents;   /* one per distinct letter, in order of first appearance */
    const int32_t* producers; /* one per operand: index of the node that produces it (smaller than this node's), or -1 */
    uint32_t fixed_letters;   /* bit l set: the l-th letter is not shardable */
} ja_plan_node_t;
ja_status_t ja_plan_optimize(const ja_plan_node_t* nodes, int32_t n_nodes, int32_t p, int32_t* counts, int64_t* total_cost);
ja_status_t ja_plan_cost(const ja_plan_node_t* nodes, int32_t n_nodes, const int32_t* counts, int64_t* total_cost);
/* Outputs with several consumers (Section 4.5): the graph (nodes in topological order; a node may be consumed any number
 * of times) is cut at every edge out of a multiply consumed tensor; the resulting trees are optimised with Algorithm 1
 * one at a time, largest first (ties: smaller root first), each subject to the specs already fixed: an operand produced
 * in an already-optimised tree enters like an input of the computation whose tiling is fixed (Cost charges the repartition
 * on a mismatch); an operand produced in a tree still to come enters like a free input; the root of a tree is chosen with
 * the repartition charges of its already-planned consumers added. total_cost is the summed Cost of the assembled plan
 * (what ja_plan_cost returns for it). On a tree the result equals ja_plan_optimize. */
ja_status_t ja_plan_optimize_graph(const ja_plan_node_t* nodes, int32_t n_nodes, int32_t p, int32_t* counts, int64_t* total_cost);
/* The greedy selector the paper compares its optimizer with (Section 6, Experiment 3): the same program without the
 * repartition sub-cost, so every operator independently takes the spec of least join + aggregation cost (the first one in
 * the enumeration order of its specs). Trees and graphs alike. *total_cost is the full Cost of the plan it returns,
 * repartition charges included: never below what ja_plan_optimize finds on a tree. */
ja_status_t ja_plan_select_greedy(const ja_plan_node_t* nodes, int32_t n_nodes, int32_t p, int32_t* counts, int64_t* total_cost);

/* ---- relayout without allocation -------------------------------------------------------------------
 * (The paper has no counterpart to this call: it exists for callers of THIS library that cannot allocate.)
 * Same data movement as ja_repartition -- every atom of the overlay of the two tilings is copied from its
 * source block to its destination block, bit-exact -- for callers that must not trigger a device (or host)
 * allocation: servers that gave all of HBM to their own pool at start-up, loops that must never take
 * cudaMalloc's implicit device synchronisation, harnesses that fail on any allocation they did not make.
 * It takes the tilings and the payload pointers directly (no relation handles), keeps its copy plan in a
 * fixed device array inside the library (16384 slabs, 512 KiB per GPU, held until process exit) and calls no
 * cudaMalloc / cudaFree / allocating routine.
 *   extents[rank]; src_nparts / dst_nparts [rank]; src_splits / dst_splits [rank] pointers to nparts+1
 *   ascending split points each (all HOST); src_device / dst_device: DEVICE payloads in block-key layout,
 *   128-byte aligned, distinct, sized as ja_relation_bytes reports for their tilings.
 * Limits (JA_ERR_UNSUPPORTED beyond them): 16384 copy slabs (one per atom row-chunk of <= 64 KiB), 4096 blocks
 * per tiling, 1024 overlay split points per dimension.
 * All calls share the plan array; it keeps the last call's contents and a call reads only what it has just
 * written, so nothing needs clearing -- but calls whose GPU work overlaps race on it: serialise them.
 * The first call on each device resolves the array's device address; issue it before any stream capture.
 * The plan reaches the device by a stream-ordered copy from a fixed host table (the host may block briefly while it is
 * read); a call on a stream that is being captured is refused with JA_ERR_UNSUPPORTED and enqueues nothing. */
ja_status_t ja_repartition_noalloc(int32_t rank, const int64_t* extents, const int32_t* src_nparts,
                                   const int64_t* const* src_splits, const int32_t* dst_nparts,
                                   const int64_t* const* dst_splits, ja_dtype_t dtype, const void* src_device,
                                   void* dst_device, void* cuda_stream);

/* Device-detected conditions (a bounded wait that ran out: JA_ERR_TIMEOUT) are recorded in a status word that belongs
 * to the stream the kernel was launched on (per device a fixed table of 64 words; the 64th and later streams of a device
 * share the last one). This call synchronizes `cuda_stream`, returns that stream's word in *device_status and clears it.
 * After JA_ERR_TIMEOUT the outputs of the launches since the last call are undefined; the context stays usable and later
 * launches run normally. */
ja_status_t ja_stream_status(void* cuda_stream, ja_status_t* device_status);

/* ---- switches and test hooks (no counterpart in the paper) ---------------------------------------------------------
 * Every device-side wait of the kernels is bounded (default 2 s; JA_WAIT_CAP=<nanoseconds> in the environment). The
 * environment (JA_* variables: the wait limit and switches that force a kernel form or a schedule) is read ONCE, when the
 * library is first used; ja_debug_set changes a value afterwards. Names: "wait_cap_ns", "attn_mma_sync", "attn_one_tile",
 * "attn_persistent", "attn_section", "attn_variant", "gemm_cta_group", "gemm_group_m", "gemm_heavy_first", "gemm_split",
 * "gemm_loader", "row_tma", "row_team"; -1 = not forced. JA_ERR_INVALID_ARG for an unknown name or a value out of range. */
ja_status_t ja_debug_set(const char* name, int64_t value);
/* Launches one CTA that waits, with the configured limit, on a barrier nothing arrives at: the wait runs out, the kernel
 * records JA_ERR_TIMEOUT in the stream's status word and returns normally (no trap, no fault). waiters_ok: optional
 * DEVICE array of two ints, set to 0 / 0 (the waiter whose limit ran out, and a second waiter that gave up on the abort
 * flag). For tests of the failure path; asynchronous on `cuda_stream`. */
ja_status_t ja_debug_wait_timeout(void* cuda_stream, int32_t* waiters_ok);
/* The same wait loop run on the HOST against a scripted barrier and clock (no CUDA call): the barrier completes at poll
 * `ready_at_poll` (counted from 1; <= 0 never), the clock advances ns_per_poll per poll, another role raises the abort
 * flag at poll abort_at_poll (<= 0 never). Outputs (any may be NULL): polls made, success, whether this waiter recorded
 * the time-out, clock at return. */
ja_status_t ja_debug_bounded_wait_host(int64_t ready_at_poll, int64_t ns_per_poll, int64_t cap_ns, int64_t abort_at_poll,
                                       int64_t* polls, int32_t* succeeded, int32_t* recorded_timeout, int64_t* elapsed_ns);

/* Number of kernels this library has launched since load (for launch accounting by callers). */
int64_t ja_launch_count(void);

const char* ja_last_error(void);
const char* ja_version(void);

#ifdef __cplusplus
}
#endif
#endif /* JA_H_ */
