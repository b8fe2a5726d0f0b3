/* ja_exprog.h -- exchange programs (Section 5, "Physical Optimization"): the ExProg language, its validity check, the
 * simulator's cost model, preamble generation, body synthesis, and the execution of a program on ONE GPU.
 *
 * Part of libja.so; same conventions as ja.h (ja_status_t, ja_last_error, opaque handles, plain pointers and sizes).
 * Every function here except ja_exchange_execute is HOST code that makes no CUDA call; all pointers are HOST pointers.
 *
 * Text form (Section 5.2; a reading of the printed examples):
 *     GPUS: 0, 1, 2, 3                       optional; default = the sites named anywhere in the program
 *     PARTITIONS: G1 {size 2} G2 {2, 3}      by size (members chosen later) or by explicit members; disjoint, covering GPUS
 *     IN:  A @ 0 (size: 1.0 GB); B @ 1       ';' or a line break between items; sizes default to 1 GB (1e9 bytes)
 *     OUT: A+B @ 0, 1; C @ G1
 *     <blank line>
 *     A @ 0 -> 1;  B @ 1 -> 0;  A+B @ 0, 1   the body, a SET of actions "aggregate @ source(s) [-> destinations]"
 * An action with an arrow has one source site; without one its source may be a list of sites or a partition name (one
 * local aggregation per site).  At most 64 atoms; sites are integers 0..63.  An aggregate is handed through this
 * interface as a 64-bit mask over the atoms in declaration order; a set of sites as a 64-bit mask over site numbers.
 * "Expanded" actions are the actions with one source site each, in body order, the sites of a list or partition in
 * their declared / ascending order, duplicates dropped; they need every partition's members to be known. */
#ifndef JA_EXPROG_H
#define JA_EXPROG_H

#include "ja.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ja_exprog ja_exprog_t;

/* ---- the simulator's machine model (Section 5.2 "Cost") ------------------------------------------------------------
 * Bandwidths in GB/s (1e9 bytes per second).  NVSWITCH: a fully non-blocking all-to-all fabric, contention only at the
 * endpoints: every site sends at most link_gbs and receives at most link_gbs; a multicast to k sites is k flows.
 * CUBE_MESH: eight sites; i <-> i + 4 are double links (double_gbs per direction), pairs inside {0..3} and inside {4..7}
 * single links (link_gbs), every other pair shares one bridge of pcie_gbs in total (the paper names the four double
 * links and says that pairs inside a CPU socket have single ones; the rest of the table is this library's reading).
 * LINKS: any point-to-point topology given as a table of directed link capacities; flows on one directed link share it,
 * flows between unlinked pairs share the bridge -- the cube mesh is the special case ja_machine_preset("dgx_v100") fills in. */
typedef enum { JA_FABRIC_NVSWITCH = 0, JA_FABRIC_CUBE_MESH = 1, JA_FABRIC_LINKS = 2 } ja_fabric_t;
typedef struct {
    int32_t fabric;    /* ja_fabric_t */
    int32_t n_sites;
    double hbm_gbs;    /* local aggregation: an aggregate of m >= 2 parts reads m and writes 1 block at this rate */
    double link_gbs;
    double double_gbs; /* CUBE_MESH only */
    double pcie_gbs;   /* CUBE_MESH and LINKS: the bridge that every transfer between unlinked pairs shares */
    const double* links; /* LINKS only: n_sites x n_sites, links[a * n_sites + b] = GB/s of the direct link a -> b, 0 = none
                            (the transfer goes over the bridge); HOST memory that outlives the calls given this machine */
} ja_machine_t;
/* "dgx_h100" (450 / 3350), "dgx_a100" (300 / 2039), "hgx_b200" (900 / 7700), "dgx_v100" (25, 50, 15.75 / 900).  The H100
 * and V100 figures reproduce the completion times of the paper's three examples. JA_ERR_INVALID_ARG for another name. */
ja_status_t ja_machine_preset(const char* name, ja_machine_t* out);

/* ---- programs ------------------------------------------------------------------------------------------------------
 * ja_exprog_parse: preamble and (possibly empty) body from text.  JA_ERR_PARSE for malformed text, an unknown atom, an
 * atom declared twice, an arrow after several sources; JA_ERR_INVALID_ARG for partitions that overlap, name an
 * undeclared site or do not cover GPUS, an atom at an undeclared site, an aggregate whose atoms differ in size, more
 * than 64 atoms or a site above 63.  The handle is owned by the caller (ja_exprog_destroy). */
ja_status_t ja_exprog_parse(const char* text, ja_exprog_t** out);
ja_status_t ja_exprog_clone(const ja_exprog_t* p, ja_exprog_t** out);
/* One program out of two over the same GPUS and PARTITIONS (names, sizes and members must agree) -- the exchanges of two
 * operands of one operator, which share the placement of its function specs and run at the same time: a's atoms, renamed
 * prefix_a + name, then b's, renamed prefix_b + name; OUT and the bodies likewise, a's first.  JA_ERR_INVALID_ARG if the
 * preambles disagree, names clash, or there are more than 64 atoms. */
ja_status_t ja_exprog_merge(const ja_exprog_t* a, const ja_exprog_t* b, const char* prefix_a, const char* prefix_b,
                            ja_exprog_t** out);
void ja_exprog_destroy(ja_exprog_t* p);
/* The program as text that ja_exprog_parse reads back to the same program.  Writes at most cap bytes including the
 * terminating zero; *needed receives the size of the whole text with its zero (JA_ERR_INVALID_ARG if cap is smaller). */
ja_status_t ja_exprog_format(const ja_exprog_t* p, char* buf, int64_t cap, int64_t* needed);
/* Any pointer may be NULL.  n_expanded is -1 while a partition used by the body has no members. */
ja_status_t ja_exprog_counts(const ja_exprog_t* p, int32_t* n_gpus, int32_t* n_partitions, int32_t* n_atoms,
                             int32_t* n_out, int32_t* n_actions, int32_t* n_expanded);
/* Expanded actions: aggregate[i], source[i], dests[i] (mask).  Arrays of n_expanded entries; JA_ERR_INVALID_ARG while a
 * partition has no members. */
ja_status_t ja_exprog_get_actions(const ja_exprog_t* p, uint64_t* aggregate, int32_t* source, uint64_t* dests);
/* Requirements of OUT, one per (aggregate, site): pass NULL arrays to get the count. */
ja_status_t ja_exprog_get_requirements(const ja_exprog_t* p, int32_t* n, uint64_t* aggregate, int32_t* site);
/* Atoms: site[i], size_gb[i] in declaration order. */
ja_status_t ja_exprog_get_atoms(const ja_exprog_t* p, int32_t* site, double* size_gb);

/* ---- partitions declared by size alone (Section 5.2: their members are the compiler's choice) ----------------------
 * The memberships are enumerated partition by partition in declaration order, each taking a combination (in
 * lexicographic order) of the sites that the explicit partitions and the earlier ones left.  ja_exprog_bind writes the
 * index-th membership into the program (partitions then have explicit members); ja_exprog_membership reports the
 * members of one partition as a site mask.  ja_exprog_num_memberships is the closed-form count; ja_exprog_bind by index
 * and ja_exprog_valid_any list the memberships and refuse (JA_ERR_UNSUPPORTED) more than a million of them. */
ja_status_t ja_exprog_num_memberships(const ja_exprog_t* p, int64_t* n);
ja_status_t ja_exprog_bind(ja_exprog_t* p, int64_t index);
ja_status_t ja_exprog_membership(const ja_exprog_t* p, const char* partition, uint64_t* members);
/* Gives one size-declared partition explicit members (n = its size; JA_ERR_INVALID_ARG if they overlap another
 * partition's, are not declared GPUs, or the partition already has members). */
ja_status_t ja_exprog_bind_members(ja_exprog_t* p, const char* partition, const int32_t* sites, int32_t n);

/* ---- Definition "Closure; validity" (Section 5.4) -------------------------------------------------------------------
 * ja_exprog_closure: S*(P) as (aggregate, site) pairs sorted by site, then by mask; NULL arrays to get the count.
 * ja_exprog_check: well_formed = every action is enabled by S*(P); valid = well-formed and every requirement of OUT is
 * in S*(P).  Both need bound memberships (JA_ERR_INVALID_ARG otherwise).  ja_exprog_valid_any: valid under SOME
 * membership of the size-declared partitions. */
ja_status_t ja_exprog_closure(const ja_exprog_t* p, int64_t* n, uint64_t* aggregate, int32_t* site);
ja_status_t ja_exprog_check(const ja_exprog_t* p, int32_t* well_formed, int32_t* valid);
ja_status_t ja_exprog_valid_any(const ja_exprog_t* p, int32_t* valid);

/* ---- the simulator (Section 5.2: an unordered body; two-stage actions; the cost model) -------------------------
 * An action starts when aggregates materialised at its source partition its aggregate (the partition with the fewest
 * parts available then); m >= 2 parts cost (m + 1) x size / hbm_gbs, one part nothing; its transfers start when the
 * aggregation ends.  Concurrent work shares a resource equally (aggregations at a site; flows at an endpoint, on a
 * directed link, on the bridge).  completion_ms = the time the last action finishes.  The three optional arrays
 * (n_expanded entries) receive per expanded action the times it started, finished aggregating and finished, in ms.
 * JA_ERR_INVALID_ARG if an action never becomes enabled (the program is not well-formed) or memberships are unbound. */
ja_status_t ja_exprog_simulate(const ja_exprog_t* p, const ja_machine_t* machine, double* completion_ms,
                               double* start_ms, double* aggregated_ms, double* finish_ms);

/* ---- bodies (Section 5.4) ----------------------------------------------------------------------------------------------
 * ja_exprog_body: replaces the body.  JA_BODY_NAIVE = the trivial valid program (one multicast per atom to the sites
 * that need it, one local aggregation per requirement); JA_BODY_BUTTERFLY = recursive doubling for every required
 * aggregate whose targets are exactly the 2^k sites that hold its atoms, equally many each (round b: position i of the
 * ascending target list sends to position i xor 2^b), the rest as in the naive body.  Needs bound memberships.
 * ja_exprog_normalise: rewrites the body as its expanded actions (one source site per action).
 * ja_exprog_rewrite: one rule application on a normalised program; *applied = 0 (and the program unchanged) when the
 * rule does not match or its guard fails -- the result of Insert must be well-formed, of every other rule valid.
 *   JA_RULE_INSERT        a = aggregate, i = source site, b = destination mask
 *   JA_RULE_DELETE        i = action
 *   JA_RULE_FISSION       i = action, a = the destinations split off            X @ s -> D1 u D2  =>  X @ s -> D1, X @ s -> D2
 *   JA_RULE_FUSION        i, j = actions                                       the reverse
 *   JA_RULE_RELAY_IN      i = action, j = destination, a = relay site          X @ s -> d  =>  X @ s -> r, X @ r -> d
 *   JA_RULE_RELAY_OUT     i, j = actions                                       the reverse
 *   JA_RULE_PUSHDOWN      i, j = actions                                       X @ r -> s, Y @ r -> s  =>  X+Y @ r -> s
 *   JA_RULE_PULLUP        i = action, a = the part split off, b != 0: put X+Y @ s back as a local aggregation
 *   JA_RULE_SOURCE        i = action, j = another site where the aggregate is materialised
 * ja_exprog_synthesize: beam search through the rules (every candidate checked by the definition and costed by the
 * simulator) from the program's own body, or, if it is empty, from the better of the naive and the butterfly body; keeps
 * the best program seen and reports its time.  The paper leaves the search procedure open.
 * ja_exprog_place: chooses the members of the size-declared partitions -- among the memberships under which the program
 * is valid the one with the least simulated time (among equal times the one that sends the fewest bytes, then the
 * first), with body = JA_BODY_OWN (the program's body as it is), JA_BODY_NAIVE, JA_BODY_BUTTERFLY or JA_BODY_BEST (the
 * better of the two constructed ones) rebuilt per membership.  Above 5000 memberships they are not enumerated: the
 * search starts from the first one (the free sites dealt to the partitions in ascending order) and repeatedly takes the
 * exchange of two sites between two partitions that lowers the simulated time most -- or, at equal time, the bytes
 * sent -- (the first of equals, pairs in ascending order), until none does.
 * The program is left bound to the chosen membership with the chosen body.  JA_ERR_INVALID_ARG if none is valid. */
typedef enum { JA_BODY_OWN = 0, JA_BODY_NAIVE = 1, JA_BODY_BUTTERFLY = 2, JA_BODY_BEST = 3 } ja_body_t;
typedef enum {
    JA_RULE_INSERT = 0, JA_RULE_DELETE = 1, JA_RULE_FISSION = 2, JA_RULE_FUSION = 3, JA_RULE_RELAY_IN = 4,
    JA_RULE_RELAY_OUT = 5, JA_RULE_PUSHDOWN = 6, JA_RULE_PULLUP = 7, JA_RULE_SOURCE = 8
} ja_rule_t;
ja_status_t ja_exprog_body(ja_exprog_t* p, int32_t body);
ja_status_t ja_exprog_normalise(ja_exprog_t* p);
ja_status_t ja_exprog_rewrite(ja_exprog_t* p, int32_t rule, int32_t i, int32_t j, uint64_t a, uint64_t b, int32_t* applied);
ja_status_t ja_exprog_synthesize(ja_exprog_t* p, const ja_machine_t* machine, int32_t depth, int32_t beam, double* ms);
ja_status_t ja_exprog_place(ja_exprog_t* p, const ja_machine_t* machine, int32_t body, double* ms);

/* ---- preamble generation (Section 5.3) ------------------------------------------------------------------------------
 * The preamble that links a compiled producer to one input of op.  The tensor has `rank` indices; producer_splits and
 * consumer_splits hold, per index, the split points of out(J_k) and of in_k(J) (n_*_splits[d] values each, first 0, last
 * the extent), one index after the other.  Copy c of producer block b (flat key, row-major over the producer's grid)
 * lives on GPU copy_site[b * m + c]; function spec i of op consumes the in_k block consumer_specs[i] (flat key) and there
 * is one spec per GPU.  Atoms are the cells of the overlay of the two tilings in row-major order; IN gets one atom per
 * (atom, copy), named "a<atom>_<copy>", listed by site and then by atom, of size cardinality x width_bytes; PARTITIONS
 * one partition "S<i+1>" of size one per function spec; OUT the aggregate of an atom's m copies at the partition of
 * every function spec whose block contains it. */
ja_status_t ja_exprog_preamble(int32_t rank, const int64_t* producer_splits, const int32_t* n_producer_splits,
                               const int64_t* consumer_splits, const int32_t* n_consumer_splits, int32_t m,
                               const int32_t* copy_site, const int32_t* consumer_specs, int32_t n_specs,
                               int32_t width_bytes, ja_exprog_t** out);

/* ---- an exchange program executed on ONE GPU (Sections 5.2 - 5.3) ----------------------------------------------------
 * The sites of the program are regions of this GPU's memory.  `partials` is a partial relation (ja.h: rank(dst) + 1, the
 * copy index in front, cut into its m unit intervals, the other indices tiled as the producer's out(J_k)); `dst` is tiled
 * as in_k(J), same cell type; copy_site and consumer_specs are those given to ja_exprog_preamble, and `prog` must be a
 * bound, valid program over exactly the preamble they generate (JA_ERR_INVALID_ARG otherwise).  Steps, all enqueued on
 * `cuda_stream`: decompose (every resident copy of a producer block is sliced into its atoms, one batched launch), the
 * actions in a firing order of the program (repeated passes over the expanded actions in body order; an action fires the
 * first time aggregates at its source partition its aggregate) -- a local aggregation of m >= 2 parts is one launch that
 * combines them in ascending order of their first atoms in f32 (SUM or MAX) and rounds once to the cell type, a transfer
 * one device-to-device copy -- and recompose (the aggregated atoms at the site of function spec i are concatenated into
 * the block it consumes; a block consumed by several specs is written from the lowest one).  At most 16 parts per
 * aggregation, tensors of rank <= 3; a second delivery of an aggregate to a site that already holds it moves nothing.  Scratch memory for the atom buffers comes from a stream-ordered memory pool of the
 * library's own and goes back to it, in stream order, at the end of the call; the pool keeps it for the next call until
 * ja_exchange_trim (which the caller synchronises before) hands it back to the driver.  Not capturable: a call on a stream
 * that is being captured is refused (JA_ERR_UNSUPPORTED, nothing enqueued); the call may block the host briefly while its
 * tables are staged.  stats (optional, HOST, 5 values):
 * local aggregations launched, transfers, bytes transferred, scratch bytes, bytes read and written by the aggregations. */
ja_status_t ja_exchange_execute(const ja_exprog_t* prog, const ja_relation_t* partials, const int32_t* copy_site,
                                const int32_t* consumer_specs, int32_t n_specs, ja_agg_t agg, ja_relation_t* dst,
                                int64_t* stats, void* cuda_stream);
ja_status_t ja_exchange_trim(void);

/* ---- an exchange plan: the executable artifact (Section 5.1: what the compiler emits is a CUDA graph of kernel nodes and
 * transfer nodes) -------------------------------------------------------------------------------------------------------
 * ja_exchange_plan_create does once what ja_exchange_execute does per call -- checks, firing order, buffers, tables --
 * and keeps the atom buffers and tables in device memory of its own (synchronous cudaMalloc / cudaMemcpy; JA_ERR_OOM if
 * the buffers do not fit).  The relations' payload addresses are bound into the plan: both relations must outlive it
 * and keep their payloads in place; what the payloads hold may change between runs.
 * ja_exchange_plan_run only enqueues: decompose on `cuda_stream`; then every step on the stream of its SITE (the plan
 * owns one stream per site that acts), after the events of the buffers that other sites' streams write -- so actions
 * proceed as dataflow allows, as Section 5.2 says a program does, and transfers (copy engines) overlap aggregations --
 * then recompose on `cuda_stream` once every site's stream has been joined.  It may be called while `cuda_stream` is
 * being captured: the capture then holds the program's dependency graph, and replaying it needs no host work.  Runs of
 * one plan must not overlap (they share the buffers); the results are those of ja_exchange_execute, bit for bit. */
typedef struct ja_exchange_plan ja_exchange_plan_t;
ja_status_t ja_exchange_plan_create(const ja_exprog_t* prog, const ja_relation_t* partials, const int32_t* copy_site,
                                    const int32_t* consumer_specs, int32_t n_specs, ja_agg_t agg, ja_relation_t* dst,
                                    int64_t* stats, ja_exchange_plan_t** out);
/* The same with the sites spread over the devices of this process: site s lives on the device with label site_device[s]
 * (s < n_site_device; other sites, and all of them when site_device is NULL, live on the HOME device, the one current at
 * creation, whose label is its ordinal).  A site's buffers are allocated on its device, its aggregations launched there on
 * its own stream, and a transfer is a copy between the two devices' buffers (cudaMemcpyAsync under unified addressing, which a
 * stream capture can record) -- no kernel ever reads another device's memory.  Both relations live on the home device: atoms of sites elsewhere are sliced
 * into a staging area at home and sent to their sites before the program starts, and the aggregates that function specs
 * elsewhere end with are brought home before recompose (on a machine whose producers and consumers run on those devices
 * these two hops are the operators' own outputs and inputs).  A label beyond the visible devices wraps around (label modulo
 * the device count), so every path of a multi-device plan also runs on fewer GPUs, down to one.  ja_exchange_plan_run must
 * be called with the home device current. */
ja_status_t ja_exchange_plan_create_on(const ja_exprog_t* prog, const ja_relation_t* partials, const int32_t* copy_site,
                                       const int32_t* consumer_specs, int32_t n_specs, ja_agg_t agg, ja_relation_t* dst,
                                       const int32_t* site_device, int32_t n_site_device, int64_t* stats, ja_exchange_plan_t** out);
ja_status_t ja_exchange_plan_run(ja_exchange_plan_t* plan, void* cuda_stream);
void ja_exchange_plan_destroy(ja_exchange_plan_t* plan);

/* ---- the pieces a program needs when its sites are different processes (one per GPU) ------------------------------------
 * ja_exprog_schedule: the firing order ja_exchange_execute uses, for a driver that issues the actions itself: fired action
 * k is expanded action action[k] and aggregates parts[part_begin[k] .. part_begin[k + 1]) (masks, in combination order;
 * one part = the aggregate is already materialised, nothing to compute).  Every process derives the same order from the
 * same program.  NULL arrays to get the two counts; part_begin has n_fired + 1 entries.  JA_ERR_INVALID_ARG if the
 * program is not well-formed.  Host only.
 * ja_exchange_combine: the local aggregation stage of one action on DEVICE buffers: out = parts[0] (+) parts[1] (+) ... in
 * that order (2..16 parts; SUM or MAX in f32, one rounding to `dtype`).  All buffers hold `bytes` bytes, a multiple of 16,
 * and are 16-byte aligned (JA_ERR_ALIGNMENT otherwise); out may not alias a part.  Asynchronous on cuda_stream. */
ja_status_t ja_exprog_schedule(const ja_exprog_t* p, int32_t* n_fired, int32_t* n_parts_total, int32_t* action,
                               int32_t* part_begin, uint64_t* parts);
ja_status_t ja_exchange_combine(const void* const* parts, int32_t n_parts, void* out, int64_t bytes, ja_dtype_t dtype,
                                ja_agg_t agg, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif
