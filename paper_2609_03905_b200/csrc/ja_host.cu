// Host side of libja: einsum parsing, join-agg spec enumeration (Definition 3.6, Section 3.3), tensor
// relation key tables (Section 1 / 3.2), overlay planning for repartition (Section 5.3), and the
// dispatch of ja_execute (Definition 3.7) to the sm_100a kernels. No arithmetic on tensor values
// happens on the host.
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <iterator>
#include <cmath>
#include <mutex>
#include <set>

#include "ja_internal.h"
#include "ja_wait.h"

// ---------------------------------------------------------------------------------------------------
// errors, counters, device status word
// ---------------------------------------------------------------------------------------------------
static thread_local char g_err[512] = "";
static std::atomic<int64_t> g_launches{0};
static std::atomic<uint64_t> g_next_id{1};
#define JA_STATUS_SLOTS 64
#define JA_MAX_DEVICES 64
__device__ int g_ja_status_words[JA_STATUS_SLOTS];

ja_status_t ja_fail(ja_status_t st, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return st;
}

ja_status_t ja_cuda_fail(cudaError_t e, const char* what) {
    return ja_fail(JA_ERR_CUDA, "CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
}

void ja_count_launch(int n) { g_launches += n; }

// ---- configuration: the environment is read once -------------------------------------------------------------
static int env_int(const char* name, int dflt) {
    const char* v = getenv(name);
    return (v && *v) ? atoi(v) : dflt;
}
JaConfig& ja_config() {
    static JaConfig cfg;
    static std::once_flag once;
    std::call_once(once, [] {
        cfg.attn_mma_sync = env_int("JA_ATTN_MMA_SYNC", -1);
        cfg.attn_one_tile = env_int("JA_ATTN_ONE_TILE", -1);
        cfg.attn_persistent = env_int("JA_ATTN_PERSISTENT", -1);
        cfg.attn_section = env_int("JA_ATTN_SECTION", -1);
        cfg.attn_variant = env_int("JA_ATTN_VARIANT", -1);
        cfg.gemm_cta_group = env_int("JA_GEMM_CTA_GROUP", -1);
        cfg.gemm_group_m = env_int("JA_GEMM_GROUP_M", -1);
        cfg.gemm_heavy_first = env_int("JA_GEMM_HEAVY_FIRST", -1);
        cfg.gemm_split = env_int("JA_GEMM_SPLIT", -1);
        cfg.gemm_loader = env_int("JA_GEMM_LOADER", -1);
        cfg.row_tma = env_int("JA_ROW_TMA", -1);
        cfg.row_team = env_int("JA_ROW_TEAM", -1);
        cfg.row_reduce = env_int("JA_ROW_REDUCE", -1);
        if (const char* v = getenv("JA_WAIT_CAP")) {
            const long long ns = atoll(v);
            if (ns >= 1000 && ns <= 4000000000000ll) cfg.wait_cap_us = ns / 1000;
        }
    });
    return cfg;
}

extern "C" ja_status_t ja_debug_set(const char* name, int64_t value) {
    if (!name) return ja_fail(JA_ERR_INVALID_ARG, "name is NULL");
    JaConfig& c = ja_config();
    const std::string n(name);
    struct { const char* key; int* field; } ints[] = {
        {"attn_mma_sync", &c.attn_mma_sync}, {"attn_one_tile", &c.attn_one_tile}, {"attn_persistent", &c.attn_persistent},
        {"attn_section", &c.attn_section}, {"attn_variant", &c.attn_variant}, {"gemm_cta_group", &c.gemm_cta_group},
        {"gemm_group_m", &c.gemm_group_m}, {"gemm_heavy_first", &c.gemm_heavy_first}, {"gemm_split", &c.gemm_split},
        {"gemm_loader", &c.gemm_loader}, {"row_tma", &c.row_tma}, {"row_team", &c.row_team},
        {"row_reduce", &c.row_reduce}};
    for (auto& e : ints)
        if (n == e.key) {
            *e.field = (int)value;
            return JA_OK;
        }
    if (n == "wait_cap_ns") {
        if (value < 1000 || value > 4000000000000ll) return ja_fail(JA_ERR_INVALID_ARG, "wait_cap_ns must lie in [1e3, 4e12]");
        c.wait_cap_us = value / 1000;
        return JA_OK;
    }
    return ja_fail(JA_ERR_INVALID_ARG, "unknown switch '%s'", name);
}

// ---- per-device state: status words, multiprocessor count ------------------------------------------------------
struct DeviceState {
    int* words = nullptr;                    // device address of g_ja_status_words on this device
    std::map<cudaStream_t, int> slot_of;     // stream -> word
    int sms = 0;
};
static std::mutex g_dev_mu;
static DeviceState g_dev[JA_MAX_DEVICES];

static DeviceState* device_state_locked() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= JA_MAX_DEVICES) return nullptr;
    DeviceState* d = &g_dev[dev];
    if (!d->words && cudaGetSymbolAddress((void**)&d->words, g_ja_status_words) != cudaSuccess) d->words = nullptr;
    if (!d->sms && (cudaDeviceGetAttribute(&d->sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || d->sms < 1)) d->sms = 148;
    return d;
}

int* ja_device_status_word(cudaStream_t st) {
    std::lock_guard<std::mutex> lk(g_dev_mu);
    DeviceState* d = device_state_locked();
    if (!d || !d->words) return nullptr;
    auto it = d->slot_of.find(st);
    if (it == d->slot_of.end()) {
        const int slot = std::min<int>((int)d->slot_of.size(), JA_STATUS_SLOTS - 1);
        it = d->slot_of.emplace(st, slot).first;
    }
    return d->words + it->second;
}

int ja_sm_count() {
    std::lock_guard<std::mutex> lk(g_dev_mu);
    DeviceState* d = device_state_locked();
    return d ? d->sms : 148;
}

extern "C" const char* ja_last_error(void) { return g_err; }
extern "C" const char* ja_version(void) { return "libja 0.2 (sm_100a)"; }
extern "C" int64_t ja_launch_count(void) { return g_launches.load(); }

extern "C" ja_status_t ja_stream_status(void* cuda_stream, ja_status_t* device_status) {
    if (!device_status) return ja_fail(JA_ERR_INVALID_ARG, "device_status is NULL");
    JA_CUDA(cudaStreamSynchronize((cudaStream_t)cuda_stream));
    int* w = ja_device_status_word((cudaStream_t)cuda_stream);
    if (!w) return ja_fail(JA_ERR_CUDA, "cannot resolve the device status word");
    int v = 0;
    JA_CUDA(cudaMemcpy(&v, w, sizeof v, cudaMemcpyDeviceToHost));
    *device_status = (ja_status_t)v;
    if (v != 0) {
        int zero = 0;
        JA_CUDA(cudaMemcpy(w, &zero, sizeof zero, cudaMemcpyHostToDevice));
        ja_attention_reset_queues();
    }
    return JA_OK;
}

// ---- the bounded wait, run on the host against a scripted barrier and clock (tests) ------------------------------
// The barrier completes at poll number `ready_at_poll` (counting from 1; <= 0: never); the clock advances `ns_per_poll`
// per poll; another role raises the abort flag at poll `abort_at_poll` (<= 0: never). Outputs: polls made, whether the
// wait succeeded, whether THIS waiter recorded the time-out, and the clock when it returned.
extern "C" ja_status_t ja_debug_bounded_wait_host(int64_t ready_at_poll, int64_t ns_per_poll, int64_t cap_ns, int64_t abort_at_poll,
                                                  int64_t* polls, int32_t* succeeded, int32_t* recorded_timeout, int64_t* elapsed_ns) {
    if (ns_per_poll < 0 || cap_ns < 0) return ja_fail(JA_ERR_INVALID_ARG, "negative time");
    int64_t n = 0;
    bool failed = false;
    const bool ok = ja_bounded_wait([&] { ++n; return ready_at_poll > 0 && n >= ready_at_poll; },
                                    [&] { return (uint64_t)(n * ns_per_poll); },
                                    [&] { return abort_at_poll > 0 && n >= abort_at_poll; }, [&] { failed = true; }, (uint64_t)cap_ns);
    if (polls) *polls = n;
    if (succeeded) *succeeded = ok ? 1 : 0;
    if (recorded_timeout) *recorded_timeout = failed ? 1 : 0;
    if (elapsed_ns) *elapsed_ns = n * ns_per_poll;
    return JA_OK;
}

// ---------------------------------------------------------------------------------------------------
// tilings
// ---------------------------------------------------------------------------------------------------
static bool splits_tile(int64_t extent, int32_t nparts, const int64_t* s) {
    if (nparts < 1 || !s || s[0] != 0 || s[nparts] != extent) return false;
    for (int32_t i = 0; i < nparts; ++i)
        if (s[i + 1] <= s[i]) return false;
    return true;
}

static int esize_of(ja_dtype_t dt) { return dt == JA_F32 ? 4 : 2; }

static ja_status_t fill_relation(ja_relation* r, int32_t rank, const int64_t* extents, const int32_t* nparts,
                                 const int64_t* const* splits, ja_dtype_t dtype) {
    if (rank < 1 || rank > JA_MAX_RANK || !extents || !nparts || !splits)
        return ja_fail(JA_ERR_INVALID_ARG, "rank must be 1..%d and extents/nparts/splits non-NULL", JA_MAX_RANK);
    if (dtype != JA_F32 && dtype != JA_BF16 && dtype != JA_F16) return ja_fail(JA_ERR_DTYPE, "unknown dtype %d", (int)dtype);
    r->rank = rank;
    r->dtype = dtype;
    r->esize = esize_of(dtype);
    r->nblocks = 1;
    r->equal_blocks = true;
    for (int d = 0; d < rank; ++d) {
        if (extents[d] < 1) return ja_fail(JA_ERR_SHAPE, "extent of dimension %d is %lld", d, (long long)extents[d]);
        if (!splits_tile(extents[d], nparts[d], splits[d]))
            return ja_fail(JA_ERR_TILING, "split points of dimension %d do not tile [0, %lld)", d, (long long)extents[d]);
        r->extent[d] = extents[d];
        r->nblk[d] = nparts[d];
        r->splits[d].assign(splits[d], splits[d] + nparts[d] + 1);
        int64_t b0 = splits[d][1] - splits[d][0];
        bool uni = true, eq = true;
        for (int i = 0; i < nparts[d]; ++i) {
            int64_t w = splits[d][i + 1] - splits[d][i];
            if (i + 1 < nparts[d] ? (w != b0) : (w > b0)) uni = false;
            if (w != b0) eq = false;
        }
        r->bs[d] = uni ? b0 : 0;
        r->equal_blocks = r->equal_blocks && eq;
        r->nblocks *= nparts[d];
    }
    // block offsets: row-major key order, back to back, 128-byte aligned
    r->blk_off.resize(r->nblocks);
    int32_t c[JA_MAX_RANK] = {0, 0, 0, 0};
    int64_t off = 0;
    for (int64_t b = 0; b < r->nblocks; ++b) {
        r->blk_off[b] = off;
        int64_t n = 1;
        for (int d = 0; d < rank; ++d) n *= r->splits[d][c[d] + 1] - r->splits[d][c[d]];
        int64_t nbytes = n * r->esize;
        off += (nbytes + JA_ALIGN - 1) / JA_ALIGN * JA_ALIGN;
        for (int d = rank - 1; d >= 0; --d) {
            if (++c[d] < r->nblk[d]) break;
            c[d] = 0;
        }
    }
    r->bytes = (size_t)off;
    return JA_OK;
}

extern "C" ja_status_t ja_relation_bytes(int32_t rank, const int64_t* extents, const int32_t* nparts,
                                         const int64_t* const* splits, ja_dtype_t dtype, size_t* bytes) {
    if (!bytes) return ja_fail(JA_ERR_INVALID_ARG, "bytes is NULL");
    ja_relation tmp;
    ja_status_t st = fill_relation(&tmp, rank, extents, nparts, splits, dtype);
    if (st != JA_OK) return st;
    *bytes = tmp.bytes;
    return JA_OK;
}

extern "C" ja_status_t ja_relation_create(int32_t rank, const int64_t* extents, const int32_t* nparts,
                                          const int64_t* const* splits, ja_dtype_t dtype, void* device_ptr,
                                          size_t bytes, ja_relation_t** out) {
    if (!out) return ja_fail(JA_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    std::unique_ptr<ja_relation> r(new ja_relation());
    ja_status_t st = fill_relation(r.get(), rank, extents, nparts, splits, dtype);
    if (st != JA_OK) return st;
    if (!device_ptr) return ja_fail(JA_ERR_INVALID_ARG, "device_ptr is NULL");
    if (((uintptr_t)device_ptr) % JA_ALIGN != 0)
        return ja_fail(JA_ERR_ALIGNMENT, "payload pointer %p is not %d-byte aligned", device_ptr, JA_ALIGN);
    if (bytes < r->bytes)
        return ja_fail(JA_ERR_INVALID_ARG, "payload buffer has %zu bytes, the tiling needs %zu", bytes, r->bytes);
    r->base = device_ptr;
    r->id = g_next_id++;
    *out = r.release();
    return JA_OK;
}

// live specs, so that ja_relation_destroy can drop the launch state cached for a relation that goes away
static std::mutex g_specs_mu;
static std::set<ja_spec*> g_specs;
static void forget_relayout_plans(uint64_t relation_id);
static void forget_exec_plans(uint64_t relation_id);

extern "C" ja_status_t ja_relation_destroy(ja_relation_t* rel) {
    if (!rel) return JA_OK;
    forget_relayout_plans(rel->id);   // cached copy plans of relayouts from / to this relation (device tables) go with it
    forget_exec_plans(rel->id);       // and the launch state (tensor maps, rotation tables) of every spec that ran on it
    if (rel->d_tables) cudaFree(rel->d_tables);
    delete rel;
    return JA_OK;
}

extern "C" ja_status_t ja_relation_num_blocks(const ja_relation_t* rel, int64_t* nblocks, int32_t* rank) {
    if (!rel) return ja_fail(JA_ERR_INVALID_ARG, "relation is NULL");
    if (nblocks) *nblocks = rel->nblocks;
    if (rank) *rank = rel->rank;
    return JA_OK;
}

extern "C" ja_status_t ja_relation_get_keys(const ja_relation_t* rel, int32_t* coords, int64_t* lower, int64_t* upper,
                                            int64_t* offsets) {
    if (!rel) return ja_fail(JA_ERR_INVALID_ARG, "relation is NULL");
    int32_t c[JA_MAX_RANK] = {0, 0, 0, 0};
    for (int64_t b = 0; b < rel->nblocks; ++b) {
        for (int d = 0; d < rel->rank; ++d) {
            if (coords) coords[b * rel->rank + d] = c[d];
            if (lower) lower[b * rel->rank + d] = rel->splits[d][c[d]];
            if (upper) upper[b * rel->rank + d] = rel->splits[d][c[d] + 1];
        }
        if (offsets) offsets[b] = rel->blk_off[b];
        for (int d = rel->rank - 1; d >= 0; --d) {
            if (++c[d] < rel->nblk[d]) break;
            c[d] = 0;
        }
    }
    return JA_OK;
}

// device copy of the key table: [splits of dim 0 | dim 1 | ... | block offsets]
ja_status_t ja_relation_to_device(const ja_relation* r) {
    static std::mutex mu;   // two threads may execute on one relation for the first time at once
    std::lock_guard<std::mutex> lk(mu);
    if (r->on_device) return JA_OK;
    std::vector<int64_t> host;
    for (int d = 0; d < r->rank; ++d) host.insert(host.end(), r->splits[d].begin(), r->splits[d].end());
    host.insert(host.end(), r->blk_off.begin(), r->blk_off.end());
    JA_CUDA(cudaMalloc((void**)&r->d_tables, host.size() * sizeof(int64_t)));
    JA_CUDA(cudaMemcpy(r->d_tables, host.data(), host.size() * sizeof(int64_t), cudaMemcpyHostToDevice));
    r->on_device = true;
    return JA_OK;
}

RelView ja_view(const ja_relation* r) {
    RelView v;
    memset(&v, 0, sizeof v);
    v.base = (char*)r->base;
    v.rank = r->rank;
    v.esize = r->esize;
    int64_t* p = r->d_tables;
    for (int d = 0; d < JA_MAX_RANK; ++d) {
        if (d < r->rank) {
            v.splits[d] = p;
            p += r->nblk[d] + 1;
            v.extent[d] = r->extent[d];
            v.bs[d] = r->bs[d];
            v.nblk[d] = r->nblk[d];
        } else {
            v.splits[d] = nullptr;
            v.extent[d] = 1;
            v.bs[d] = 1;
            v.nblk[d] = 1;
        }
    }
    v.blk_off = p;
    v.blk_stride = r->equal_blocks ? (r->nblocks > 1 ? r->blk_off[1] - r->blk_off[0] : (int64_t)r->bytes) : 0;
    return v;
}

// ---------------------------------------------------------------------------------------------------
// join-agg spec
// ---------------------------------------------------------------------------------------------------
static int letter_pos(const std::string& letters, char c) {
    size_t p = letters.find(c);
    return p == std::string::npos ? -1 : (int)p;
}

extern "C" ja_status_t ja_spec_create(const char* einsum, const ja_index_part_t* parts, int32_t n_parts, ja_fn_t fn,
                                      const double* fn_params, int32_t n_fn_params, ja_agg_t agg,
                                      ja_dtype_t accum_dtype, ja_spec_t** out) {
    if (!out) return ja_fail(JA_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (!einsum || !parts || n_parts < 1) return ja_fail(JA_ERR_INVALID_ARG, "einsum / parts missing");
    if (accum_dtype != JA_F32) return ja_fail(JA_ERR_DTYPE, "accumulation dtype must be JA_F32");
    if ((int)fn < 0 || (int)fn > (int)JA_FN_SWIGLU_UP) return ja_fail(JA_ERR_INVALID_ARG, "unknown fn %d", (int)fn);
    if ((int)agg < 0 || (int)agg > (int)JA_AGG_ONLINE_SOFTMAX) return ja_fail(JA_ERR_INVALID_ARG, "unknown agg %d", (int)agg);
    if (n_fn_params < 0 || (n_fn_params > 0 && !fn_params)) return ja_fail(JA_ERR_INVALID_ARG, "fn_params missing");

    std::unique_ptr<ja_spec> s(new ja_spec());
    // ---- parse ------------------------------------------------------------------------------------
    std::string e;
    for (const char* c = einsum; *c; ++c)
        if (*c != ' ') e.push_back(*c);
    size_t arrow = e.find("->");
    if (arrow == std::string::npos || e.find("->", arrow + 2) != std::string::npos)
        return ja_fail(JA_ERR_PARSE, "einsum '%s' needs exactly one '->'", einsum);
    std::string lhs = e.substr(0, arrow);
    s->out = e.substr(arrow + 2);
    size_t pos = 0;
    while (true) {
        size_t comma = lhs.find(',', pos);
        s->ins.push_back(lhs.substr(pos, comma == std::string::npos ? std::string::npos : comma - pos));
        if (comma == std::string::npos) break;
        pos = comma + 1;
    }
    if (s->ins.empty() || s->ins.size() > JA_MAX_IN) return ja_fail(JA_ERR_PARSE, "1..%d operands expected", JA_MAX_IN);
    std::vector<std::string> terms = s->ins;
    terms.push_back(s->out);
    for (size_t t = 0; t < terms.size(); ++t) {
        const std::string& term = terms[t];
        bool is_out = (t + 1 == terms.size());
        if ((term.empty() && !is_out) || term.size() > JA_MAX_RANK)
            return ja_fail(JA_ERR_PARSE, "operand '%s' must have rank 1..%d", term.c_str(), JA_MAX_RANK);
        for (size_t i = 0; i < term.size(); ++i) {
            char c = term[i];
            if (c < 'a' || c > 'z') return ja_fail(JA_ERR_PARSE, "bad character '%c' in einsum", c);
            if (term.find(c, i + 1) != std::string::npos)
                return ja_fail(JA_ERR_PARSE, "letter '%c' repeated inside one operand", c);
            if (is_out) {
                if (letter_pos(s->letters, c) < 0)
                    return ja_fail(JA_ERR_PARSE, "output letter '%c' appears in no input", c);
            } else if (letter_pos(s->letters, c) < 0) {
                s->letters.push_back(c);
            }
        }
    }
    if (s->out.empty()) return ja_fail(JA_ERR_UNSUPPORTED, "scalar outputs are not supported");
    s->einsum = e;
    // ---- partitions ---------------------------------------------------------------------------------
    s->parts.resize(s->letters.size());
    for (int32_t i = 0; i < n_parts; ++i) {
        int lp = letter_pos(s->letters, parts[i].name);
        if (lp < 0) return ja_fail(JA_ERR_SHAPE, "partition given for letter '%c' which the einsum does not use", parts[i].name);
        if (!s->parts[lp].empty()) return ja_fail(JA_ERR_SHAPE, "two partitions for letter '%c'", parts[i].name);
        if (parts[i].extent < 1 || !splits_tile(parts[i].extent, parts[i].nparts, parts[i].splits))
            return ja_fail(JA_ERR_TILING, "split points of index '%c' do not tile [0, %lld)", parts[i].name,
                           (long long)parts[i].extent);
        s->parts[lp].assign(parts[i].splits, parts[i].splits + parts[i].nparts + 1);
    }
    for (size_t l = 0; l < s->letters.size(); ++l)
        if (s->parts[l].empty()) return ja_fail(JA_ERR_SHAPE, "no partition for index '%c'", s->letters[l]);
    bool has_agg_index = false;
    for (char c : s->letters)
        if (s->out.find(c) == std::string::npos) has_agg_index = true;
    if (agg == JA_AGG_NONE && has_agg_index && fn != JA_FN_RMSNORM && fn != JA_FN_SOFTMAX)
        return ja_fail(JA_ERR_TILING,
                       "an index is absent from the output, so several function specs share an output type, "
                       "but no aggregation was given");
    s->fn = fn;
    s->agg = agg;
    s->params.assign(fn_params, fn_params + n_fn_params);

    // ---- enumerate J: one function spec per cell of the interval grid (Section 3.3) ------------------
    const int L = (int)s->letters.size();
    std::vector<int32_t> nb(L);
    int64_t p = 1;
    for (int l = 0; l < L; ++l) {
        nb[l] = (int32_t)s->parts[l].size() - 1;
        p *= nb[l];
        if (p > (int64_t)1 << 26) return ja_fail(JA_ERR_UNSUPPORTED, "more than 2^26 function specs");
    }
    // Attention (Example 3.10). Three selections remove cells of the interval grid:
    //   band      causal attention: a (q-block, k-block) pair is a tuple only if some k <= some q;
    //   induced   grouped-query attention "bqhd,bkgd,bkgd->bqhd": h is not shardable by itself, its intervals are
    //             those of g scaled by group = extent(h)/extent(g), and interval m of g pairs with interval m of h;
    //   segments  packed sequences ending at params[2..]: q and k may be cut so that every sequence end is a split
    //             point, and a pair of blocks is a tuple only if both lie in the same sequence.
    int band_q = -1, band_k = -1, ind_h = -1, ind_g = -1, seg_q = -1, seg_k = -1;
    std::vector<int64_t> ends;
    if (fn == JA_FN_ATTENTION && s->ins.size() == 3 && s->ins[0].size() == 4 && s->ins[1].size() == 4) {
        const int lq = letter_pos(s->letters, s->ins[0][1]), lk = letter_pos(s->letters, s->ins[1][1]);
        if (s->params.size() >= 2 && s->params[1] != 0.0) { band_q = lq; band_k = lk; }
        if (s->ins[1][2] != s->ins[0][2]) {
            ind_h = letter_pos(s->letters, s->ins[0][2]);
            ind_g = letter_pos(s->letters, s->ins[1][2]);
            const int64_t eh = s->parts[ind_h].back(), eg = s->parts[ind_g].back();
            if (eh % eg) return ja_fail(JA_ERR_SHAPE, "query heads (%lld) must be a multiple of key/value heads (%lld)", (long long)eh, (long long)eg);
            const int64_t group = eh / eg;
            bool same = s->parts[ind_h].size() == s->parts[ind_g].size();
            for (size_t i = 0; same && i < s->parts[ind_g].size(); ++i) same = s->parts[ind_h][i] == group * s->parts[ind_g][i];
            if (!same)
                return ja_fail(JA_ERR_TILING, "index '%c' is not shardable by itself: its intervals must be those of '%c' scaled by %lld",
                               s->ins[0][2], s->ins[1][2], (long long)group);
        }
        for (size_t i = 2; i < s->params.size(); ++i) ends.push_back((int64_t)s->params[i]);
        if (!ends.empty()) {
            if (s->parts[lq].back() != s->parts[lk].back()) return ja_fail(JA_ERR_SHAPE, "packed sequences need equal query and key extents");
            if (ends.size() > JA_MAX_SEQ) return ja_fail(JA_ERR_UNSUPPORTED, "more than %d packed sequences", JA_MAX_SEQ);
            for (size_t i = 0; i < ends.size(); ++i) {
                if ((double)ends[i] != s->params[2 + i] || ends[i] <= (i ? ends[i - 1] : 0))
                    return ja_fail(JA_ERR_INVALID_ARG, "sequence ends must be ascending positive integers");
                for (int l : {lq, lk})
                    if (!std::binary_search(s->parts[l].begin(), s->parts[l].end(), ends[i]))
                        return ja_fail(JA_ERR_TILING, "index '%c' may only be cut so that every sequence end (%lld) is a split point",
                                       s->letters[l], (long long)ends[i]);
            }
            if (ends.back() != s->parts[lq].back()) return ja_fail(JA_ERR_INVALID_ARG, "the last sequence must end at the extent of the sequence index");
            seg_q = lq;
            seg_k = lk;
        }
    }
    auto seq_of = [&](int64_t x) { return (int)(std::upper_bound(ends.begin(), ends.end(), x) - ends.begin()); };
    const int n_in = (int)s->ins.size();
    std::vector<int32_t> cell(L, 0);
    for (int64_t t = 0; t < p; ++t) {
        bool keep = true;
        if (band_q >= 0) keep = s->parts[band_k][cell[band_k]] <= s->parts[band_q][cell[band_q] + 1] - 1;
        if (keep && ind_h >= 0) keep = cell[ind_h] == cell[ind_g];
        if (keep && seg_q >= 0) keep = seq_of(s->parts[seg_k][cell[seg_k]]) == seq_of(s->parts[seg_q][cell[seg_q]]);
        if (keep) {
            for (int k = 0; k <= n_in; ++k) {
                const std::string& term = (k < n_in) ? s->ins[k] : s->out;
                int32_t key = 0;
                for (char c : term) {
                    int lp = letter_pos(s->letters, c);
                    key = key * nb[lp] + cell[lp];
                }
                if (k < n_in) s->in_keys.push_back(key);
                else s->out_keys.push_back(key);
            }
        }
        for (int l = L - 1; l >= 0; --l) {
            if (++cell[l] < nb[l]) break;
            cell[l] = 0;
        }
    }
    s->p = (int64_t)s->out_keys.size();
    *out = s.release();
    {
        std::lock_guard<std::mutex> lk(g_specs_mu);
        g_specs.insert(*out);
    }
    return JA_OK;
}


static void forget_exec_plans(uint64_t relation_id) {
    std::lock_guard<std::mutex> lk(g_specs_mu);
    for (ja_spec* s : g_specs) {
        std::lock_guard<std::mutex> lk2(s->plans_mu);
        for (auto it = s->plans.begin(); it != s->plans.end();)
            it = std::find(it->first.begin(), it->first.end(), relation_id) != it->first.end() ? s->plans.erase(it) : std::next(it);
    }
}

extern "C" ja_status_t ja_spec_destroy(ja_spec_t* spec) {
    if (spec) {
        std::lock_guard<std::mutex> lk(g_specs_mu);
        g_specs.erase(spec);
    }
    delete spec;
    return JA_OK;
}

extern "C" ja_status_t ja_spec_num_tuples(const ja_spec_t* spec, int64_t* p, int32_t* n_inputs) {
    if (!spec) return ja_fail(JA_ERR_INVALID_ARG, "spec is NULL");
    if (p) *p = spec->p;
    if (n_inputs) *n_inputs = (int32_t)spec->ins.size();
    return JA_OK;
}

extern "C" ja_status_t ja_spec_get_tuples(const ja_spec_t* spec, int32_t* in_keys, int32_t* out_keys) {
    if (!spec) return ja_fail(JA_ERR_INVALID_ARG, "spec is NULL");
    if (in_keys) memcpy(in_keys, spec->in_keys.data(), spec->in_keys.size() * sizeof(int32_t));
    if (out_keys) memcpy(out_keys, spec->out_keys.data(), spec->out_keys.size() * sizeof(int32_t));
    return JA_OK;
}

static const std::string& spec_term(const ja_spec* s, int operand) {
    return operand < 0 ? s->out : s->ins[operand];
}

extern "C" ja_status_t ja_spec_operand_tiling(const ja_spec_t* spec, int32_t operand, int32_t* rank, int32_t* nblocks,
                                              int64_t* splits_flat) {
    if (!spec) return ja_fail(JA_ERR_INVALID_ARG, "spec is NULL");
    if (operand < -1 || operand >= (int32_t)spec->ins.size()) return ja_fail(JA_ERR_INVALID_ARG, "operand %d out of range", operand);
    const std::string& term = spec_term(spec, operand);
    if (rank) *rank = (int32_t)term.size();
    size_t w = 0;
    for (size_t d = 0; d < term.size(); ++d) {
        const std::vector<int64_t>& sp = spec->parts[letter_pos(spec->letters, term[d])];
        if (nblocks) nblocks[d] = (int32_t)sp.size() - 1;
        if (splits_flat) {
            memcpy(splits_flat + w, sp.data(), sp.size() * sizeof(int64_t));
            w += sp.size();
        }
    }
    return JA_OK;
}

extern "C" ja_status_t ja_spec_cost_terms(const ja_spec_t* spec, int64_t* join_elems, int64_t* agg_elems) {
    if (!spec) return ja_fail(JA_ERR_INVALID_ARG, "spec is NULL");
    const int n_in = (int)spec->ins.size();
    auto card = [&](int operand, int32_t key) {
        const std::string& term = spec_term(spec, operand);
        int64_t n = 1;
        for (int d = (int)term.size() - 1; d >= 0; --d) {
            const std::vector<int64_t>& sp = spec->parts[letter_pos(spec->letters, term[d])];
            int32_t nbd = (int32_t)sp.size() - 1;
            int32_t c = key % nbd;
            key /= nbd;
            n *= sp[c + 1] - sp[c];
        }
        return n;
    };
    int64_t join = 0;
    std::map<int32_t, int64_t> mult;
    for (int64_t t = 0; t < spec->p; ++t) {
        for (int k = 0; k < n_in; ++k) join += card(k, spec->in_keys[t * n_in + k]);
        mult[spec->out_keys[t]] += 1;
    }
    int64_t ag = 0;
    for (auto& kv : mult) ag += (kv.second - 1) * card(-1, kv.first);
    if (join_elems) *join_elems = join;
    if (agg_elems) *agg_elems = ag;
    return JA_OK;
}

// ---------------------------------------------------------------------------------------------------
// repartition: overlay -> atoms -> slab copies (Section 5.3)
// ---------------------------------------------------------------------------------------------------
struct Atom {
    int64_t lo[JA_MAX_RANK], hi[JA_MAX_RANK];
    int32_t sb, db;
};

static ja_status_t check_same_tensor(const ja_relation* a, const ja_relation* b) {
    if (!a || !b) return ja_fail(JA_ERR_INVALID_ARG, "relation is NULL");
    if (a->rank != b->rank) return ja_fail(JA_ERR_SHAPE, "ranks differ (%d vs %d)", a->rank, b->rank);
    if (a->dtype != b->dtype) return ja_fail(JA_ERR_DTYPE, "dtypes differ");
    for (int d = 0; d < a->rank; ++d)
        if (a->extent[d] != b->extent[d]) return ja_fail(JA_ERR_SHAPE, "extent of dimension %d differs", d);
    return JA_OK;
}

static void build_atoms(const ja_relation* src, const ja_relation* dst, std::vector<Atom>* atoms) {
    const int r = src->rank;
    std::vector<int64_t> over[JA_MAX_RANK];
    for (int d = 0; d < r; ++d) {
        over[d] = src->splits[d];
        over[d].insert(over[d].end(), dst->splits[d].begin(), dst->splits[d].end());
        std::sort(over[d].begin(), over[d].end());
        over[d].erase(std::unique(over[d].begin(), over[d].end()), over[d].end());
    }
    auto owner = [](const std::vector<int64_t>& sp, int64_t x) {
        return (int32_t)(std::upper_bound(sp.begin(), sp.end(), x) - sp.begin() - 1);
    };
    int32_t c[JA_MAX_RANK] = {0, 0, 0, 0};
    int64_t n = 1;
    for (int d = 0; d < r; ++d) n *= (int64_t)over[d].size() - 1;
    atoms->reserve(n);
    for (int64_t a = 0; a < n; ++a) {
        Atom at;
        at.sb = at.db = 0;
        for (int d = 0; d < r; ++d) {
            at.lo[d] = over[d][c[d]];
            at.hi[d] = over[d][c[d] + 1];
            at.sb = at.sb * src->nblk[d] + owner(src->splits[d], at.lo[d]);
            at.db = at.db * dst->nblk[d] + owner(dst->splits[d], at.lo[d]);
        }
        atoms->push_back(at);
        for (int d = r - 1; d >= 0; --d) {
            if (++c[d] < (int32_t)over[d].size() - 1) break;
            c[d] = 0;
        }
    }
}

extern "C" ja_status_t ja_overlay_atoms(const ja_relation_t* src, const ja_relation_t* dst, int64_t* n_atoms,
                                        int64_t* lower, int64_t* upper, int32_t* src_block, int32_t* dst_block) {
    ja_status_t st = check_same_tensor(src, dst);
    if (st != JA_OK) return st;
    std::vector<Atom> atoms;
    build_atoms(src, dst, &atoms);
    if (n_atoms) *n_atoms = (int64_t)atoms.size();
    for (size_t a = 0; a < atoms.size(); ++a) {
        for (int d = 0; d < src->rank; ++d) {
            if (lower) lower[a * src->rank + d] = atoms[a].lo[d];
            if (upper) upper[a * src->rank + d] = atoms[a].hi[d];
        }
        if (src_block) src_block[a] = atoms[a].sb;
        if (dst_block) dst_block[a] = atoms[a].db;
    }
    return JA_OK;
}

struct RepartPlan {
    CopySlab* d_slabs = nullptr;
    int64_t n_slabs = 0;
    int vec_bytes = 16;
    ~RepartPlan() {
        if (d_slabs) cudaFree(d_slabs);
    }
};
static std::mutex g_repart_mu;
static std::map<std::pair<uint64_t, uint64_t>, std::shared_ptr<RepartPlan>> g_repart_plans;

// element offset of coordinate x inside block `b` of relation r (row-major inside the block)
static int64_t in_block_offset(const ja_relation* r, int32_t b, const int64_t* x, int64_t* last_width) {
    int32_t c[JA_MAX_RANK];
    for (int d = r->rank - 1; d >= 0; --d) {
        c[d] = b % r->nblk[d];
        b /= r->nblk[d];
    }
    int64_t off = 0;
    for (int d = 0; d < r->rank; ++d) {
        int64_t lo = r->splits[d][c[d]], w = r->splits[d][c[d] + 1] - lo;
        off = off * w + (x[d] - lo);
        if (d == r->rank - 1 && last_width) *last_width = w;
    }
    return off;
}

// Cuts every atom of the overlay of src and dst into 2-D slabs: (rows of the second-to-last dimension) x (contiguous run
// of the last dimension), one per assignment of the outer dimensions, at most 64 KiB of source bytes each. Offsets and
// pitches are in bytes of the respective relation (their element sizes may differ); row_bytes counts source bytes.
// src_or / dst_or: OR of every quantity that limits the access width on that side.
static void plan_slabs(const ja_relation* src, const ja_relation* dst, std::vector<CopySlab>* slabs, int64_t* src_or, int64_t* dst_or) {
    std::vector<Atom> atoms;
    build_atoms(src, dst, &atoms);
    const int r = src->rank, es = src->esize, ed = dst->esize;
    const int64_t slab_bytes = 64 * 1024;
    for (const Atom& at : atoms) {
        int64_t rows = r >= 2 ? at.hi[r - 2] - at.lo[r - 2] : 1;
        int64_t row_bytes = (at.hi[r - 1] - at.lo[r - 1]) * es;
        int64_t outer = 1;
        for (int d = 0; d + 2 < r; ++d) outer *= at.hi[d] - at.lo[d];
        int64_t rows_per = std::max<int64_t>(1, slab_bytes / row_bytes);
        for (int64_t o = 0; o < outer; ++o) {
            int64_t x[JA_MAX_RANK];
            int64_t rem = o;
            for (int d = r - 3; d >= 0; --d) {
                int64_t e = at.hi[d] - at.lo[d];
                x[d] = at.lo[d] + rem % e;
                rem /= e;
            }
            for (int64_t r0 = 0; r0 < rows; r0 += rows_per) {
                if (r >= 2) x[r - 2] = at.lo[r - 2] + r0;
                x[r - 1] = at.lo[r - 1];
                int64_t sw = 0, dw = 0;
                CopySlab s;
                s.src_off = src->blk_off[at.sb] + in_block_offset(src, at.sb, x, &sw) * es;
                s.dst_off = dst->blk_off[at.db] + in_block_offset(dst, at.db, x, &dw) * ed;
                s.rows = (int32_t)std::min(rows_per, rows - r0);
                s.row_bytes = (int32_t)row_bytes;
                s.src_pitch = (int32_t)(sw * es);
                s.dst_pitch = (int32_t)(dw * ed);
                *src_or |= s.src_off | s.row_bytes | s.src_pitch;
                *dst_or |= s.dst_off | s.dst_pitch;
                slabs->push_back(s);
            }
        }
    }
}

extern "C" ja_status_t ja_repartition(const ja_relation_t* src, ja_relation_t* dst, void* cuda_stream) {
    ja_status_t st = check_same_tensor(src, dst);
    if (st != JA_OK) return st;
    if (src->base == dst->base) return ja_fail(JA_ERR_INVALID_ARG, "repartition in place is not supported");
    std::shared_ptr<RepartPlan> plan;
    {
        std::lock_guard<std::mutex> lk(g_repart_mu);
        auto it = g_repart_plans.find({src->id, dst->id});
        if (it != g_repart_plans.end()) plan = it->second;
    }
    if (!plan) {
        const int es = src->esize;
        std::vector<CopySlab> slabs;
        int64_t src_or = 0, dst_or = 0;
        plan_slabs(src, dst, &slabs, &src_or, &dst_or);
        const int64_t all_or = src_or | dst_or;
        plan.reset(new RepartPlan());
        plan->vec_bytes = 16;
        while (plan->vec_bytes > es && (all_or % plan->vec_bytes) != 0) plan->vec_bytes /= 2;
        plan->n_slabs = (int64_t)slabs.size();
        JA_CUDA(cudaMalloc((void**)&plan->d_slabs, slabs.size() * sizeof(CopySlab)));
        JA_CUDA(cudaMemcpy(plan->d_slabs, slabs.data(), slabs.size() * sizeof(CopySlab), cudaMemcpyHostToDevice));
        std::lock_guard<std::mutex> lk(g_repart_mu);
        g_repart_plans[{src->id, dst->id}] = plan;
    }
    return ja_launch_repartition((const char*)src->base, (char*)dst->base, plan->d_slabs, plan->n_slabs,
                                 plan->vec_bytes, (cudaStream_t)cuda_stream);
}

// ---------------------------------------------------------------------------------------------------
// aggregating relayout (Sections 5.1, 5.3): m unaggregated copies of every producer block -> aggregated consumer blocks
// ---------------------------------------------------------------------------------------------------
static std::map<std::vector<uint64_t>, std::shared_ptr<RepartPlan>> g_repart_agg_plans;

static void forget_relayout_plans(uint64_t relation_id) {
    std::lock_guard<std::mutex> lk(g_repart_mu);
    for (auto it = g_repart_plans.begin(); it != g_repart_plans.end();)
        it = (it->first.first == relation_id || it->first.second == relation_id) ? g_repart_plans.erase(it) : std::next(it);
    for (auto it = g_repart_agg_plans.begin(); it != g_repart_agg_plans.end();)
        it = (it->first[0] == relation_id || it->first[1] == relation_id) ? g_repart_agg_plans.erase(it) : std::next(it);
}

// partials must be [c, x...] with the copy index c cut into its unit intervals and x... the tensor of `like`
static ja_status_t check_partial_relation(const ja_relation* partials, const ja_relation* like, int like_rank, const int64_t* like_extent) {
    if (!partials) return ja_fail(JA_ERR_INVALID_ARG, "partial relation is NULL");
    if (partials->rank != like_rank + 1)
        return ja_fail(JA_ERR_SHAPE, "a partial relation has the copy index in front: rank %d expected, got %d", like_rank + 1, partials->rank);
    if (partials->nblk[0] != partials->extent[0])
        return ja_fail(JA_ERR_TILING, "the copy index of a partial relation must be cut into unit intervals");
    for (int d = 0; d < like_rank; ++d)
        if (partials->extent[d + 1] != like_extent[d]) return ja_fail(JA_ERR_SHAPE, "extent of dimension %d differs", d);
    (void)like;
    return JA_OK;
}

extern "C" ja_status_t ja_repartition_agg(const ja_relation_t* partials, ja_agg_t agg, ja_relation_t* dst, void* cuda_stream) {
    if (!dst) return ja_fail(JA_ERR_INVALID_ARG, "relation is NULL");
    ja_status_t st = check_partial_relation(partials, dst, dst->rank, dst->extent);
    if (st != JA_OK) return st;
    const int m = (int)partials->extent[0];
    if (agg != JA_AGG_SUM && agg != JA_AGG_MAX && !(agg == JA_AGG_NONE && m == 1))
        return ja_fail(JA_ERR_INVALID_ARG, "%d copies of every atom need SUM or MAX aggregation", m);
    if (partials->base == dst->base) return ja_fail(JA_ERR_INVALID_ARG, "repartition in place is not supported");
    std::shared_ptr<RepartPlan> plan;
    const std::vector<uint64_t> key = {partials->id, dst->id};
    {
        std::lock_guard<std::mutex> lk(g_repart_mu);
        auto it = g_repart_agg_plans.find(key);
        if (it != g_repart_agg_plans.end()) plan = it->second;
    }
    const int64_t ntrail = partials->nblocks / m;
    const int64_t copy_stride = m > 1 ? partials->blk_off[ntrail] - partials->blk_off[0] : 0;
    if (!plan) {
        // copy 0 of the partial relation seen as a relation over the consumer's tensor
        ja_relation view;
        view.rank = dst->rank;
        view.esize = partials->esize;
        view.dtype = partials->dtype;
        for (int d = 0; d < dst->rank; ++d) {
            view.extent[d] = partials->extent[d + 1];
            view.nblk[d] = partials->nblk[d + 1];
            view.splits[d] = partials->splits[d + 1];
        }
        view.blk_off.assign(partials->blk_off.begin(), partials->blk_off.begin() + ntrail);
        for (int c = 1; c < m; ++c)   // every copy has the block structure of copy 0, copy_stride bytes further on
            for (int64_t b = 0; b < ntrail; ++b)
                if (partials->blk_off[c * ntrail + b] != view.blk_off[b] + c * copy_stride)
                    return ja_fail(JA_ERR_UNSUPPORTED, "copies of the partial relation are not equally spaced");
        std::vector<CopySlab> slabs;
        int64_t src_or = copy_stride, dst_or = 0;
        plan_slabs(&view, dst, &slabs, &src_or, &dst_or);
        const int vec = partials->esize == 4 ? 4 : 8;                       // cells per 16-byte source access
        const int dst_access = std::min(16, vec * dst->esize);
        plan.reset(new RepartPlan());
        plan->vec_bytes = (src_or % 16 == 0 && dst_or % dst_access == 0) ? vec : 1;   // here: cells per access
        plan->n_slabs = (int64_t)slabs.size();
        JA_CUDA(cudaMalloc((void**)&plan->d_slabs, std::max<size_t>(1, slabs.size()) * sizeof(CopySlab)));
        JA_CUDA(cudaMemcpy(plan->d_slabs, slabs.data(), slabs.size() * sizeof(CopySlab), cudaMemcpyHostToDevice));
        std::lock_guard<std::mutex> lk(g_repart_mu);
        g_repart_agg_plans[key] = plan;
    }
    return ja_launch_repartition_agg((const char*)partials->base, (char*)dst->base, plan->d_slabs, plan->n_slabs, m, copy_stride,
                                     partials->dtype, dst->dtype, agg, plan->vec_bytes, (cudaStream_t)cuda_stream);
}

// ---------------------------------------------------------------------------------------------------
// ja_execute
// ---------------------------------------------------------------------------------------------------
struct ExecPlan {
    std::shared_ptr<GemmTcPlan> gemm;
    bool gemm_checked = false;
    AttnTcCache attn;
    float2* rope_table = nullptr;
    int64_t* rope_splits = nullptr;  // split points of the collapsed (h d) index
    ~ExecPlan() {
        if (rope_table) cudaFree(rope_table);
        if (rope_splits) cudaFree(rope_splits);
    }
};

// True when a "bshd" relation has uniform blocks along b and h, an unsplit d, and every block starts where the closed
// form used by the tensor-memory attention kernel puts it: blocks in key order, each a dense run of rows of
// hblk * extent(d) cells, so block (bb, sb, hb) starts (bb*bblk*S + bblk*start(sb)) * nhb + hb*bblk*rows(sb) rows in.
static bool bshd_rows_layout(const ja_relation* r) {
    if (r->rank != 4 || !r->bs[0] || !r->bs[2] || r->nblk[3] != 1) return false;
    const int64_t S = r->extent[1], bblk = r->bs[0], hblk = r->bs[2], nhb = r->nblk[2];
    const int64_t row_bytes = hblk * r->extent[3] * r->esize;
    if (r->extent[0] * S * nhb >= ((int64_t)1 << 31)) return false;
    for (int32_t bb = 0; bb < r->nblk[0]; ++bb)
        for (int32_t sb = 0; sb < r->nblk[1]; ++sb)
            for (int32_t hb = 0; hb < r->nblk[2]; ++hb) {
                const int64_t start = r->splits[1][sb], rows = r->splits[1][sb + 1] - start;
                const int64_t want = ((bb * bblk * S + bblk * start) * nhb + hb * bblk * rows) * row_bytes;
                if (r->blk_off[((int64_t)bb * r->nblk[1] + sb) * r->nblk[2] + hb] != want) return false;
            }
    return true;
}

static ja_status_t check_tiling(const ja_spec* s, int operand, const ja_relation* r) {
    const std::string& term = spec_term(s, operand);
    if (!r) return ja_fail(JA_ERR_INVALID_ARG, "relation for operand %d is NULL", operand);
    if (r->rank != (int)term.size())
        return ja_fail(JA_ERR_SHAPE, "operand %d has rank %d, the einsum term '%s' needs %zu", operand, r->rank,
                       term.c_str(), term.size());
    for (int d = 0; d < r->rank; ++d) {
        const std::vector<int64_t>& sp = s->parts[letter_pos(s->letters, term[d])];
        if (r->extent[d] != sp.back())
            return ja_fail(JA_ERR_SHAPE, "operand %d dimension %d has extent %lld, index '%c' has %lld", operand, d,
                           (long long)r->extent[d], term[d], (long long)sp.back());
        if (r->splits[d] != sp)
            return ja_fail(JA_ERR_PARTITION_MISMATCH,
                           "operand %d is not tiled as the join-agg spec requires along index '%c': repartition it first",
                           operand, term[d]);
    }
    return JA_OK;
}

// "Rj" style helpers: lead = all letters but the last
static std::string lead_of(const std::string& t) { return t.substr(0, t.size() - 1); }

extern "C" ja_status_t ja_execute(const ja_spec_t* spec, const ja_relation_t* const* inputs, int32_t n_inputs,
                                  ja_relation_t* const* outputs, int32_t n_outputs, void* cuda_stream) {
    if (!spec || !inputs || !outputs) return ja_fail(JA_ERR_INVALID_ARG, "spec / inputs / outputs is NULL");
    const int n_in = (int)spec->ins.size();
    if (n_inputs != n_in) return ja_fail(JA_ERR_INVALID_ARG, "spec has %d operands, %d relations given", n_in, n_inputs);
    if (n_outputs != 1 && !(n_outputs == 2 && spec->fn == JA_FN_ATTENTION))
        return ja_fail(JA_ERR_UNSUPPORTED, "one output relation, or two for ATTENTION (O and the log of the softmax denominator)");
    ja_status_t st;
    for (int k = 0; k < n_in; ++k)
        if ((st = check_tiling(spec, k, inputs[k])) != JA_OK) return st;
    ja_relation* out = outputs[0];
    if ((st = check_tiling(spec, -1, out)) != JA_OK) return st;
    for (int k = 0; k < n_in; ++k)
        if (inputs[k]->base == out->base) return ja_fail(JA_ERR_INVALID_ARG, "output aliases input %d", k);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const ja_fn_t fn = spec->fn;
    const ja_agg_t agg = spec->agg;
    const std::vector<std::string>& in = spec->ins;
    const std::string& o = spec->out;

    // plan cache
    std::vector<uint64_t> key;
    for (int k = 0; k < n_in; ++k) key.push_back(inputs[k]->id);
    key.push_back(out->id);
    std::lock_guard<std::mutex> plans_lock(spec->plans_mu);   // held to the end: plan building and the launch that uses the plan
    std::shared_ptr<ExecPlan> plan = spec->plans[key];
    if (!plan) spec->plans[key] = plan = std::make_shared<ExecPlan>();

    for (int k = 0; k < n_in; ++k)
        if ((st = ja_relation_to_device(inputs[k])) != JA_OK) return st;
    if ((st = ja_relation_to_device(out)) != JA_OK) return st;

    // ---- matmul: "ij,jk->ik" MUL / SUM --------------------------------------------------------------
    if (fn == JA_FN_MUL && agg == JA_AGG_SUM && n_in == 2 && in[0].size() == 2 && in[1].size() == 2 && o.size() == 2 &&
        in[0][1] == in[1][0] && o[0] == in[0][0] && o[1] == in[1][1] && in[0][0] != in[1][1]) {
        const ja_relation *A = inputs[0], *B = inputs[1];
        if (A->dtype != B->dtype || A->dtype != out->dtype) return ja_fail(JA_ERR_DTYPE, "matmul operands must share one dtype");
        if (A->dtype != JA_F32) {   // bf16 or f16: tensor cores
            const int loader = ja_config().gemm_loader;
            if (!plan->gemm_checked) {
                bool ok = false;
                if ((st = ja_gemm_tc_plan(A, B, out, nullptr, &plan->gemm, &ok)) != JA_OK) return st;
                if (!ok) plan->gemm.reset();
                plan->gemm_checked = true;
            }
            if (plan->gemm && loader != 1) return ja_launch_gemm_tc(*plan->gemm, stream);
            if (loader != 0) {   // tilings TMA cannot address: the tensor cores fed by plain loads
                bool launched = false;
                if ((st = ja_launch_gemm_ld(A, B, out, stream, &launched)) != JA_OK || launched) return st;
            }
        }
        return ja_launch_matmul_simt(A, B, out, stream);
    }

    // ---- fused chains on the tensor-core matmul -------------------------------------------------------------------
    if ((fn == JA_FN_MATMUL_ADD || fn == JA_FN_MATMUL_ROPE || fn == JA_FN_SWIGLU_UP) && agg == JA_AGG_SUM && n_in >= 2 &&
        in[0].size() == 2 && in[1].size() == 2 && o.size() == 2 && in[0][1] == in[1][0] && o[0] == in[0][0] && o[1] == in[1][1] &&
        in[0][0] != in[1][1]) {
        const ja_relation *A = inputs[0], *B = inputs[1];
        for (int k = 0; k < n_in; ++k)
            if (inputs[k]->dtype == JA_F32 || inputs[k]->dtype != out->dtype)
                return ja_fail(JA_ERR_UNSUPPORTED, "fused matmul chains need relations of one 16-bit dtype");
        GemmEpilogue ep;
        memset(&ep, 0, sizeof ep);
        if (fn == JA_FN_MATMUL_ADD) {
            if (n_in != 3 || in[2] != o) return ja_fail(JA_ERR_SHAPE, "MATMUL_ADD needs \"ij,jk,ik->ik\"");
            ep.epi = 1;
            ep.addend = inputs[2];
        } else if (fn == JA_FN_SWIGLU_UP) {
            if (n_in != 3 || in[2] != in[1]) return ja_fail(JA_ERR_SHAPE, "SWIGLU_UP needs \"ij,jk,jk->ik\"");
            ep.epi = 3;
            ep.B2 = inputs[2];
        } else {
            if (n_in != 2 || spec->params.size() < 3) return ja_fail(JA_ERR_INVALID_ARG, "MATMUL_ROPE needs \"ij,jk->ik\" and [theta, seq_len, head_dim]");
            const double theta = spec->params[0];
            const int64_t S = (int64_t)spec->params[1], D = (int64_t)spec->params[2];
            if (S < 1 || D < 2 || D % 2 || A->extent[0] % S || B->extent[1] % D) return ja_fail(JA_ERR_SHAPE, "MATMUL_ROPE: rows must be whole sequences and columns whole heads");
            if (!plan->rope_table) {
                std::vector<float2> tab((size_t)S * (D / 2));
                for (int64_t s = 0; s < S; ++s)
                    for (int64_t pp = 0; pp < D / 2; ++pp) {
                        double phi = (double)s * std::pow(theta, -2.0 * (double)pp / (double)D);
                        tab[s * (D / 2) + pp] = make_float2((float)std::cos(phi), (float)std::sin(phi));
                    }
                JA_CUDA(cudaMalloc((void**)&plan->rope_table, tab.size() * sizeof(float2)));
                JA_CUDA(cudaMemcpy(plan->rope_table, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice));
            }
            ep.epi = 2;
            ep.rope_table = plan->rope_table;
            ep.rope_S = (int)S;
            ep.rope_D = (int)D;
        }
        if (!plan->gemm_checked) {
            bool ok = false;
            if ((st = ja_gemm_tc_plan(A, B, out, &ep, &plan->gemm, &ok)) != JA_OK) return st;
            if (!ok) plan->gemm.reset();
            plan->gemm_checked = true;
        }
        if (!plan->gemm) return ja_fail(JA_ERR_UNSUPPORTED, "this tiling cannot run the fused matmul chain: execute the join-aggs one by one");
        return ja_launch_gemm_tc(*plan->gemm, stream);
    }

    // ---- key-aligned maps "X,X->X" ----------------------------------------------------------------------
    if ((fn == JA_FN_ADD || fn == JA_FN_SILU_MUL) && agg == JA_AGG_NONE && n_in == 2 && in[0] == in[1] && in[0] == o) {
        if (inputs[0]->dtype != inputs[1]->dtype || inputs[0]->dtype != out->dtype)
            return ja_fail(JA_ERR_DTYPE, "key-aligned join needs one dtype");
        // identical tilings => identical payload layouts: the join pairs blocks with equal keys, and inside a
        // block cells with equal offsets
        return ja_launch_flat(fn, inputs[0]->base, inputs[1]->base, out->base, (int64_t)(out->bytes / out->esize),
                              out->dtype, stream);
    }

    // ---- row-structured forms -------------------------------------------------------------------------------
    RowArgs ra;
    memset(&ra, 0, sizeof ra);
    const std::string& x = in[0];
    const std::string R = lead_of(x);
    const bool x_ok = x.size() >= 2;
    auto stat_ok = [&](const ja_relation* r) { return r->dtype == JA_F32; };
    if (x_ok && fn == JA_FN_SQUARE && agg == JA_AGG_SUM && n_in == 1 && o == R) {
        if (!stat_ok(out)) return ja_fail(JA_ERR_DTYPE, "statistics relations are f32");
        ra.x = ja_view(inputs[0]); ra.s0 = ja_view(out);
        return ja_launch_row(ROW_SUMSQ, ra, inputs[0]->dtype, stream);
    }
    if (x_ok && fn == JA_FN_IDENT && agg == JA_AGG_MAX && n_in == 1 && o == R) {
        if (!stat_ok(out)) return ja_fail(JA_ERR_DTYPE, "statistics relations are f32");
        ra.x = ja_view(inputs[0]); ra.s0 = ja_view(out);
        return ja_launch_row(ROW_MAX, ra, inputs[0]->dtype, stream);
    }
    if (x_ok && fn == JA_FN_EXP_SUB && agg == JA_AGG_SUM && n_in == 2 && in[1] == R && o == R) {
        if (!stat_ok(out) || !stat_ok(inputs[1])) return ja_fail(JA_ERR_DTYPE, "statistics relations are f32");
        ra.x = ja_view(inputs[0]); ra.s0 = ja_view(inputs[1]); ra.s1 = ja_view(out);
        return ja_launch_row(ROW_EXPSUM, ra, inputs[0]->dtype, stream);
    }
    if (x_ok && fn == JA_FN_RMS_SCALE && agg == JA_AGG_NONE && n_in == 3 && in[1] == R && in[2] == x.substr(x.size() - 1) && o == x) {
        if (!stat_ok(inputs[1]) || inputs[2]->dtype != inputs[0]->dtype || out->dtype != inputs[0]->dtype)
            return ja_fail(JA_ERR_DTYPE, "RMS_SCALE: x, g, y share a dtype; ss is f32");
        ra.x = ja_view(inputs[0]); ra.s0 = ja_view(inputs[1]); ra.g = ja_view(inputs[2]); ra.y = ja_view(out);
        ra.eps = spec->params.empty() ? 1e-5f : (float)spec->params[0];
        return ja_launch_row(ROW_RMS_SCALE, ra, inputs[0]->dtype, stream);
    }
    if (x_ok && fn == JA_FN_EXP_SUB_DIV && agg == JA_AGG_NONE && n_in == 3 && in[1] == R && in[2] == R && o == x) {
        if (!stat_ok(inputs[1]) || !stat_ok(inputs[2]) || out->dtype != inputs[0]->dtype)
            return ja_fail(JA_ERR_DTYPE, "EXP_SUB_DIV: x, y share a dtype; m, l are f32");
        ra.x = ja_view(inputs[0]); ra.s0 = ja_view(inputs[1]); ra.s1 = ja_view(inputs[2]); ra.y = ja_view(out);
        return ja_launch_row(ROW_EXP_SUB_DIV, ra, inputs[0]->dtype, stream);
    }
    if (x_ok && fn == JA_FN_RMSNORM && agg == JA_AGG_NONE && n_in == 2 && in[1] == x.substr(x.size() - 1) && o == x) {
        if (inputs[1]->dtype != inputs[0]->dtype || out->dtype != inputs[0]->dtype)
            return ja_fail(JA_ERR_DTYPE, "RMSNORM: x, g, y share a dtype");
        ra.x = ja_view(inputs[0]); ra.g = ja_view(inputs[1]); ra.y = ja_view(out);
        ra.eps = spec->params.empty() ? 1e-5f : (float)spec->params[0];
        return ja_launch_row(ROW_RMSNORM, ra, inputs[0]->dtype, stream);
    }
    if (x_ok && fn == JA_FN_SOFTMAX && agg == JA_AGG_NONE && n_in == 1 && o == x) {
        if (out->dtype != inputs[0]->dtype) return ja_fail(JA_ERR_DTYPE, "SOFTMAX: x, y share a dtype");
        ra.x = ja_view(inputs[0]); ra.y = ja_view(out);
        return ja_launch_row(ROW_SOFTMAX, ra, inputs[0]->dtype, stream);
    }
    if (fn == JA_FN_ROPE && agg == JA_AGG_NONE && n_in == 1 && x.size() == 4 && o == x) {
        if (out->dtype != inputs[0]->dtype) return ja_fail(JA_ERR_DTYPE, "ROPE: x, y share a dtype");
        const ja_relation* X = inputs[0];
        const int64_t S = X->extent[1], D = X->extent[3];
        if (D % 2) return ja_fail(JA_ERR_SHAPE, "ROPE needs an even last extent");
        for (int64_t sp : X->splits[3])
            if (sp % 2) return ja_fail(JA_ERR_TILING, "ROPE: the last index may be split at even positions only");
        if (!plan->rope_table) {
            // rotation relation R[s,p] = (cos, sin)(s * theta^(-2p/d)), evaluated in fp64, stored in f32
            const double theta = spec->params.empty() ? 1e4 : spec->params[0];
            std::vector<float2> tab((size_t)S * (D / 2));
            for (int64_t s = 0; s < S; ++s)
                for (int64_t p = 0; p < D / 2; ++p) {
                    double phi = (double)s * std::pow(theta, -2.0 * (double)p / (double)D);
                    tab[s * (D / 2) + p] = make_float2((float)std::cos(phi), (float)std::sin(phi));
                }
            JA_CUDA(cudaMalloc((void**)&plan->rope_table, tab.size() * sizeof(float2)));
            JA_CUDA(cudaMemcpy(plan->rope_table, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice));
        }
        ra.x = ja_view(X); ra.y = ja_view(out); ra.rope_table = plan->rope_table; ra.rope_d = (int)D;
        if (X->nblk[3] == 1) {
            // d is unsplit: a block stores, for every (b, s), its heads back to back, so (h, d) collapses into one
            // index of extent H*d whose column blocks are whole heads -- long contiguous rows for the row kernel
            if (!plan->rope_splits) {
                std::vector<int64_t> sp(X->splits[2]);
                for (int64_t& v : sp) v *= D;
                JA_CUDA(cudaMalloc((void**)&plan->rope_splits, sp.size() * sizeof(int64_t)));
                JA_CUDA(cudaMemcpy(plan->rope_splits, sp.data(), sp.size() * sizeof(int64_t), cudaMemcpyHostToDevice));
            }
            for (RelView* v : {&ra.x, &ra.y}) {
                v->rank = 3;
                v->extent[2] *= D; v->bs[2] *= D; v->splits[2] = plan->rope_splits;
                v->extent[3] = 1; v->bs[3] = 1; v->nblk[3] = 1; v->splits[3] = nullptr;
            }
        }
        return ja_launch_row(ROW_ROPE, ra, X->dtype, stream);
    }

    // ---- attention: "bqhd,bkhd,bkhd->bqhd" (or "bqhd,bkgd,bkgd->bqhd", grouped-query) ATTENTION / ONLINE_SOFTMAX ----
    if (fn == JA_FN_ATTENTION && agg == JA_AGG_ONLINE_SOFTMAX && n_in == 3 && x.size() == 4 && in[1].size() == 4 &&
        in[1] == in[2] && o == x && in[1][0] == x[0] && in[1][3] == x[3] && in[1][1] != x[1] && in[1][2] != x[1] &&
        in[1][2] != x[0] && in[1][2] != x[3]) {
        const ja_relation *Q = inputs[0], *K = inputs[1], *V = inputs[2];
        if (Q->dtype == JA_F32 || K->dtype != Q->dtype || V->dtype != Q->dtype || out->dtype != Q->dtype)
            return ja_fail(JA_ERR_DTYPE, "attention relations must share one 16-bit dtype");
        if (Q->extent[3] != 128 || Q->nblk[3] != 1) return ja_fail(JA_ERR_UNSUPPORTED, "attention needs an unsplit last index of extent 128");
        if (Q->extent[1] != K->extent[1]) return ja_fail(JA_ERR_UNSUPPORTED, "attention needs equal query and key extents");
        AttnArgs aa;
        memset(&aa, 0, sizeof aa);
        aa.cache = &plan->attn;
        aa.q = ja_view(Q); aa.k = ja_view(K); aa.v = ja_view(V); aa.o = ja_view(out);
        aa.f16 = Q->dtype == JA_F16;
        if (n_outputs == 2) {   // second output: lse[b, q, h], f32, tiled like the (b, q, h) indices of the output
            ja_relation* L = outputs[1];
            if (!L || L->rank != 3 || L->dtype != JA_F32) return ja_fail(JA_ERR_DTYPE, "the second attention output is an f32 relation over (b, q, h)");
            for (int d = 0; d < 3; ++d)
                if (L->extent[d] != out->extent[d] || L->splits[d] != out->splits[d])
                    return ja_fail(JA_ERR_PARTITION_MISMATCH, "the second attention output must be tiled like the first along its three indices");
            if ((st = ja_relation_to_device(L)) != JA_OK) return st;
            aa.lse = ja_view(L);
            // same closed form as bshd_rows_layout, for cells of 4 bytes and no last index
            bool okl = L->bs[0] && L->bs[2];
            const int64_t S = L->extent[1], bblk = L->bs[0], hblk = L->bs[2], nhb = L->nblk[2];
            for (int32_t bb = 0; okl && bb < L->nblk[0]; ++bb)
                for (int32_t sb = 0; okl && sb < L->nblk[1]; ++sb)
                    for (int32_t hb = 0; okl && hb < L->nblk[2]; ++hb) {
                        const int64_t start = L->splits[1][sb], rows = L->splits[1][sb + 1] - start;
                        okl = L->blk_off[((int64_t)bb * L->nblk[1] + sb) * L->nblk[2] + hb] ==
                              ((bb * bblk * S + bblk * start) * nhb + hb * bblk * rows) * hblk * 4;
                    }
            aa.lse_rows_layout = okl;
        }
        aa.B = (int32_t)Q->extent[0]; aa.S = (int32_t)Q->extent[1]; aa.H = (int32_t)Q->extent[2]; aa.D = 128;
        aa.group = (int32_t)(Q->extent[2] / K->extent[2]);
        int64_t g = Q->extent[1];
        for (int64_t v : Q->splits[1]) g = std::__gcd(g, v);
        for (int64_t v : K->splits[1]) g = std::__gcd(g, v);
        aa.n_ends = spec->params.size() > 2 ? (int32_t)spec->params.size() - 2 : 0;
        for (int i = 0; i < aa.n_ends; ++i) {
            aa.ends[i] = (int32_t)spec->params[2 + i];
            g = std::__gcd(g, (int64_t)aa.ends[i]);
        }
        aa.align = (int32_t)g;
        aa.scale = spec->params.size() >= 1 ? (float)spec->params[0] : 0.08838834764831845f;
        aa.causal = spec->params.size() >= 2 ? (spec->params[1] != 0.0) : 1;
        std::vector<int32_t> qs(Q->splits[1].begin(), Q->splits[1].end()), ks(K->splits[1].begin(), K->splits[1].end());
        aa.q_split = qs.data();
        aa.k_split = ks.data();
        aa.rows_layout = (n_outputs == 1 || aa.lse_rows_layout) && bshd_rows_layout(Q) && bshd_rows_layout(K) && bshd_rows_layout(V) && bshd_rows_layout(out) &&
                         V->splits[1] == K->splits[1] && V->bs[0] == K->bs[0] && V->bs[2] == K->bs[2] &&
                         out->splits[1] == Q->splits[1] && out->bs[0] == Q->bs[0] && out->bs[2] == Q->bs[2];
        return ja_launch_attention(aa, stream);
    }

    // ---- anything else whose operator is a scalar function of the joined cells: the definition, cell by cell --------
    if (n_outputs == 1) {
        bool launched = false;
        if ((st = ja_launch_generic(spec, inputs, out, stream, &launched)) != JA_OK || launched) return st;
    }
    return ja_fail(JA_ERR_UNSUPPORTED, "no kernel for einsum '%s' with fn %d / agg %d", spec->einsum.c_str(), (int)fn,
                   (int)agg);
}

// ---------------------------------------------------------------------------------------------------
// ja_attention_combine: the online-softmax aggregation of partial attention results as a step of its own
// ---------------------------------------------------------------------------------------------------
extern "C" ja_status_t ja_attention_combine(const ja_relation_t* const* o_parts, const ja_relation_t* const* lse_parts, int32_t m,
                                            ja_relation_t* o, ja_relation_t* lse, void* cuda_stream) {
    if (!o_parts || !lse_parts || !o) return ja_fail(JA_ERR_INVALID_ARG, "o_parts / lse_parts / o is NULL");
    if (m < 1 || m > 8) return ja_fail(JA_ERR_UNSUPPORTED, "between 1 and 8 partial results, %d given", m);
    if (o->rank != 4 || o->extent[3] != 128 || o->nblk[3] != 1) return ja_fail(JA_ERR_SHAPE, "o is a [b, s, h, 128] relation with an unsplit last index");
    if (o->dtype != JA_F32 && o->dtype != JA_BF16 && o->dtype != JA_F16) return ja_fail(JA_ERR_DTYPE, "unknown dtype");
    auto stat_like = [&](const ja_relation* r) {
        if (!r || r->rank != 3 || r->dtype != JA_F32) return false;
        for (int d = 0; d < 3; ++d)
            if (r->extent[d] != o->extent[d]) return false;
        return true;
    };
    if (lse && !stat_like(lse)) return ja_fail(JA_ERR_SHAPE, "lse is an f32 relation over (b, s, h)");
    ja_status_t st;
    for (int c = 0; c < m; ++c) {
        const ja_relation* p = o_parts[c];
        if (!p || p->rank != 4 || p->dtype != o->dtype || p->nblk[3] != 1) return ja_fail(JA_ERR_SHAPE, "partial result %d: a relation like o (same dtype, unsplit last index)", c);
        for (int d = 0; d < 4; ++d)
            if (p->extent[d] != o->extent[d]) return ja_fail(JA_ERR_SHAPE, "partial result %d: extents differ from o", c);
        if (!stat_like(lse_parts[c])) return ja_fail(JA_ERR_SHAPE, "lse of partial result %d: an f32 relation over (b, s, h)", c);
        if (p->base == o->base || (lse && lse_parts[c]->base == lse->base)) return ja_fail(JA_ERR_INVALID_ARG, "an output aliases partial result %d", c);
        if ((st = ja_relation_to_device(p)) != JA_OK || (st = ja_relation_to_device(lse_parts[c])) != JA_OK) return st;
    }
    if ((st = ja_relation_to_device(o)) != JA_OK) return st;
    if (lse && (st = ja_relation_to_device(lse)) != JA_OK) return st;
    return ja_launch_attention_combine(o_parts, lse_parts, m, o, lse, (cudaStream_t)cuda_stream);
}

// ---------------------------------------------------------------------------------------------------
// ja_execute_join: step (1) of Definition 3.7 alone (Section 5.1: a producer compiled through its join)
// ---------------------------------------------------------------------------------------------------
extern "C" ja_status_t ja_execute_join(const ja_spec_t* spec, const ja_relation_t* const* inputs, int32_t n_inputs,
                                       ja_relation_t* partials, void* cuda_stream) {
    if (!spec || !inputs || !partials) return ja_fail(JA_ERR_INVALID_ARG, "spec / inputs / partials is NULL");
    const int n_in = (int)spec->ins.size();
    if (n_inputs != n_in) return ja_fail(JA_ERR_INVALID_ARG, "spec has %d operands, %d relations given", n_in, n_inputs);
    ja_status_t st;
    for (int k = 0; k < n_in; ++k)
        if ((st = check_tiling(spec, k, inputs[k])) != JA_OK) return st;
    // multiplicity of every output type: the number of function specs that share it
    int64_t n_out = 1;
    for (char c : spec->out) n_out *= (int64_t)spec->parts[letter_pos(spec->letters, c)].size() - 1;
    std::vector<int32_t> mult((size_t)n_out, 0);
    for (int32_t k : spec->out_keys) ++mult[k];
    const int32_t m = mult.empty() ? 0 : mult[0];
    for (int32_t v : mult)
        if (v != m) return ja_fail(JA_ERR_UNSUPPORTED, "output types have different multiplicities: no rectangular partial relation");
    // partials: [c, out...], c cut into m unit intervals, the rest tiled as out(J)
    const int orank = (int)spec->out.size();
    int64_t oext[JA_MAX_RANK] = {0, 0, 0, 0};
    for (int d = 0; d < orank; ++d) oext[d] = spec->parts[letter_pos(spec->letters, spec->out[d])].back();
    if ((st = check_partial_relation(partials, nullptr, orank, oext)) != JA_OK) return st;
    if (partials->extent[0] != m)
        return ja_fail(JA_ERR_SHAPE, "every output type has %d function specs, the partial relation holds %lld copies", m, (long long)partials->extent[0]);
    for (int d = 0; d < orank; ++d)
        if (partials->splits[d + 1] != spec->parts[letter_pos(spec->letters, spec->out[d])])
            return ja_fail(JA_ERR_PARTITION_MISMATCH, "the partial relation is not tiled as out(J) along index '%c'", spec->out[d]);
    for (int k = 0; k < n_in; ++k)
        if (inputs[k]->base == partials->base) return ja_fail(JA_ERR_INVALID_ARG, "output aliases input %d", k);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const std::vector<std::string>& in = spec->ins;
    const std::string& o = spec->out;
    for (int k = 0; k < n_in; ++k)
        if ((st = ja_relation_to_device(inputs[k])) != JA_OK) return st;
    if ((st = ja_relation_to_device(partials)) != JA_OK) return st;

    if (spec->fn == JA_FN_MUL && spec->agg == JA_AGG_SUM && n_in == 2 && in[0].size() == 2 && in[1].size() == 2 && o.size() == 2 &&
        in[0][1] == in[1][0] && o[0] == in[0][0] && o[1] == in[1][1] && in[0][0] != in[1][1]) {
        const ja_relation *A = inputs[0], *B = inputs[1];
        if (A->dtype != B->dtype) return ja_fail(JA_ERR_DTYPE, "matmul operands must share one dtype");
        std::vector<uint64_t> key = {A->id, B->id, partials->id, ~(uint64_t)0};
        std::lock_guard<std::mutex> plans_lock(spec->plans_mu);
        std::shared_ptr<ExecPlan> plan = spec->plans[key];
        if (!plan) spec->plans[key] = plan = std::make_shared<ExecPlan>();
        if (A->dtype != JA_F32) {
            if (!plan->gemm_checked) {
                bool ok = false;
                GemmEpilogue ep;
                memset(&ep, 0, sizeof ep);
                ep.partials = 1;
                if ((st = ja_gemm_tc_plan(A, B, partials, &ep, &plan->gemm, &ok)) != JA_OK) return st;
                if (!ok) plan->gemm.reset();
                plan->gemm_checked = true;
            }
            if (plan->gemm) return ja_launch_gemm_tc(*plan->gemm, stream);
        }
        if (partials->dtype != A->dtype) return ja_fail(JA_ERR_UNSUPPORTED, "this tiling needs a partial relation of the operands' dtype");
        return ja_launch_matmul_simt(A, B, partials, stream, true);
    }
    return ja_fail(JA_ERR_UNSUPPORTED, "join-only execution has no kernel for einsum '%s' with fn %d / agg %d", spec->einsum.c_str(),
                   (int)spec->fn, (int)spec->agg);
}
