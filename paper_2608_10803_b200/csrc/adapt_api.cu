// C ABI of the library: plan cache (online O(1) dispatch, Section 3.2), launch_map (TilingKey ->
// compiled kernel), tensor-map construction, workspace management and the launches themselves.
#include <atomic>
#include <chrono>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <tuple>
#include <unordered_map>
#include <vector>

#include <cuda.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>

#include "adapt_internal.h"
#include "aux_kernels.cuh"
#include "skinny_gemm.cuh"
#include "cluster_gemm.cuh"
#include "umma_gemm.cuh"

using namespace adapt;

// ---------------------------------------------------------------------------------------------
// error reporting (thread-local)
// ---------------------------------------------------------------------------------------------
static thread_local adapt_status_t tl_status = ADAPT_OK;
static thread_local char tl_message[256] = "";

static adapt_status_t fail(adapt_status_t st, const char* fmt, const char* detail = "")
{
    tl_status = st;
    snprintf(tl_message, sizeof(tl_message), fmt, detail);
    return st;
}

#define CUDA_TRY(expr)                                                        \
    do {                                                                      \
        cudaError_t e__ = (expr);                                             \
        if (e__ != cudaSuccess) return fail(ADAPT_ERR_CUDA, #expr ": %s", cudaGetErrorString(e__)); \
    } while (0)

// ---------------------------------------------------------------------------------------------
// plans and the plan cache
// ---------------------------------------------------------------------------------------------
// One cached encoding of an operand's tensor map(s).  The key is everything the encoding depends on: the base
// pointer, the row pitch, the extents and the box (one plan can reach the same buffer with two geometries:
// a k-class plan falls back to plain tiles when B's pointer is unaligned), and the number of maps.
struct MapSlot {
    const void* ptr = nullptr;
    int64_t pitch = 0, inner = 0, outer = 0;
    int box_inner = 0, box_outer = 0;
    int count = 0;            // 1, or the number of per-class maps (8 or 16)
    std::vector<CUtensorMap> map;
    bool matches(const void* p, int64_t pi, int64_t in, int64_t ou, int bi, int bo, int n) const
    {
        return ptr == p && pitch == pi && inner == in && outer == ou && box_inner == bi && box_outer == bo && count == n;
    }
};
constexpr int kMapSlots = 8;   // most recent distinct (pointer, geometry) pairs kept per operand and plan

struct adapt_plan_s {
    Shape s;
    Config c;
    bool selected = false;    // the plan adapt_matmul_plan returns for its shape (not a forced-key plan)
    bool noop = false;        // M == 0 or N == 0
    bool zero_fill = false;   // K == 0
    std::mutex mu;            // guards the tensor-map slots
    std::vector<MapSlot> maps[3];   // per operand (kMapA, kMapB, kMapC): up to kMapSlots entries, replaced round-robin
    int next[3] = {0, 0, 0};
};
enum { kMapA = 0, kMapB = 1, kMapC = 2 };
typedef adapt_plan_s Plan;

namespace {

// Open-addressing table keyed by a 64-bit shape word.  Readers take no lock: an entry's plan
// pointer is published before its key.  Inserts and growth are serialised by a mutex; a grown
// table replaces the old one, which is kept until shutdown so that concurrent readers stay valid.
struct Table {
    size_t cap;
    std::atomic<uint64_t>* keys;
    std::atomic<Plan*>* vals;
    explicit Table(size_t c) : cap(c)
    {
        keys = new std::atomic<uint64_t>[c];
        vals = new std::atomic<Plan*>[c];
        for (size_t i = 0; i < c; ++i) { keys[i].store(0, std::memory_order_relaxed); vals[i].store(nullptr, std::memory_order_relaxed); }
    }
    ~Table() { delete[] keys; delete[] vals; }
};

inline uint64_t mix64(uint64_t x)
{
    x ^= x >> 33; x *= 0xff51afd7ed558ccdull; x ^= x >> 33; x *= 0xc4ceb9fe1a85ec53ull; x ^= x >> 33;
    return x;
}

// dims below 2^20 pack into one word: [63] valid, [62] dtype, [61] layoutA, [60] layoutB, 3 x 20 bits
inline bool shape_word(const Shape& s, uint64_t* w)
{
    if ((uint64_t)s.M >= (1u << 20) || (uint64_t)s.N >= (1u << 20) || (uint64_t)s.K >= (1u << 20)) return false;
    *w = (1ull << 63) | ((uint64_t)s.dtype << 62) | ((uint64_t)s.layoutA << 61) | ((uint64_t)s.layoutB << 60) |
         ((uint64_t)s.M << 40) | ((uint64_t)s.N << 20) | (uint64_t)s.K;
    return true;
}

struct State {
    std::mutex mu;                       // inserts, slow-path maps, workspace table, init
    std::atomic<Table*> table{nullptr};
    size_t count = 0;
    std::vector<Table*> retired;
    std::vector<Plan*> all_plans;
    typedef std::tuple<int64_t, int64_t, int64_t, int, int, int, uint64_t> BigKey;
    std::map<BigKey, Plan*> big;         // huge dims, and forced plans (last field = tiling key + 1)

    bool inited = false;
    int device = -1;
    Machine machine;
    Calib calib;
    unsigned int* d_status = nullptr;
    unsigned long long* d_trace = nullptr;   // diagnostic builds only
    struct Workspace { void* ptr = nullptr; size_t bytes = 0; unsigned int epoch = 0; };
    std::unordered_map<cudaStream_t, Workspace> ws;
    // adapt_matmul_host: one three-stage pipeline per caller stream (copy in | kernels | copy out, each on
    // its own stream) with two staging slots, so the copies of consecutive calls overlap the kernels and
    // each other (PCIe is full duplex); a slot is reused once the copy-out of the call that used it last is done
    static constexpr int kHostSlots = 2;
    struct HostPipe {
        cudaStream_t in = nullptr, comp = nullptr, out = nullptr;
        cudaEvent_t ev_in[kHostSlots] = {}, ev_comp[kHostSlots] = {}, ev_out[kHostSlots] = {};
        Workspace stage[kHostSlots];
        int next = 0;
    };
    std::unordered_map<cudaStream_t, HostPipe> pipes;
    PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    std::atomic<int64_t> launches{0};
    std::atomic<int64_t> map_encodes{0};   // tensor maps encoded on the host so far (a cached call encodes none)
    std::atomic<int> map_cache{1};         // 0: every call encodes its maps afresh (measurement of the miss cost)
    int log = 0;
    int shuffle_k = 0;                 // ShuffleK analogue (ADAPT_SHUFFLE_K=1): rotated k-block order per tile; measured, off by default
    // adapt_matmul_batch: up to four internal streams (lanes) between a fork from and a join to the caller's stream
    struct BatchLanes {
        cudaStream_t s[4] = {nullptr, nullptr, nullptr, nullptr};
        cudaEvent_t fork = nullptr, join[4] = {nullptr, nullptr, nullptr, nullptr}, cross[4] = {nullptr, nullptr, nullptr, nullptr};
        bool ready = false;
    } lanes;
    std::mutex batch_mu;               // one batch at a time uses the lanes
    int batch_lanes = 4;               // "batch_streams" option (1 to 4): 1 = the calls of a batch run one after the other on the caller's stream
    int prefetch = 1;                  // L2 prefetch of a kernel's first operands ahead of its dependency wait (ADAPT_PREFETCH=0 turns it off)
    bool class_promo128 = true;        // 128-byte L2 promotion for the strided class views (ADAPT_CLASS_PROMO128=0: 256 as for dense operands)
};

State& st()
{
    static State* s = new State();     // never destroyed: handles stay valid during process exit
    return *s;
}

void apply_env(State& S)
{
    if (const char* e = getenv("ADAPT_FAMILY_MASK")) S.machine.family_mask = (unsigned)strtoul(e, nullptr, 0);
    if (const char* e = getenv("ADAPT_LOG")) S.log = atoi(e);
    if (const char* e = getenv("ADAPT_NO_PDL")) pdl_enabled() = atoi(e) == 0;
    if (const char* e = getenv("ADAPT_PREFETCH")) S.prefetch = atoi(e);
    if (const char* e = getenv("ADAPT_SHUFFLE_K")) S.shuffle_k = atoi(e);
    if (const char* e = getenv("ADAPT_CLASS_PROMO128")) S.class_promo128 = atoi(e) != 0;
    if (const char* e = getenv("ADAPT_WORKSPACE_LIMIT_MB")) S.machine.workspace_limit = (int64_t)atoll(e) << 20;
}

Plan* table_find(Table* t, uint64_t w)
{
    size_t i = (size_t)mix64(w) & (t->cap - 1);
    for (;;) {
        const uint64_t k = t->keys[i].load(std::memory_order_acquire);
        if (k == w) return t->vals[i].load(std::memory_order_relaxed);
        if (k == 0) return nullptr;
        i = (i + 1) & (t->cap - 1);
    }
}

void table_put(Table* t, uint64_t w, Plan* p)
{
    size_t i = (size_t)mix64(w) & (t->cap - 1);
    while (t->keys[i].load(std::memory_order_relaxed) != 0) i = (i + 1) & (t->cap - 1);
    t->vals[i].store(p, std::memory_order_relaxed);
    t->keys[i].store(w, std::memory_order_release);
}

bool valid_shape(int64_t M, int64_t N, int64_t K, int dtype, int lA, int lB)
{
    const int64_t lim = 2147483647ll;
    if (M < 0 || N < 0 || K < 0) { fail(ADAPT_ERR_INVALID_ARG, "negative dimension%s"); return false; }
    if (M > lim || N > lim || K > lim) { fail(ADAPT_ERR_UNSUPPORTED, "dimension above 2^31-1%s"); return false; }
    if ((dtype != 0 && dtype != 1) || (lA != 0 && lA != 1) || (lB != 0 && lB != 1)) {
        fail(ADAPT_ERR_INVALID_ARG, "bad dtype or layout value%s");
        return false;
    }
    return true;
}

Plan* make_plan(State& S, const Shape& s, const uint64_t* forced_key)
{
    Plan* p = new Plan();
    p->s = s;
    if (s.M == 0 || s.N == 0) { p->noop = true; return p; }
    if (s.K == 0) { p->zero_fill = true; return p; }
    if (forced_key) {
        if (!config_from_key(s, *forced_key, S.machine, S.calib, &p->c)) {
            delete p;
            fail(ADAPT_ERR_UNSUPPORTED, "tiling key is not legal for this shape%s");
            return nullptr;
        }
        return p;
    }
    std::vector<Config> cands;
    enumerate_configs(s, S.machine, S.calib, &cands);
    if (cands.empty()) {
        delete p;
        fail(ADAPT_ERR_UNSUPPORTED, "no legal configuration%s");
        return nullptr;
    }
    p->c = cands[0];
    if (S.log) {
        fprintf(stderr, "[adapt] plan %lldx%lldx%lld dt%d: fam %d class %d tile %dx%dx%d st %d P_k %d src %d/%d pred %.2f us (%zu candidates)\n",
                (long long)s.M, (long long)s.N, (long long)s.K, s.dtype, p->c.family, p->c.cls, p->c.BM, p->c.BN, p->c.BK,
                p->c.stages, p->c.P_k, p->c.srcA, p->c.srcB, p->c.predicted_us, cands.size());
    }
    return p;
}

// The plan a shape's adapt_matmul_plan calls return from now on (the caller holds S.mu and has checked that the
// shape has none yet).
void insert_selected(State& S, const Shape& s, Plan* p)
{
    p->selected = true;
    S.all_plans.push_back(p);
    uint64_t w;
    if (!shape_word(s, &w)) {
        S.big[State::BigKey(s.M, s.N, s.K, s.dtype, s.layoutA, s.layoutB, 0)] = p;
        return;
    }
    Table* t = S.table.load(std::memory_order_acquire);
    if (!t || (S.count + 1) * 2 > t->cap) {
        Table* nt = new Table(t ? t->cap * 2 : (size_t)1 << 14);
        if (t) {
            for (size_t i = 0; i < t->cap; ++i) {
                const uint64_t k = t->keys[i].load(std::memory_order_relaxed);
                if (k) table_put(nt, k, t->vals[i].load(std::memory_order_relaxed));
            }
            S.retired.push_back(t);
        }
        S.table.store(nt, std::memory_order_release);
        t = nt;
    }
    table_put(t, w, p);
    ++S.count;
}

Plan* find_selected(State& S, const Shape& s)
{
    uint64_t w;
    if (shape_word(s, &w)) {
        Table* t = S.table.load(std::memory_order_acquire);
        return t ? table_find(t, w) : nullptr;
    }
    auto it = S.big.find(State::BigKey(s.M, s.N, s.K, s.dtype, s.layoutA, s.layoutB, 0));
    return it == S.big.end() ? nullptr : it->second;
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// C ABI: errors
// ---------------------------------------------------------------------------------------------
extern "C" adapt_status_t adapt_last_error(void) { return tl_status; }
extern "C" const char* adapt_last_error_message(void) { return tl_message; }
extern "C" const char* adapt_status_string(adapt_status_t s)
{
    switch (s) {
        case ADAPT_OK: return "ok";
        case ADAPT_ERR_INVALID_ARG: return "invalid argument";
        case ADAPT_ERR_UNSUPPORTED: return "unsupported";
        case ADAPT_ERR_NOMEM: return "out of memory";
        case ADAPT_ERR_CUDA: return "CUDA error";
        case ADAPT_ERR_TIMEOUT: return "device-side wait timed out";
        case ADAPT_ERR_NOT_INIT: return "not initialised";
    }
    return "unknown";
}

// ---------------------------------------------------------------------------------------------
// C ABI: planning
// ---------------------------------------------------------------------------------------------
extern "C" adapt_handle_t adapt_matmul_plan(int64_t M, int64_t N, int64_t K, adapt_dtype_t dtype,
                                            adapt_layout_t layoutA, adapt_layout_t layoutB)
{
    State& S = st();
    Shape s;
    s.M = M; s.N = N; s.K = K; s.dtype = (int)dtype; s.layoutA = (int)layoutA; s.layoutB = (int)layoutB;
    uint64_t w;
    // fast path: a plain hash probe, no lock, no validation beyond what the key packing implies
    if ((uint64_t)s.dtype < 2 && (uint64_t)s.layoutA < 2 && (uint64_t)s.layoutB < 2 && shape_word(s, &w)) {
        Table* t = S.table.load(std::memory_order_acquire);
        if (t) {
            Plan* p = table_find(t, w);
            if (p) return p;
        }
    }
    if (!valid_shape(M, N, K, s.dtype, s.layoutA, s.layoutB)) return nullptr;
    std::lock_guard<std::mutex> lock(S.mu);
    if (!S.inited && S.all_plans.empty()) apply_env(S);
    const bool small = shape_word(s, &w);
    Table* t = S.table.load(std::memory_order_acquire);
    if (small && t) {
        Plan* p = table_find(t, w);
        if (p) return p;
    }
    State::BigKey bk(M, N, K, s.dtype, s.layoutA, s.layoutB, 0);
    if (!small) {
        auto it = S.big.find(bk);
        if (it != S.big.end()) return it->second;
    }
    Plan* p = make_plan(S, s, nullptr);
    if (!p) return nullptr;
    insert_selected(S, s, p);
    return p;
}

extern "C" adapt_handle_t adapt_matmul_plan_forced(int64_t M, int64_t N, int64_t K, adapt_dtype_t dtype,
                                                   adapt_layout_t layoutA, adapt_layout_t layoutB, uint64_t tiling_key)
{
    State& S = st();
    if (!valid_shape(M, N, K, (int)dtype, (int)layoutA, (int)layoutB)) return nullptr;
    if (M == 0 || N == 0 || K == 0) return adapt_matmul_plan(M, N, K, dtype, layoutA, layoutB);
    Shape s;
    s.M = M; s.N = N; s.K = K; s.dtype = (int)dtype; s.layoutA = (int)layoutA; s.layoutB = (int)layoutB;
    std::lock_guard<std::mutex> lock(S.mu);
    if (!S.inited && S.all_plans.empty()) apply_env(S);
    State::BigKey bk(M, N, K, s.dtype, s.layoutA, s.layoutB, tiling_key + 1);
    auto it = S.big.find(bk);
    if (it != S.big.end()) return it->second;
    // a forced plan may use any compiled family, whatever the selection mask says
    Machine saved = S.machine;
    S.machine.family_mask = 0x1Fu;
    Plan* p = make_plan(S, s, &tiling_key);
    S.machine = saved;
    if (!p) return nullptr;
    S.all_plans.push_back(p);
    S.big[bk] = p;
    return p;
}

extern "C" adapt_status_t adapt_plan_info(adapt_handle_t plan, adapt_plan_info_t* out)
{
    if (!plan || !out) return fail(ADAPT_ERR_INVALID_ARG, "null argument%s");
    memset(out, 0, sizeof(*out));
    if (plan->noop || plan->zero_fill) {
        out->M = plan->s.M; out->N = plan->s.N; out->K = plan->s.K;
        out->dtype = plan->s.dtype; out->layoutA = plan->s.layoutA; out->layoutB = plan->s.layoutB;
        return ADAPT_OK;
    }
    fill_info(plan->s, plan->c, out);
    return ADAPT_OK;
}

extern "C" int adapt_plan_candidates(int64_t M, int64_t N, int64_t K, adapt_dtype_t dtype, adapt_layout_t layoutA,
                                     adapt_layout_t layoutB, adapt_plan_info_t* out, int cap)
{
    State& S = st();
    if (!valid_shape(M, N, K, (int)dtype, (int)layoutA, (int)layoutB)) return -1;
    Shape s;
    s.M = M; s.N = N; s.K = K; s.dtype = (int)dtype; s.layoutA = (int)layoutA; s.layoutB = (int)layoutB;
    Machine m;
    {
        std::lock_guard<std::mutex> lock(S.mu);
        if (!S.inited && S.all_plans.empty()) apply_env(S);
        m = S.machine;
    }
    m.family_mask = 0x1Fu;    // list every compiled family, selected or not
    std::vector<Config> cands;
    enumerate_configs(s, m, S.calib, &cands);
    for (int i = 0; i < (int)cands.size() && i < cap && out; ++i) fill_info(s, cands[i], &out[i]);
    return (int)cands.size();
}

extern "C" int adapt_classify(int64_t M, int64_t N, int64_t m, int64_t n, int64_t m1, int64_t n1, int64_t n_core, int64_t acc_bytes)
{
    return classify(M, N, m, n, m1, n1, n_core, acc_bytes);
}
extern "C" double adapt_model_read_volume(int64_t M, int64_t N, int64_t K, int64_t m1, int64_t n1)
{
    return read_volume(M, N, K, m1, n1);
}
extern "C" double adapt_model_write_volume(int cls, int64_t M, int64_t N, int64_t K, int64_t k, int64_t k1)
{
    return write_volume(cls, M, N, K, k, k1);
}
extern "C" double adapt_model_pipeline(int schedule, int64_t Q, int64_t L, double t_M, double t_P, double T_drain)
{
    return pipeline_time(schedule, Q, L, t_M, t_P, T_drain);
}
extern "C" int64_t adapt_plan_cache_size(void)
{
    State& S = st();
    std::lock_guard<std::mutex> lock(S.mu);
    return (int64_t)S.all_plans.size();
}
extern "C" int64_t adapt_launch_count(void) { return st().launches.load(); }
extern "C" int64_t adapt_map_encode_count(void) { return st().map_encodes.load(); }
extern "C" void adapt_set_map_cache(int enabled) { st().map_cache.store(enabled ? 1 : 0); }
// the model's calibration constants by name (the fields of Calib that are plain doubles)
#define ADAPT_CALIB_FIELDS(X) X(launch_us) X(prologue_launch_us) X(hbm_bw) X(l2_bw_per_sm) X(tensor_flops) X(eta_mma_bn128) X(eta_mma_bn64) \
    X(eta_2cta) X(mem_latency_us) X(hbm_latency_us) X(hbm_latency_views_us) X(umma_fixed_us) X(epi_tile_fixed_us) X(epi_us_per_kb) \
    X(pair_drain_factor) X(epi_partial_fixed_us) X(epi_partial_us_per_kb) X(epi_tile_fixed_unaligned_us) X(epi_us_per_kb_unaligned) \
    X(thread_store_exposed) X(thread_store_exposed_pair) X(simt_flops) X(simt_fixed_us) X(simt_step_us) X(halo_edge_tile_us) X(simt_bw_eff) \
    X(skinny_bw_eff_aligned) X(skinny_bw_eff_unaligned) X(skinny_fixed_us) X(skinny_pass_us) X(skinny_step_unaligned_us) X(skinny_mac_rate) \
    X(cluster_fixed_us) X(cluster_stage_us) X(cluster_reduce_us) X(cluster_crowd_us) X(cluster_crowd_stage_us) X(cluster_wave_us) \
    X(cluster_bw_eff) X(streamk_fixup_us) X(streamk_peer_us) X(fused_reduce_us) X(fused_wave_us) X(reduce_launch_us) X(dsmem_bw_per_sm) \
    X(copy_bw_eff) X(hbm_bw_per_sm) X(class_view_sm_eff) X(class_tile_fixed_us) X(class_tile_fixed_unaligned_us) X(pair_class_tile_us) X(kclass_view_sm_eff) \
    X(kclass_unit_fixed_us) X(kclass_tile_drain_us) X(oob_box_penalty) X(reduce_batch_us) X(class_split_bw_eff) \
    X(class_split_bw_eff_per_log2m) X(class_split_fused_bw_eff) X(regroup_bw_eff) X(class_view_bw_eff)

static double* calib_field(Calib& c, const char* name)
{
#define X(f) if (!strcmp(name, #f)) return &c.f;
    ADAPT_CALIB_FIELDS(X)
#undef X
    return nullptr;
}
extern "C" adapt_status_t adapt_set_calibration(const char* name, double value)
{
    State& S = st();
    if (!name || !(value == value)) return fail(ADAPT_ERR_INVALID_ARG, "calibration: null name or NaN%s");
    std::lock_guard<std::mutex> lock(S.mu);
    double* f = calib_field(S.calib, name);
    if (!f) return fail(ADAPT_ERR_INVALID_ARG, "unknown calibration constant %s", name);
    *f = value;
    return ADAPT_OK;
}
extern "C" adapt_status_t adapt_get_calibration(const char* name, double* value)
{
    State& S = st();
    if (!name || !value) return fail(ADAPT_ERR_INVALID_ARG, "calibration: null argument%s");
    std::lock_guard<std::mutex> lock(S.mu);
    const double* f = calib_field(S.calib, name);
    if (!f) return fail(ADAPT_ERR_INVALID_ARG, "unknown calibration constant %s", name);
    *value = *f;
    return ADAPT_OK;
}
extern "C" int adapt_calibration_names(char* out, int cap)
{
    static const char names[] =
#define X(f) #f ","
        ADAPT_CALIB_FIELDS(X)
#undef X
        ;
    const int need = (int)sizeof(names) - 1;      // drop the last comma
    if (out && cap > 0) {
        const int n = need - 1 < cap - 1 ? need - 1 : cap - 1;
        memcpy(out, names, (size_t)n);
        out[n] = 0;
    }
    return need;
}

extern "C" adapt_status_t adapt_set_option(const char* name, int value)
{
    State& S = st();
    if (!name) return fail(ADAPT_ERR_INVALID_ARG, "null option name%s");
    std::lock_guard<std::mutex> lock(S.mu);
    if (!strcmp(name, "shuffle_k")) S.shuffle_k = value ? 1 : 0;
    else if (!strcmp(name, "prefetch")) S.prefetch = value ? 1 : 0;
    else if (!strcmp(name, "batch_streams")) S.batch_lanes = value >= 4 ? 4 : (value >= 2 ? value : 1);
    else return fail(ADAPT_ERR_INVALID_ARG, "unknown option %s", name);
    return ADAPT_OK;
}


// ---------------------------------------------------------------------------------------------
// the persisted offline table (Section 3.2: explore offline, look up online)
// ---------------------------------------------------------------------------------------------
static const char* kTableHeader = "# adapt_matmul plan table v2: M N K dtype layoutA layoutB tiling_key";

extern "C" int64_t adapt_plan_table_save(const char* path)
{
    State& S = st();
    if (!path) { fail(ADAPT_ERR_INVALID_ARG, "null path%s"); return -1; }
    FILE* f = fopen(path, "w");
    if (!f) { fail(ADAPT_ERR_INVALID_ARG, "cannot open %s for writing", path); return -1; }
    std::lock_guard<std::mutex> lock(S.mu);
    int64_t n = 0;
    fprintf(f, "%s\n", kTableHeader);
    for (Plan* p : S.all_plans) {
        if (!p->selected || p->noop || p->zero_fill) continue;
        fprintf(f, "%lld %lld %lld %d %d %d %016llx\n", (long long)p->s.M, (long long)p->s.N, (long long)p->s.K, p->s.dtype,
                p->s.layoutA, p->s.layoutB, (unsigned long long)pack_tiling_key(p->s, p->c));
        ++n;
    }
    fclose(f);
    return n;
}

extern "C" int64_t adapt_plan_table_load(const char* path)
{
    State& S = st();
    if (!path) { fail(ADAPT_ERR_INVALID_ARG, "null path%s"); return -1; }
    FILE* f = fopen(path, "r");
    if (!f) { fail(ADAPT_ERR_INVALID_ARG, "cannot open %s", path); return -1; }
    char line[256];
    if (!fgets(line, sizeof(line), f) || strncmp(line, kTableHeader, strlen(kTableHeader)) != 0) {
        fclose(f);
        fail(ADAPT_ERR_UNSUPPORTED, "%s is not a plan table of this library version", path);
        return -1;
    }
    std::lock_guard<std::mutex> lock(S.mu);
    if (!S.inited && S.all_plans.empty()) apply_env(S);
    int64_t loaded = 0;
    while (fgets(line, sizeof(line), f)) {
        long long M, N, K;
        int dt, lA, lB;
        unsigned long long key;
        if (line[0] == '#' || sscanf(line, "%lld %lld %lld %d %d %d %llx", &M, &N, &K, &dt, &lA, &lB, &key) != 7) continue;
        if (M < 1 || N < 1 || K < 1 || M > 2147483647ll || N > 2147483647ll || K > 2147483647ll || (dt | lA | lB) < 0 || dt > 1 || lA > 1 || lB > 1)
            continue;
        Shape s;
        s.M = M; s.N = N; s.K = K; s.dtype = dt; s.layoutA = lA; s.layoutB = lB;
        if (find_selected(S, s)) continue;                   // a shape keeps the plan it already has
        // a key is taken over only if it is a legal configuration of this shape on this machine; the selection mask
        // does not apply (the table's author chose it)
        Machine saved = S.machine;
        S.machine.family_mask = 0x1Fu;
        const uint64_t k64 = (uint64_t)key;
        Plan* p = make_plan(S, s, &k64);
        S.machine = saved;
        if (!p) continue;
        insert_selected(S, s, p);
        ++loaded;
    }
    fclose(f);
    return loaded;
}

extern "C" int64_t adapt_plan_many(int64_t count, const int64_t* dims, const int32_t* flags, adapt_handle_t* handles)
{
    if (count < 0 || (count > 0 && (!dims || !flags))) { fail(ADAPT_ERR_INVALID_ARG, "null array%s"); return -1; }
    int64_t planned = 0;
    for (int64_t i = 0; i < count; ++i) {
        adapt_handle_t h = adapt_matmul_plan(dims[3 * i], dims[3 * i + 1], dims[3 * i + 2], (adapt_dtype_t)flags[3 * i],
                                             (adapt_layout_t)flags[3 * i + 1], (adapt_layout_t)flags[3 * i + 2]);
        if (handles) handles[i] = h;
        if (h) ++planned;
    }
    return planned;
}

// ---------------------------------------------------------------------------------------------
// launch_map: (family, BN, A major, B major) -> compiled kernel
// ---------------------------------------------------------------------------------------------
typedef const void* UmmaKernel;     // the parameter pack's type depends on the kernel mode: launched through cudaLaunchKernelExC

template <int CG>
static UmmaKernel umma_lookup(int BN, bool a_mn, bool b_mn)
{
#define ADAPT_PICK(bn)                                                               \
    if (BN == bn) {                                                                  \
        if (!a_mn && !b_mn) return (const void*)umma_gemm_kernel<bn, false, false, CG, 0>;    \
        if (!a_mn && b_mn) return (const void*)umma_gemm_kernel<bn, false, true, CG, 0>;      \
        if (a_mn && !b_mn) return (const void*)umma_gemm_kernel<bn, true, false, CG, 0>;      \
        return (const void*)umma_gemm_kernel<bn, true, true, CG, 0>;                          \
    }
    if constexpr (CG == 1) { ADAPT_PICK(64) }
    ADAPT_PICK(128)
    ADAPT_PICK(256)
#undef ADAPT_PICK
    return nullptr;
}

// fused split-K instantiations (1-CTA tiles; the k splits of a tile are one cluster)
static UmmaKernel umma_lookup_fused(int BN, bool a_mn, bool b_mn)
{
#define ADAPT_PICK(bn)                                                                         \
    if (BN == bn) {                                                                            \
        if (!a_mn && !b_mn) return (const void*)umma_gemm_kernel<bn, false, false, 1, 0, true>; \
        if (!a_mn && b_mn) return (const void*)umma_gemm_kernel<bn, false, true, 1, 0, true>;   \
        if (a_mn && !b_mn) return (const void*)umma_gemm_kernel<bn, true, false, 1, 0, true>;   \
        return (const void*)umma_gemm_kernel<bn, true, true, 1, 0, true>;                       \
    }
    ADAPT_PICK(64)
    ADAPT_PICK(128)
    ADAPT_PICK(256)
#undef ADAPT_PICK
    return nullptr;
}

// stream-K instantiations (plain tiles, both families)
template <int CG>
static UmmaKernel umma_lookup_sk(int BN, bool a_mn, bool b_mn)
{
#define ADAPT_PICK(bn)                                                                                \
    if (BN == bn) {                                                                                   \
        if (!a_mn && !b_mn) return (const void*)umma_gemm_kernel<bn, false, false, CG, 0, false, true>; \
        if (!a_mn && b_mn) return (const void*)umma_gemm_kernel<bn, false, true, CG, 0, false, true>;   \
        if (a_mn && !b_mn) return (const void*)umma_gemm_kernel<bn, true, false, CG, 0, false, true>;   \
        return (const void*)umma_gemm_kernel<bn, true, true, CG, 0, false, true>;                       \
    }
    if constexpr (CG == 1) { ADAPT_PICK(64) }
    ADAPT_PICK(128)
    ADAPT_PICK(256)
#undef ADAPT_PICK
    return nullptr;
}
static UmmaKernel launch_map_umma_sk(int family, int BN, bool a_mn, bool b_mn)
{
    return family == ADAPT_FAM_UMMA_1CTA ? umma_lookup_sk<1>(BN, a_mn, b_mn) : umma_lookup_sk<2>(BN, a_mn, b_mn);
}

static UmmaKernel launch_map_umma(int family, int BN, bool a_mn, bool b_mn, int mode = 0, bool fused = false)
{
    if (fused) {
        if (family != ADAPT_FAM_UMMA_1CTA) return nullptr;
        if (mode == 0) return umma_lookup_fused(BN, a_mn, b_mn);
        if (mode == 1) {
            if (BN == 64) return (const void*)umma_gemm_kernel<64, false, true, 1, 1, true>;
            if (BN == 128) return (const void*)umma_gemm_kernel<128, false, true, 1, 1, true>;
            if (BN == 256) return (const void*)umma_gemm_kernel<256, false, true, 1, 1, true>;
            return nullptr;
        }
        if (BN == 128) return (const void*)umma_gemm_kernel<128, false, true, 1, 3, true>;
        if (BN == 256) return (const void*)umma_gemm_kernel<256, false, true, 1, 3, true>;
        return nullptr;
    }
    if (mode == 1 && family == ADAPT_FAM_UMMA_2CTA) {     // 256 rows of one row class per SM pair
        if (BN == 128) return (const void*)umma_gemm_kernel<128, false, true, 2, 1>;
        if (BN == 256) return (const void*)umma_gemm_kernel<256, false, true, 2, 1>;
        if (BN == 144) return (const void*)umma_gemm_kernel<144, false, true, 2, 1>;    // 128 / 192 owned + 16 halo columns, 16 row classes
        if (BN == 208) return (const void*)umma_gemm_kernel<208, false, true, 2, 1>;
        return nullptr;
    }
    if (mode == 1) {                     // row-major A read through per-row-class maps (1-CTA tiles, row-major B)
        if (BN == 64) return (const void*)umma_gemm_kernel<64, false, true, 1, 1>;
        if (BN == 128) return (const void*)umma_gemm_kernel<128, false, true, 1, 1>;
        if (BN == 256) return (const void*)umma_gemm_kernel<256, false, true, 1, 1>;
        if (BN == 80) return (const void*)umma_gemm_kernel<80, false, true, 1, 1>;      // 64 / 128 / 192 owned + 16 halo columns
        if (BN == 144) return (const void*)umma_gemm_kernel<144, false, true, 1, 1>;
        if (BN == 208) return (const void*)umma_gemm_kernel<208, false, true, 1, 1>;
        return nullptr;
    }
    if (mode == 2) {                     // B through per-k-class maps: eight accumulators (BN = 64), or classes as k splits
        if (BN == 64) return (const void*)umma_gemm_kernel<64, false, true, 1, 2>;
        if (BN == 128) return (const void*)umma_gemm_kernel<128, false, true, 1, 3>;
        if (BN == 256) return family == ADAPT_FAM_UMMA_2CTA ? (const void*)umma_gemm_kernel<256, false, true, 2, 3>
                                                             : (const void*)umma_gemm_kernel<256, false, true, 1, 3>;
        return nullptr;
    }
    return family == ADAPT_FAM_UMMA_1CTA ? umma_lookup<1>(BN, a_mn, b_mn) : umma_lookup<2>(BN, a_mn, b_mn);
}

// ---------------------------------------------------------------------------------------------
// init / shutdown
// ---------------------------------------------------------------------------------------------
extern "C" adapt_status_t adapt_init(int device)
{
    State& S = st();
    std::lock_guard<std::mutex> lock(S.mu);
    if (S.inited && S.device == device) return ADAPT_OK;
    if (S.inited) return fail(ADAPT_ERR_INVALID_ARG, "already initialised on another device%s");
    CUDA_TRY(cudaSetDevice(device));
    cudaDeviceProp prop;
    CUDA_TRY(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) {
        char name[128];            // the message buffer holds 256 bytes
        snprintf(name, sizeof(name), "%.120s", prop.name);
        return fail(ADAPT_ERR_UNSUPPORTED, "device is not sm_100 (%s)", name);
    }
    if (S.all_plans.empty()) apply_env(S);
    S.machine.n_sm = prop.multiProcessorCount;
    S.machine.smem_bytes = (int)prop.sharedMemPerBlockOptin;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    CUDA_TRY(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) return fail(ADAPT_ERR_CUDA, "cuTensorMapEncodeTiled not available%s");
    S.encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    CUDA_TRY(cudaMalloc(&S.d_status, sizeof(unsigned int)));
    CUDA_TRY(cudaMemset(S.d_status, 0, sizeof(unsigned int)));
#ifdef ADAPT_TRACE_BUILD
    CUDA_TRY(cudaMalloc(&S.d_trace, 8 * 60002));
    CUDA_TRY(cudaMemset(S.d_trace, 0, 8 * 60002));
#endif
    // opt every tensor-core kernel into the full shared-memory carve-out
    for (int fam = ADAPT_FAM_UMMA_1CTA; fam <= ADAPT_FAM_UMMA_2CTA; ++fam)
        for (int BN : {64, 128, 256})
            for (int a = 0; a < 2; ++a)
                for (int b = 0; b < 2; ++b) {
                    UmmaKernel k = launch_map_umma(fam, BN, a != 0, b != 0);
                    if (!k) continue;
                    CUDA_TRY(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, S.machine.smem_bytes));
                }
    for (int BN : {64, 128, 256, 80, 144, 208})
        CUDA_TRY(cudaFuncSetAttribute(launch_map_umma(ADAPT_FAM_UMMA_1CTA, BN, false, true, 1),
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, S.machine.smem_bytes));
    for (int BN : {64, 128, 256})
        CUDA_TRY(cudaFuncSetAttribute(launch_map_umma(ADAPT_FAM_UMMA_1CTA, BN, false, true, 2),
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, S.machine.smem_bytes));
    CUDA_TRY(cudaFuncSetAttribute(launch_map_umma(ADAPT_FAM_UMMA_2CTA, 256, false, true, 2),
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, S.machine.smem_bytes));
    for (int BN : {128, 256, 144, 208})
        CUDA_TRY(cudaFuncSetAttribute(launch_map_umma(ADAPT_FAM_UMMA_2CTA, BN, false, true, 1),
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, S.machine.smem_bytes));
    for (int BN : {64, 128, 256}) {
        for (int a = 0; a < 2; ++a)
            for (int b = 0; b < 2; ++b)
                CUDA_TRY(cudaFuncSetAttribute(launch_map_umma(ADAPT_FAM_UMMA_1CTA, BN, a != 0, b != 0, 0, true),
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, S.machine.smem_bytes));
        CUDA_TRY(cudaFuncSetAttribute(launch_map_umma(ADAPT_FAM_UMMA_1CTA, BN, false, true, 1, true),
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, S.machine.smem_bytes));
        if (BN != 64)
            CUDA_TRY(cudaFuncSetAttribute(launch_map_umma(ADAPT_FAM_UMMA_1CTA, BN, false, true, 2, true),
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, S.machine.smem_bytes));
    }
    for (int fam = ADAPT_FAM_UMMA_1CTA; fam <= ADAPT_FAM_UMMA_2CTA; ++fam)
        for (int BN : {64, 128, 256})
            for (int a = 0; a < 2; ++a)
                for (int b = 0; b < 2; ++b) {
                    UmmaKernel k = launch_map_umma_sk(fam, BN, a != 0, b != 0);
                    if (k) CUDA_TRY(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, S.machine.smem_bytes));
                }
    // clusters of 2, 4, 8 CTAs of the tcgen05 kernel (one CTA per SM) that the device runs at a time
    for (int i = 0; i < 3; ++i) {
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        const int cs = 2 << i;
        cfg.gridDim = dim3((unsigned)(cs * S.machine.n_sm), 1, 1);
        cfg.blockDim = dim3(kUmmaThreads, 1, 1);
        cfg.dynamicSmemBytes = (size_t)160 * 1024;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cs;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, launch_map_umma(ADAPT_FAM_UMMA_1CTA, 128, false, true, 0, true), &cfg) == cudaSuccess && n >= 1)
            S.machine.umma_clusters[i] = n;
        (void)cudaGetLastError();
    }
    CUDA_TRY(cluster_set_attributes());
    S.machine.max_cluster = cluster_max_size();
    S.device = device;
    S.inited = true;
    return ADAPT_OK;
}

extern "C" void adapt_shutdown(void)
{
    State& S = st();
    std::lock_guard<std::mutex> lock(S.mu);
    if (S.inited) {
        cudaDeviceSynchronize();
        for (auto& kv : S.ws) if (kv.second.ptr) cudaFree(kv.second.ptr);
        S.ws.clear();
        for (auto& kv : S.pipes) {
            State::HostPipe& hp = kv.second;
            for (int b = 0; b < State::kHostSlots; ++b) {
                if (hp.stage[b].ptr) cudaFree(hp.stage[b].ptr);
                if (hp.ev_in[b]) cudaEventDestroy(hp.ev_in[b]);
                if (hp.ev_comp[b]) cudaEventDestroy(hp.ev_comp[b]);
                if (hp.ev_out[b]) cudaEventDestroy(hp.ev_out[b]);
            }
            if (hp.in) cudaStreamDestroy(hp.in);
            if (hp.comp) cudaStreamDestroy(hp.comp);
            if (hp.out) cudaStreamDestroy(hp.out);
        }
        S.pipes.clear();
        if (S.lanes.ready) {
            for (int l = 0; l < 4; ++l) {
                cudaStreamDestroy(S.lanes.s[l]);
                cudaEventDestroy(S.lanes.join[l]);
                cudaEventDestroy(S.lanes.cross[l]);
            }
            cudaEventDestroy(S.lanes.fork);
            S.lanes = State::BatchLanes();
        }
        if (S.d_status) cudaFree(S.d_status);
        S.d_status = nullptr;
    }
    for (Plan* p : S.all_plans) delete p;
    S.all_plans.clear();
    S.big.clear();
    Table* t = S.table.exchange(nullptr);
    delete t;
    for (Table* r : S.retired) delete r;
    S.retired.clear();
    S.count = 0;
    S.inited = false;
    S.device = -1;
    S.launches.store(0);
    S.map_encodes.store(0);
    S.map_cache.store(1);
}

extern "C" adapt_status_t adapt_poll_device_status(void* cuda_stream)
{
    State& S = st();
    if (!S.inited) return fail(ADAPT_ERR_NOT_INIT, "adapt_init has not been called%s");
    CUDA_TRY(cudaStreamSynchronize((cudaStream_t)cuda_stream));
    unsigned int w = 0;
    CUDA_TRY(cudaMemcpy(&w, S.d_status, sizeof(w), cudaMemcpyDeviceToHost));
    if (w) {
        CUDA_TRY(cudaMemset(S.d_status, 0, sizeof(unsigned int)));
        return fail(ADAPT_ERR_TIMEOUT, "a kernel's bounded barrier wait expired%s");
    }
    return ADAPT_OK;
}

// ---------------------------------------------------------------------------------------------
// the online call
// ---------------------------------------------------------------------------------------------
namespace {

// The stream's workspace, at least `bytes` large.  Its first kUmmaFlagBytes are the stream-K flag words: zeroed when the
// workspace is allocated, afterwards only ever set to the epoch of a launch, and *epoch (if asked for) is a value no
// earlier launch on this workspace has used.  The caller's regions start at *out (after the flags).
adapt_status_t get_workspace(State& S, cudaStream_t stream, size_t bytes, void** out, unsigned int* epoch = nullptr, void** flags = nullptr)
{
    *out = nullptr;
    if (bytes == 0 && !epoch) return ADAPT_OK;
    bytes += kUmmaFlagBytes;
    std::lock_guard<std::mutex> lock(S.mu);
    State::Workspace& w = S.ws[stream];
    if (epoch) {
        if (++w.epoch == 0) ++w.epoch;       // 0 is what fresh flags hold
        *epoch = w.epoch;
    }
    if (w.bytes < bytes) {
        if (w.ptr) {
            CUDA_TRY(cudaStreamSynchronize(stream));
            CUDA_TRY(cudaFree(w.ptr));
            w.ptr = nullptr;
            w.bytes = 0;
        }
        const size_t want = (size_t)round_up((int64_t)bytes + (bytes >> 3), 1 << 20);
        cudaError_t e = cudaMalloc(&w.ptr, want);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            w.ptr = nullptr;
            return fail(ADAPT_ERR_NOMEM, "workspace allocation failed: %s", cudaGetErrorString(e));
        }
        w.bytes = want;
        CUDA_TRY(cudaMemsetAsync(w.ptr, 0, kUmmaFlagBytes, stream));
    }
    *out = (uint8_t*)w.ptr + kUmmaFlagBytes;
    if (flags) *flags = w.ptr;
    return ADAPT_OK;
}

// 2D tensor map over a dense 16-bit matrix [outer][pitch] whose logical inner extent is `inner`.
adapt_status_t encode_map(State& S, CUtensorMap* map, const void* base, int dtype, int64_t inner, int64_t outer,
                          int64_t pitch, int box_inner, int box_outer, bool strided_view = false)
{
    const cuuint64_t gdim[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    const cuuint64_t gstride[1] = {(cuuint64_t)pitch * 2};
    const cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = S.encode(map, dtype == 0 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                                const_cast<void*>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                CU_TENSOR_MAP_SWIZZLE_128B,
                                // the class views touch 128 bytes of a row and then jump 8 or 16 rows: fetching 256
                                // bytes around each piece doubles their L2 traffic
                                (strided_view && S.class_promo128) ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char buf[32];
        snprintf(buf, sizeof(buf), "%d", (int)r);
        return fail(ADAPT_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %s", buf);
    }
    return ADAPT_OK;
}

// The slot a new encoding goes to: a fresh one while fewer than kMapSlots exist, then round-robin.
MapSlot& take_slot(Plan* pl, int which)
{
    std::vector<MapSlot>& slots = pl->maps[which];
    if ((int)slots.size() < kMapSlots) { slots.emplace_back(); return slots.back(); }
    int& next = pl->next[which];
    MapSlot& sl = slots[next];
    next = (next + 1) % kMapSlots;
    return sl;
}

adapt_status_t cached_map(State& S, Plan* pl, int which, const void* base, int64_t inner, int64_t outer, int64_t pitch,
                          int box_inner, int box_outer, CUtensorMap* out)
{
    std::lock_guard<std::mutex> lock(pl->mu);
    std::vector<MapSlot>& slots = pl->maps[which];
    const bool use_cache = S.map_cache.load(std::memory_order_relaxed) != 0;
    for (const MapSlot& sl : slots)
        if (use_cache && sl.matches(base, pitch, inner, outer, box_inner, box_outer, 1)) { *out = sl.map[0]; return ADAPT_OK; }
    S.map_encodes.fetch_add(1, std::memory_order_relaxed);
    MapSlot& sl = take_slot(pl, which);
    sl.ptr = nullptr;
    sl.map.resize(1);
    adapt_status_t r = encode_map(S, &sl.map[0], base, pl->s.dtype, inner, outer, pitch, box_inner, box_outer);
    if (r != ADAPT_OK) return r;
    sl.ptr = base; sl.pitch = pitch; sl.inner = inner; sl.outer = outer;
    sl.box_inner = box_inner; sl.box_outer = box_outer; sl.count = 1;
    *out = sl.map[0];
    return ADAPT_OK;
}

// Per-class maps of a row-major matrix (rows x cols, 16-byte aligned base): class j holds the rows with
// row % ncls == j, which all start the same distance sigma_j (elements) after an `align`-byte boundary
// (ncls * cols * 2 is a multiple of `align`: ncls = 8 for 16 bytes, 16 for 32).  Map j: base rounded down
// to that boundary, rows ncls * cols * 2 bytes apart, inner extent cols + sigma_j, so a load reads zeros
// past the row's end.  Used for A (rows = M, cols = K), in k-class mode for B (rows = K, cols = N), and for
// C's stores: there `whole_units` cuts the extent down to whole `align`-byte units (returned in
// extent[]), because TMA clips a stored row in 16-byte units and would overwrite the next row's head.
adapt_status_t cached_class_maps(State& S, Plan* pl, int which, const void* base_ptr, int64_t rows_total, int64_t cols,
                                 int box_rows, int ncls, int align, bool whole_units, CUtensorMap* out, int* sigma,
                                 int* extent = nullptr)
{
    std::lock_guard<std::mutex> lock(pl->mu);
    const int unit = align / 2;                               // elements per aligned unit
    for (int j = 0; j < ncls; ++j) {
        sigma[j] = (int)(((2 * j * cols) & (align - 1)) / 2);
        if (extent) extent[j] = (int)(whole_units ? (cols + sigma[j]) / unit * unit : cols + sigma[j]);
    }
    std::vector<MapSlot>& slots = pl->maps[which];
    const bool use_cache = S.map_cache.load(std::memory_order_relaxed) != 0;
    for (const MapSlot& sl : slots)
        if (use_cache && sl.matches(base_ptr, cols, whole_units ? 1 : 0, rows_total, 64, box_rows, ncls)) {
            memcpy(out, sl.map.data(), ncls * sizeof(CUtensorMap));
            return ADAPT_OK;
        }
    S.map_encodes.fetch_add(ncls, std::memory_order_relaxed);
    MapSlot& sl = take_slot(pl, which);
    sl.ptr = nullptr;
    sl.map.resize(ncls);
    for (int j = 0; j < ncls; ++j) {
        const uint8_t* base = (const uint8_t*)base_ptr + ((2 * j * cols) & ~(int64_t)(align - 1));
        const int64_t rows = std::max<int64_t>(1, ceil_div(rows_total - j, ncls));
        int64_t inner = cols + sigma[j];
        if (whole_units) inner = std::max<int64_t>(unit, inner / unit * unit);
        adapt_status_t r = encode_map(S, &sl.map[j], base, pl->s.dtype, inner, rows, (int64_t)ncls * cols, 64, box_rows, true);
        if (r != ADAPT_OK) return r;
    }
    sl.ptr = base_ptr; sl.pitch = cols; sl.inner = whole_units ? 1 : 0; sl.outer = rows_total;
    sl.box_inner = 64; sl.box_outer = box_rows; sl.count = ncls;
    memcpy(out, sl.map.data(), ncls * sizeof(CUtensorMap));
    return ADAPT_OK;
}

adapt_status_t launch_pad(State& S, const void* src, void* dst, int64_t outer, int64_t inner, int64_t pitch, cudaStream_t stream)
{
    const int64_t chunks = outer * (pitch / 8);
    const int blocks = (int)std::min<int64_t>(ceil_div(chunks, 256), (int64_t)S.machine.n_sm * 16);
    CUDA_TRY(launch_pdl(pad_copy_kernel, dim3(blocks), dim3(256), 0, stream, (const unsigned short*)src, (unsigned short*)dst, outer, inner, pitch));
    S.launches.fetch_add(1, std::memory_order_relaxed);
    CUDA_TRY(cudaGetLastError());
    return ADAPT_OK;
}

// A and B of one call re-pitched by one launch (blocks in proportion to the chunks of each).
adapt_status_t launch_pad2(State& S, const void* srcA, void* dstA, int64_t outerA, int64_t innerA, int64_t pitchA,
                           const void* srcB, void* dstB, int64_t outerB, int64_t innerB, int64_t pitchB, cudaStream_t stream)
{
    const int64_t cap = (int64_t)S.machine.n_sm * 16;
    const int64_t chunksA = outerA * (pitchA / 8), chunksB = outerB * (pitchB / 8);
    const int64_t blocks = std::min<int64_t>(ceil_div(chunksA, 256) + ceil_div(chunksB, 256), cap);
    int64_t blocksA = std::max<int64_t>(1, std::min<int64_t>(blocks - 1, (blocks * chunksA + (chunksA + chunksB) / 2) / (chunksA + chunksB)));
    blocksA = std::min<int64_t>(blocksA, ceil_div(chunksA, 256));
    PadPair q;
    q.src[0] = (const unsigned short*)srcA; q.dst[0] = (unsigned short*)dstA; q.outer[0] = outerA; q.inner[0] = innerA; q.pitch[0] = pitchA;
    q.src[1] = (const unsigned short*)srcB; q.dst[1] = (unsigned short*)dstB; q.outer[1] = outerB; q.inner[1] = innerB; q.pitch[1] = pitchB;
    q.blocks_a = (int)blocksA;
    const int64_t blocksB = std::max<int64_t>(1, std::min<int64_t>(blocks - blocksA, ceil_div(chunksB, 256)));
    CUDA_TRY(launch_pdl(pad_copy2_kernel, dim3((unsigned)(blocksA + blocksB)), dim3(256), 0, stream, q));
    S.launches.fetch_add(1, std::memory_order_relaxed);
    CUDA_TRY(cudaGetLastError());
    return ADAPT_OK;
}

adapt_status_t launch_reduce(State& S, const float* partial, void* C, int64_t M, int64_t N, int P_k, int dtype, cudaStream_t stream,
                             const ReduceEpilogue* epi = nullptr)
{
    ReduceEpilogue ep;
    ep.D = nullptr; ep.d_is_vector = 0; ep.alpha = 1.f; ep.beta = 0.f;
    if (epi) ep = *epi;
    const int64_t Np = partial_pitch(N);
    const int64_t work = M * (Np / 4);
    const int blocks = (int)std::min<int64_t>(ceil_div(work, 256), (int64_t)S.machine.n_sm * 8);
    CUDA_TRY(launch_pdl(splitk_reduce_kernel, dim3(blocks), dim3(256), 0, stream, (const float*)partial, (unsigned short*)C, (int)M, (int)N, (int)Np, (int)P_k, (int)dtype, ep));
    S.launches.fetch_add(1, std::memory_order_relaxed);
    CUDA_TRY(cudaGetLastError());
    return ADAPT_OK;
}

adapt_status_t run_umma(State& S, Plan* pl, const void* A, const void* B, void* C, cudaStream_t stream, const ReduceEpilogue* epi = nullptr)
{
    const Shape& s = pl->s;
    const Config& c = pl->c;
    const bool b_mn = s.layoutB == ADAPT_ROW_MAJOR;       // N contiguous
    // class tiles read A through per-row-class maps: in place when its base is 16-byte aligned (whatever K
    // is), else over a re-pitched copy; the k-class views of B need an aligned base, else B is copied
    const bool classesA = c.srcA == ADAPT_SRC_TMA_CLASSES;
    const bool kclsB = c.srcB == ADAPT_SRC_TMA_CLASSES && ((uintptr_t)B & 15) == 0;
    const bool a_mn = !kclsB && s.layoutA == ADAPT_COL_MAJOR;   // M contiguous (the regrouped A' is always K-major)
    const int64_t Kc = round_up(ceil_div(s.K, 8), 64);          // k-class mode: padded class segment of A'
    const int64_t inA = kclsB ? 8 * Kc : (a_mn ? s.M : s.K), outA = a_mn ? s.K : s.M;
    const int64_t inB = b_mn ? s.N : s.K, outB = b_mn ? s.K : s.N;
    // in place when the rows suit TMA (16-byte multiples, narrow operands whole sectors) and the base is aligned
    const bool a_inner_ok = tma_friendly(s.layoutA == ADAPT_COL_MAJOR ? s.M : s.K);
    const bool padA = classesA ? (((uintptr_t)A & 15) != 0 || class_tiles_copy_a(s))
                               : (!kclsB && (!a_inner_ok || ((uintptr_t)A & 15) != 0));
    const bool padB = !kclsB && (!tma_friendly(inB) || ((uintptr_t)B & 15) != 0);
    const int64_t pitchA = padA ? padded_pitch(inA) : inA;
    const int64_t pitchB = padB ? padded_pitch(inB) : inB;
    // a re-pitched operand is read with its pad columns (zeros): whole sectors per row, also in the last box of a row
    const int64_t extA = padA ? pitchA : inA, extB = padB ? pitchB : inB;
    const size_t szA = (padA || kclsB) ? (size_t)round_up(outA * pitchA * 2, 256) : 0;
    const size_t szB = padB ? (size_t)round_up(outB * pitchB * 2, 256) : 0;

    const int cg = c.cluster;
    const bool halo = classesA && c.BN % 64 != 0;           // class tiles with 16 halo columns (C's rows off 32-byte boundaries)
    const int ncls = halo ? halo_row_classes(s) : 8;        // row classes of a class tile
    struct { CUtensorMap a[16], b[8], c[16]; } maps;
    UmmaParams p;
    int a_box_rows = 128;
    int b_box_k = 64;                                       // k rows one box of a row-major B brings
    memset(p.a_sigma, 0, sizeof(p.a_sigma));
    memset(p.b_sigma, 0, sizeof(p.b_sigma));
    p.cls_kc = (int)Kc;
    p.M = (int)s.M; p.N = (int)s.N; p.K = (int)s.K;
    p.P_m = c.P_m;
    // a plan made for k-class views that has to fall back to a copy of B (unaligned pointer) uses plain tiles
    p.P_n = (c.srcB == ADAPT_SRC_TMA_CLASSES && !kclsB) ? (int)ceil_div(s.N, c.BN) : c.P_n;
    p.kb_total = kclsB ? (int)(Kc / kUmmaBK) : (int)ceil_div(s.K + (classesA ? class_k_slack(s) : 0), kUmmaBK);
    const bool ksplit_cls = kclsB && c.BN != 64;            // k classes as k splits: P_k = 8 * (splits per class)
    if (ksplit_cls) {
        p.kb_per_split = (int)ceil_div(p.kb_total, c.P_k / 8);
        p.P_k = c.P_k;
    } else {
        p.kb_per_split = (int)ceil_div(p.kb_total, c.P_k);
        p.P_k = (int)ceil_div(p.kb_total, p.kb_per_split);    // equals the plan's count unless a fallback changed kb_total
    }
    p.num_units = p.P_m * p.P_n * p.P_k;

    // the plan's fused reduction stands unless a fallback changed the tiling (then: partials in the workspace)
    // (a fused-add epilogue runs in the reduction kernel: the GEMM then always leaves fp32 partials in the workspace)
    const bool fused = !epi && c.fused != 0 && p.P_k == c.P_k && !(c.srcB == ADAPT_SRC_TMA_CLASSES && !kclsB);
    const size_t szP = ((p.P_k > 1 || epi) && !fused) ? (size_t)round_up((int64_t)p.P_k * s.M * partial_pitch(s.N) * 4, 256) : 0;
    // stream-K stands unless a fallback changed the tiling; one fp32 partial tile per CTA
    const bool streamk = !epi && c.streamk != 0 && p.P_k == 1 && !classesA && !kclsB;
    const int sk_slots = S.machine.n_sm / c.cluster;
    const size_t szS = streamk ? (size_t)sk_slots * c.cluster * 128 * c.BN * 4 : 0;
    void* ws = nullptr;
    void* ws_flags = nullptr;
    unsigned int epoch = 0;
    adapt_status_t r = get_workspace(S, stream, szA + szB + szP + szS, &ws, streamk ? &epoch : nullptr, &ws_flags);
    if (r != ADAPT_OK) return r;
    uint8_t* w8 = (uint8_t*)ws;
    const void* a_src = A;
    const void* b_src = B;
    if (kclsB) {
        const int64_t a_sm = s.layoutA == ADAPT_ROW_MAJOR ? s.K : 1, a_sk = s.layoutA == ADAPT_ROW_MAJOR ? 1 : s.M;
        const int64_t work = a_sk == 1 ? s.M * (Kc / 8) : s.M * Kc;   // row-major A: a thread per 64 k of a row; else per 16-byte chunk of A'
        const int blocks = (int)std::min<int64_t>(ceil_div(work, 256), (int64_t)S.machine.n_sm * 16);
        CUDA_TRY(launch_pdl(regroup_a_kernel, dim3(blocks), dim3(256), 0, stream, (const unsigned short*)A, (unsigned short*)w8,
                            (int)s.M, (int)s.K, (int)Kc, a_sm, a_sk));
        S.launches.fetch_add(1, std::memory_order_relaxed);
        CUDA_TRY(cudaGetLastError());
        a_src = w8;
    } else if (padA && padB) {
        if ((r = launch_pad2(S, A, w8, outA, inA, pitchA, B, w8 + szA, outB, inB, pitchB, stream)) != ADAPT_OK) return r;
        a_src = w8;
        b_src = w8 + szA;
    } else if (padA) {
        if ((r = launch_pad(S, A, w8, outA, inA, pitchA, stream)) != ADAPT_OK) return r;
        a_src = w8;
    }
    if (padB && !(padA && !kclsB)) {
        if ((r = launch_pad(S, B, w8 + szA, outB, inB, pitchB, stream)) != ADAPT_OK) return r;
        b_src = w8 + szA;
    }
    float* partial = ((p.P_k > 1 || epi) && !fused) ? (float*)(w8 + szA + szB) : nullptr;

    // K-major operand: one box of 64 k x (rows this CTA owns); MN-major operand: boxes of 64 x 64
    if (classesA) {
        a_box_rows = umma_a_box_rows(s, cg, ncls, false);       // rows of the largest class
        if ((r = cached_class_maps(S, pl, kMapA, a_src, s.M, padA ? pitchA : s.K, a_box_rows, ncls, 16, false, maps.a,
                                   p.a_sigma)) != ADAPT_OK) return r;
    } else {
        // a K-major A of fewer than 128 rows is loaded with a box of just those rows (rounded up to 8):
        // the rows of the stage it leaves untouched only feed accumulator rows that are never stored
        a_box_rows = umma_a_box_rows(s, cg, 0, kclsB);
        if ((r = cached_map(S, pl, kMapA, a_src, extA, outA, pitchA, 64, a_mn ? 64 : a_box_rows, &maps.a[0])) != ADAPT_OK) return r;
    }
    if (kclsB) {
        // rows of B (K x N, N % 8 != 0) by class k % 8: the same construction as A's row classes, 64 x 64 boxes
        if ((r = cached_class_maps(S, pl, kMapB, B, s.K, s.N, 64, 8, 16, false, maps.b, p.b_sigma)) != ADAPT_OK) return r;
    } else {
        // a row-major B whose K fits one k-block is loaded with boxes of just the k rows that exist (rounded up to 8; class
        // tiles shift B's rows by up to 7): boxes of 64 rows that lie mostly beyond K load several times slower when B is wide
        if (b_mn && p.kb_total == 1) b_box_k = (int)std::min<int64_t>(64, round_up(s.K + (classesA ? class_k_slack(s) : 0), 8));
        if ((r = cached_map(S, pl, kMapB, b_src, extB, outB, pitchB, 64, b_mn ? b_box_k : c.BN / cg, &maps.b[0])) != ADAPT_OK) return r;
    }

    // 16-bit output leaves through TMA stores (boxes of 64 elements x 32 rows, one epilogue warp) when the
    // boxes cover whole 32-byte sectors: rows of C on 32-byte boundaries (N % 16 == 0; class tiles then use
    // one map per row class), or halo class tiles, whose maps shift each class onto such a boundary
    p.c_mode = 0;
    // a C too large to stay in L2 is written with an evict-first policy (94851 x 69977 x 12: 3495 -> 3219 us)
    p.c_hint = 2 * s.M * s.N >= ((int64_t)32 << 20) ? 1 : 0;
    // partials that fit in L2 are stored evict-last, so the reduction kernel finds them there (256 x 256 x 262144: 63 -> 59 us)
    p.part_hint = (p.P_k > 1 && szP <= ((size_t)100 << 20)) ? 1 : 0;
    memset(p.c_sigma, 0, sizeof(p.c_sigma));
    memset(p.c_extent, 0, sizeof(p.c_extent));
    if (p.P_k == 1 && !epi && !kclsB && (halo ? ((uintptr_t)C & 15) == 0 : (((uintptr_t)C & 31) == 0 && s.N % 16 == 0))) {
        if (classesA) {
            if ((r = cached_class_maps(S, pl, kMapC, C, s.M, s.N, 32, ncls, 32, true, maps.c, p.c_sigma, p.c_extent)) != ADAPT_OK)
                return r;
        } else {
            if ((r = cached_map(S, pl, kMapC, C, s.N, s.M, s.N, 64, 32, &maps.c[0])) != ADAPT_OK) return r;
        }
        p.c_mode = 1;
    }

    // write-bound shapes (C outweighs the operands) walk the tiles row block by row block
    // (2048 x 97328 x 64: 80 -> 71 us, 94851 x 69977 x 12: 2740 -> 2580 us), unless K is so short that the one A tile all
    // concurrent CTAs of a row block then read is a handful of cache lines and the rows are few (2048 x 97328 x 8: 74 -> 84 us
    // that way; from 64 row blocks on the row-block order wins again: 16384 x 97328 x 8: 653 -> 600 us, 40000 x 40000 x 8: 638 -> 592 us)
    p.raster = (p.P_k == 1 && (double)s.M * (double)s.N >= (double)s.K * ((double)s.M + (double)s.N) &&
                (s.K >= 32 || p.P_n <= 64 || classesA || p.P_m > 32)) ? 1 : 0;
    if (const char* e = getenv("ADAPT_RASTER")) p.raster = atoi(e);
    p.prefetch = S.prefetch;
    p.shuffle_k = S.shuffle_k;
    p.ncls_log2 = ncls == 16 ? 4 : (ncls == 8 ? 3 : (ncls == 4 ? 2 : 1));
    p.force_partial = epi ? 1 : 0;
    p.a_shift_any = 0;
    for (int j = 0; j < 16; ++j) p.a_shift_any |= p.a_sigma[j];
    if (p.a_shift_any) p.a_shift_any = 1;
    p.dtype = s.dtype;
    // the plan's ring depth assumed its own A box; a fallback to copies may need a shallower ring
    p.stages = c.stages;
    const int fused_bytes = fused ? umma_fused_bytes(c.BN, a_box_rows) : 0;
    p.x_rows = a_box_rows;
    p.x_pitch = umma_fused_pitch(c.BN);
    p.sk_tiles = p.sk_q0 = p.sk_rem = 0;
    p.sk_partial = nullptr;
    p.sk_flags = (unsigned int*)ws_flags;
    p.sk_epoch = epoch;
    if (streamk) {
        const StreamK sk = streamk_schedule(p.num_units, sk_slots, p.kb_total);
        p.sk_tiles = (int)sk.sk_tiles; p.sk_q0 = (int)sk.q0; p.sk_rem = (int)sk.rem;
        p.sk_partial = (float*)(w8 + szA + szB + szP);
        p.part_hint = 1;                                    // the partial tiles are read back within microseconds: keep them in L2
    }
    while (p.stages > 2 && umma_smem_bytes(c.BN, cg, p.stages, a_box_rows, p.P_k == 1, fused_bytes) > S.machine.smem_bytes) --p.stages;
    p.a_tx_bytes = a_box_rows * kUmmaBK * 2;
    {
        const int bn_cta = c.BN / cg;
        p.b_tx_bytes = b_mn ? ((bn_cta + 63) / 64) * 64 * b_box_k * 2 : bn_cta * kUmmaBK * 2;
    }
    p.idesc = umma_idesc(s.dtype, a_mn, b_mn, 128 * cg, c.BN);
    p.C = C;
    p.partial = partial;
    p.Np = (int)partial_pitch(s.N);
    p.status = S.d_status;
    p.trace = nullptr;
    p.trace_cta = 0;
#ifdef ADAPT_TRACE_BUILD
    p.trace = S.d_trace;
    if (const char* e = getenv("ADAPT_TRACE_CTA")) p.trace_cta = atoi(e);
#endif

    UmmaKernel k = streamk ? launch_map_umma_sk(c.family, c.BN, a_mn, b_mn)
                           : launch_map_umma(c.family, c.BN, a_mn, b_mn, classesA ? 1 : (kclsB ? 2 : 0), fused);
    if (!k) return fail(ADAPT_ERR_UNSUPPORTED, "no compiled kernel for this tiling key%s");
    const int slots = fused ? umma_cluster_slots(S.machine, p.P_k) : S.machine.n_sm / cg;
    const int launch_cluster = fused ? p.P_k : cg;            // fused split-K: the splits of a tile are one cluster
    const int grid = fused ? std::min(p.P_m * p.P_n, slots) * p.P_k : (streamk ? slots : std::min(p.num_units, slots)) * cg;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(kUmmaThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)umma_smem_bytes(c.BN, cg, p.stages, a_box_rows, p.P_k == 1, fused_bytes);
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)launch_cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    pdl_attribute(&attr[1]);
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    // the kernel takes the maps its mode uses
    TmapPackT<0> pack0;
    TmapPackT<1> pack1;
    TmapPackT<2> pack2;                                     // modes 2 and 3 take the same maps
    static_assert(sizeof(TmapPackT<2>) == sizeof(TmapPackT<3>), "k-class packs share their layout");
    void* args[2] = {nullptr, &p};
    size_t arg_bytes[2] = {sizeof(pack0), sizeof(p)};
    if (classesA) {
        arg_bytes[0] = sizeof(pack1);
        memcpy(pack1.a, maps.a, sizeof(pack1.a)); pack1.b[0] = maps.b[0]; memcpy(pack1.c, maps.c, sizeof(pack1.c));
        args[0] = &pack1;
    } else if (kclsB) {
        arg_bytes[0] = sizeof(pack2);
        pack2.a[0] = maps.a[0]; memcpy(pack2.b, maps.b, sizeof(pack2.b)); pack2.c[0] = maps.c[0];
        args[0] = &pack2;
    } else {
        pack0.a[0] = maps.a[0]; pack0.b[0] = maps.b[0]; pack0.c[0] = maps.c[0];
        args[0] = &pack0;
    }
    CUDA_TRY(launch_exc(&cfg, k, args, arg_bytes, 2));
    S.launches.fetch_add(1, std::memory_order_relaxed);
    if ((p.P_k > 1 || epi) && !fused) return launch_reduce(S, partial, C, s.M, s.N, p.P_k, s.dtype, stream, epi);
    return ADAPT_OK;
}

// The CUDA-core kernel with an explicit split count (the plan's own family, and the stand-in of the families that have
// no fp32 partial path when a fused-add epilogue is asked for).
adapt_status_t run_simt_splits(State& S, const Shape& s, int P_k, const void* A, const void* B, void* C, cudaStream_t stream,
                               const ReduceEpilogue* epi)
{
    const bool partials = P_k > 1 || epi;
    const size_t szP = partials ? (size_t)round_up((int64_t)P_k * s.M * partial_pitch(s.N) * 4, 256) : 0;
    void* ws = nullptr;
    adapt_status_t r = get_workspace(S, stream, szP, &ws);
    if (r != ADAPT_OK) return r;
    SimtParams p;
    p.M = (int)s.M; p.N = (int)s.N; p.K = (int)s.K;
    if (s.layoutA == ADAPT_ROW_MAJOR) { p.a_sm = s.K; p.a_sk = 1; } else { p.a_sm = 1; p.a_sk = s.M; }
    if (s.layoutB == ADAPT_ROW_MAJOR) { p.b_sk = s.N; p.b_sn = 1; } else { p.b_sk = 1; p.b_sn = s.K; }
    p.P_n = (int)ceil_div(s.N, 64);
    p.P_k = partials ? std::max(P_k, 2) : 1;                  // any value > 1 makes the kernel write fp32 partials
    p.Np = (int)partial_pitch(s.N);
    p.kb_per_split = (int)ceil_div(ceil_div(s.K, 16), P_k);
    p.dtype = s.dtype;
    p.prefetch = S.prefetch;
    p.C = (unsigned short*)C;
    p.partial = (float*)ws;
    dim3 grid((unsigned)(ceil_div(s.M, 64) * ceil_div(s.N, 64)), (unsigned)P_k, 1);
    CUDA_TRY(launch_pdl(simt_gemm_kernel, grid, dim3(256), 0, stream, (const unsigned short*)A, (const unsigned short*)B, p));
    S.launches.fetch_add(1, std::memory_order_relaxed);
    CUDA_TRY(cudaGetLastError());
    if (partials) return launch_reduce(S, (const float*)ws, C, s.M, s.N, P_k, s.dtype, stream, epi);
    return ADAPT_OK;
}

adapt_status_t run_simt(State& S, Plan* pl, const void* A, const void* B, void* C, cudaStream_t stream)
{
    const Shape& s = pl->s;
    const Config& c = pl->c;
    const size_t szP = c.P_k > 1 ? (size_t)round_up((int64_t)c.P_k * s.M * partial_pitch(s.N) * 4, 256) : 0;
    void* ws = nullptr;
    adapt_status_t r = get_workspace(S, stream, szP, &ws);
    if (r != ADAPT_OK) return r;
    SimtParams p;
    p.M = (int)s.M; p.N = (int)s.N; p.K = (int)s.K;
    if (s.layoutA == ADAPT_ROW_MAJOR) { p.a_sm = s.K; p.a_sk = 1; } else { p.a_sm = 1; p.a_sk = s.M; }
    if (s.layoutB == ADAPT_ROW_MAJOR) { p.b_sk = s.N; p.b_sn = 1; } else { p.b_sk = 1; p.b_sn = s.K; }
    p.P_n = c.P_n;
    p.P_k = c.P_k;
    p.Np = (int)partial_pitch(s.N);
    p.kb_per_split = (int)ceil_div(ceil_div(s.K, 16), c.P_k);
    p.dtype = s.dtype;
    p.prefetch = S.prefetch;
    p.C = (unsigned short*)C;
    p.partial = (float*)ws;
    dim3 grid((unsigned)((int64_t)c.P_m * c.P_n), (unsigned)c.P_k, 1);
    CUDA_TRY(launch_pdl(simt_gemm_kernel, grid, dim3(256), 0, stream, (const unsigned short*)A, (const unsigned short*)B, p));
    S.launches.fetch_add(1, std::memory_order_relaxed);
    CUDA_TRY(cudaGetLastError());
    if (c.P_k > 1) return launch_reduce(S, (const float*)ws, C, s.M, s.N, c.P_k, s.dtype, stream);
    return ADAPT_OK;
}

adapt_status_t run_cluster(State& S, Plan* pl, const void* A, const void* B, void* C, cudaStream_t stream)
{
    if (launch_cluster(pl->s, pl->c, A, B, C, S.d_status, stream, S.prefetch) != ADAPT_OK) return fail(ADAPT_ERR_CUDA, "cluster kernel launch failed%s");
    S.launches.fetch_add(1, std::memory_order_relaxed);
    CUDA_TRY(cudaGetLastError());
    return ADAPT_OK;
}

adapt_status_t run_skinny(State& S, Plan* pl, const void* A, const void* B, void* C, cudaStream_t stream)
{
    const Shape& s = pl->s;
    const Config& c = pl->c;
    const size_t szP = c.P_k > 1 ? (size_t)round_up((int64_t)c.P_k * s.M * partial_pitch(s.N) * 4, 256) : 0;
    void* ws = nullptr;
    adapt_status_t r = get_workspace(S, stream, szP, &ws);
    if (r != ADAPT_OK) return r;
    r = launch_skinny(s, c, A, B, C, (float*)ws, stream);
    if (r != ADAPT_OK) return fail(r, "skinny kernel launch failed%s");
    S.launches.fetch_add(1, std::memory_order_relaxed);
    CUDA_TRY(cudaGetLastError());
    if (c.P_k > 1) return launch_reduce(S, (const float*)ws, C, s.M, s.N, c.P_k, s.dtype, stream);
    return ADAPT_OK;
}

bool overlaps(const void* a, size_t an, const void* b, size_t bn)
{
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + bn && b0 < a0 + an;
}

}  // namespace

extern "C" adapt_status_t adapt_matmul(adapt_handle_t plan, const void* A, const void* B, void* C, void* cuda_stream)
{
    State& S = st();
    if (!plan) return fail(ADAPT_ERR_INVALID_ARG, "null plan%s");
    if (!S.inited) return fail(ADAPT_ERR_NOT_INIT, "adapt_init has not been called%s");
    Plan* pl = plan;
    const Shape& s = pl->s;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (pl->noop) return ADAPT_OK;
    if (!C) return fail(ADAPT_ERR_INVALID_ARG, "null C%s");
    if (pl->zero_fill) {
        CUDA_TRY(cudaMemsetAsync(C, 0, (size_t)s.M * s.N * 2, stream));
        return ADAPT_OK;
    }
    if (!A || !B) return fail(ADAPT_ERR_INVALID_ARG, "null operand%s");
    if (((uintptr_t)A | (uintptr_t)B | (uintptr_t)C) & 1) return fail(ADAPT_ERR_INVALID_ARG, "operands must be 2-byte aligned%s");
    const size_t nA = (size_t)s.M * s.K * 2, nB = (size_t)s.K * s.N * 2, nC = (size_t)s.M * s.N * 2;
    if (overlaps(C, nC, A, nA) || overlaps(C, nC, B, nB)) return fail(ADAPT_ERR_INVALID_ARG, "C overlaps an input%s");
    switch (pl->c.family) {
        case ADAPT_FAM_UMMA_1CTA:
        case ADAPT_FAM_UMMA_2CTA: return run_umma(S, pl, A, B, C, stream);
        case ADAPT_FAM_SKINNY: return run_skinny(S, pl, A, B, C, stream);
        case ADAPT_FAM_SIMT: return run_simt(S, pl, A, B, C, stream);
        case ADAPT_FAM_CLUSTER: return run_cluster(S, pl, A, B, C, stream);
    }
    return fail(ADAPT_ERR_UNSUPPORTED, "unknown kernel family%s");
}

extern "C" adapt_status_t adapt_addmm(adapt_handle_t plan, const void* A, const void* B, const void* D, int d_is_vector,
                                      float alpha, float beta, void* C, void* cuda_stream)
{
    State& S = st();
    if (!plan) return fail(ADAPT_ERR_INVALID_ARG, "null plan%s");
    if (!S.inited) return fail(ADAPT_ERR_NOT_INIT, "adapt_init has not been called%s");
    Plan* pl = plan;
    const Shape& s = pl->s;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (pl->noop) return ADAPT_OK;
    if (!C || !D) return fail(ADAPT_ERR_INVALID_ARG, "null C or D%s");
    if ((!A || !B) && !pl->zero_fill) return fail(ADAPT_ERR_INVALID_ARG, "null operand%s");
    if (((uintptr_t)A | (uintptr_t)B | (uintptr_t)C | (uintptr_t)D) & 1) return fail(ADAPT_ERR_INVALID_ARG, "operands must be 2-byte aligned%s");
    const size_t nA = (size_t)s.M * s.K * 2, nB = (size_t)s.K * s.N * 2, nC = (size_t)s.M * s.N * 2;
    const size_t nD = d_is_vector ? (size_t)s.N * 2 : nC;
    if (overlaps(C, nC, A, nA) || overlaps(C, nC, B, nB)) return fail(ADAPT_ERR_INVALID_ARG, "C overlaps an input%s");
    // C may be D itself (the in-place update beta * C + alpha * A * B): every element is read before it is written, by the
    // same thread; any other overlap is refused
    if (D != C && overlaps(C, nC, D, nD)) return fail(ADAPT_ERR_INVALID_ARG, "C overlaps D without being D%s");
    ReduceEpilogue ep;
    ep.D = (const unsigned short*)D; ep.d_is_vector = d_is_vector ? 1 : 0; ep.alpha = alpha; ep.beta = beta;
    if (pl->zero_fill) {
        // K == 0: the product is zero; the reduction kernel over zero partial slabs leaves beta * D
        return launch_reduce(S, nullptr, C, s.M, s.N, 0, s.dtype, stream, &ep);
    }
    switch (pl->c.family) {
        case ADAPT_FAM_UMMA_1CTA:
        case ADAPT_FAM_UMMA_2CTA: return run_umma(S, pl, A, B, C, stream, &ep);
        default: break;
    }
    // the warp-level and one-launch families have no fp32 partial path: the CUDA-core kernel stands in, with enough k
    // splits to fill the machine (their shapes are small or skinny)
    const int64_t tiles = ceil_div(s.M, 64) * ceil_div(s.N, 64), ksteps = ceil_div(s.K, 16);
    int64_t pk = pl->c.family == ADAPT_FAM_SIMT ? pl->c.P_k : std::max<int64_t>(1, std::min<int64_t>((4 * (int64_t)S.machine.n_sm) / tiles, ksteps / 4));
    pk = std::max<int64_t>(1, std::min<int64_t>(pk, 256));
    pk = ceil_div(ksteps, ceil_div(ksteps, pk));               // no empty split
    return run_simt_splits(S, s, (int)pk, A, B, C, stream, &ep);
}

extern "C" adapt_status_t adapt_matmul_strided_batch(adapt_handle_t plan, const void* A, int64_t stride_a, const void* B,
                                                     int64_t stride_b, void* C, int64_t stride_c, int64_t batch, void* cuda_stream)
{
    if (batch < 0 || stride_a < 0 || stride_b < 0 || stride_c < 0) return fail(ADAPT_ERR_INVALID_ARG, "negative batch count or stride%s");
    if (!plan) return fail(ADAPT_ERR_INVALID_ARG, "null plan%s");
    if (batch > 1 && !plan->noop && stride_c < plan->s.M * plan->s.N) return fail(ADAPT_ERR_INVALID_ARG, "outputs of the batch overlap%s");
    for (int64_t i = 0; i < batch; ++i) {
        const adapt_status_t r = adapt_matmul(plan, (const unsigned short*)A + i * stride_a, (const unsigned short*)B + i * stride_b,
                                              (unsigned short*)C + i * stride_c, cuda_stream);
        if (r != ADAPT_OK) return r;
    }
    return ADAPT_OK;
}

extern "C" adapt_status_t adapt_matmul_host(adapt_handle_t plan, const void* A_host, const void* B_host, void* C_host,
                                            void* cuda_stream)
{
    State& S = st();
    if (!plan) return fail(ADAPT_ERR_INVALID_ARG, "null plan%s");
    if (!S.inited) return fail(ADAPT_ERR_NOT_INIT, "adapt_init has not been called%s");
    const Shape& s = plan->s;
    if (plan->noop) return ADAPT_OK;
    if (!C_host || ((!A_host || !B_host) && !plan->zero_fill)) return fail(ADAPT_ERR_INVALID_ARG, "null operand%s");
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const size_t nA = (size_t)round_up(s.M * s.K * 2, 256), nB = (size_t)round_up(s.K * s.N * 2, 256);
    const size_t nC = (size_t)round_up(s.M * s.N * 2, 256);
    State::HostPipe* hp = nullptr;
    {
        std::lock_guard<std::mutex> lock(S.mu);
        hp = &S.pipes[stream];
        if (!hp->in) {
            CUDA_TRY(cudaStreamCreateWithFlags(&hp->in, cudaStreamNonBlocking));
            CUDA_TRY(cudaStreamCreateWithFlags(&hp->comp, cudaStreamNonBlocking));
            CUDA_TRY(cudaStreamCreateWithFlags(&hp->out, cudaStreamNonBlocking));
            for (int b = 0; b < State::kHostSlots; ++b) {
                CUDA_TRY(cudaEventCreateWithFlags(&hp->ev_in[b], cudaEventDisableTiming));
                CUDA_TRY(cudaEventCreateWithFlags(&hp->ev_comp[b], cudaEventDisableTiming));
                CUDA_TRY(cudaEventCreateWithFlags(&hp->ev_out[b], cudaEventDisableTiming));
            }
        }
    }
    const int b = hp->next;
    hp->next = (hp->next + 1) % State::kHostSlots;
    // the slot is free once the copy-out of the call that used it last has finished
    State::Workspace& w = hp->stage[b];
    if (w.bytes < nA + nB + nC) {
        CUDA_TRY(cudaStreamSynchronize(hp->out));
        if (w.ptr) CUDA_TRY(cudaFree(w.ptr));
        w.ptr = nullptr;
        w.bytes = 0;
        const size_t want = (size_t)round_up((int64_t)(nA + nB + nC) + (int64_t)((nA + nB + nC) >> 3), 1 << 20);
        cudaError_t e = cudaMalloc(&w.ptr, want);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            w.ptr = nullptr;
            return fail(ADAPT_ERR_NOMEM, "staging allocation failed: %s", cudaGetErrorString(e));
        }
        w.bytes = want;
    } else {
        CUDA_TRY(cudaStreamWaitEvent(hp->in, hp->ev_out[b], 0));
    }
    uint8_t* d8 = (uint8_t*)w.ptr;
    if (s.K > 0) {
        CUDA_TRY(cudaMemcpyAsync(d8, A_host, (size_t)s.M * s.K * 2, cudaMemcpyHostToDevice, hp->in));
        CUDA_TRY(cudaMemcpyAsync(d8 + nA, B_host, (size_t)s.K * s.N * 2, cudaMemcpyHostToDevice, hp->in));
    }
    CUDA_TRY(cudaEventRecord(hp->ev_in[b], hp->in));
    CUDA_TRY(cudaStreamWaitEvent(hp->comp, hp->ev_in[b], 0));
    adapt_status_t r = adapt_matmul(plan, d8, d8 + nA, d8 + nA + nB, (void*)hp->comp);
    if (r != ADAPT_OK) return r;
    CUDA_TRY(cudaEventRecord(hp->ev_comp[b], hp->comp));
    CUDA_TRY(cudaStreamWaitEvent(hp->out, hp->ev_comp[b], 0));
    CUDA_TRY(cudaMemcpyAsync(C_host, d8 + nA + nB, (size_t)s.M * s.N * 2, cudaMemcpyDeviceToHost, hp->out));
    CUDA_TRY(cudaEventRecord(hp->ev_out[b], hp->out));
    // work the caller enqueues on its stream after this call sees C_host complete
    CUDA_TRY(cudaStreamWaitEvent(stream, hp->ev_out[b], 0));
    return ADAPT_OK;
}


// ---------------------------------------------------------------------------------------------
// batched call, measurement support, self-test
// ---------------------------------------------------------------------------------------------
extern "C" adapt_status_t adapt_matmul_batch(int64_t count, const adapt_handle_t* plans, const void* const* A,
                                             const void* const* B, void* const* C, void* cuda_stream)
{
    if (count < 0 || (count > 0 && (!plans || !A || !B || !C))) return fail(ADAPT_ERR_INVALID_ARG, "null array%s");
    State& S = st();
    if (count < 8 || S.batch_lanes < 2 || !S.inited) {
        for (int64_t i = 0; i < count; ++i) {
            const adapt_status_t r = adapt_matmul(plans[i], A[i], B[i], C[i], cuda_stream);
            if (r != ADAPT_OK) return r;
        }
        return ADAPT_OK;
    }
    // Lanes.  The calls of a batch are handed in turn to the lane with the least predicted work queued, so that the
    // launch gaps and the tail of one call fill with the next call's work.  The result is the one of running the calls in
    // order: a call whose output overlaps what the other lane still reads or writes, or whose inputs overlap what it
    // writes, first waits for that lane; a lane remembers the buffers of its last 16 calls, and when that memory is
    // full all other lanes are made to wait for it.  A stream-K call runs with nothing beside it: its CTAs wait for one another and
    // must all be resident, which two such kernels sharing the SMs could deny each other.
    std::lock_guard<std::mutex> batch_lock(S.batch_mu);
    State::BatchLanes& L = S.lanes;
    if (!L.ready) {
        for (int l = 0; l < 4; ++l) {
            CUDA_TRY(cudaStreamCreateWithFlags(&L.s[l], cudaStreamNonBlocking));
            CUDA_TRY(cudaEventCreateWithFlags(&L.join[l], cudaEventDisableTiming));
            CUDA_TRY(cudaEventCreateWithFlags(&L.cross[l], cudaEventDisableTiming));
        }
        CUDA_TRY(cudaEventCreateWithFlags(&L.fork, cudaEventDisableTiming));
        L.ready = true;
    }
    const int NL = S.batch_lanes;
    cudaStream_t user = (cudaStream_t)cuda_stream;
    CUDA_TRY(cudaEventRecord(L.fork, user));
    for (int l = 0; l < NL; ++l) CUDA_TRY(cudaStreamWaitEvent(L.s[l], L.fork, 0));
    struct Range { uintptr_t lo, hi; };
    constexpr size_t kLaneMemory = 32;
    std::vector<Range> reads[4], writes[4];
    double queued[4] = {0.0, 0.0, 0.0, 0.0};
    auto hits = [](const std::vector<Range>& v, uintptr_t lo, uintptr_t hi) {
        for (const Range& r : v) if (lo < r.hi && r.lo < hi) return true;
        return false;
    };
    auto wait_for = [&](int lane, int other) -> adapt_status_t {      // `lane` continues after everything queued on `other`
        CUDA_TRY(cudaEventRecord(L.cross[other], L.s[other]));
        CUDA_TRY(cudaStreamWaitEvent(L.s[lane], L.cross[other], 0));
        return ADAPT_OK;
    };
    adapt_status_t status = ADAPT_OK;
    for (int64_t i = 0; i < count && status == ADAPT_OK; ++i) {
        Plan* pl = plans[i];
        if (!pl) { status = fail(ADAPT_ERR_INVALID_ARG, "null plan%s"); break; }
        const Shape& sh = pl->s;
        const uintptr_t a0 = (uintptr_t)A[i], b0 = (uintptr_t)B[i], c0 = (uintptr_t)C[i];
        const uintptr_t a1 = a0 + (uintptr_t)sh.M * sh.K * 2, b1 = b0 + (uintptr_t)sh.K * sh.N * 2, c1 = c0 + (uintptr_t)sh.M * sh.N * 2;
        int lane = 0;
        for (int l = 1; l < NL; ++l) if (queued[l] < queued[lane]) lane = l;
        const bool alone = pl->c.streamk != 0;
        for (int o = 0; o < NL && status == ADAPT_OK; ++o) {
            if (o == lane) continue;
            if (alone || hits(reads[o], c0, c1) || hits(writes[o], c0, c1) || hits(writes[o], a0, a1) || hits(writes[o], b0, b1)) {
                // everything lane o has queued comes first; what o did before is then ordered before all of this lane's
                // later calls as well, but the other lanes still have to see it: keep o's memory
                status = wait_for(lane, o);
            }
        }
        if (status != ADAPT_OK) break;
        if (reads[lane].size() >= kLaneMemory) {
            // this lane's memory is full: every other lane waits for it, and it starts a new memory
            for (int o = 0; o < NL && status == ADAPT_OK; ++o)
                if (o != lane) status = wait_for(o, lane);
            if (status != ADAPT_OK) break;
            reads[lane].clear();
            writes[lane].clear();
        }
        status = adapt_matmul(pl, A[i], B[i], C[i], (void*)L.s[lane]);
        if (status != ADAPT_OK) break;
        reads[lane].push_back({a0, a1});
        reads[lane].push_back({b0, b1});
        writes[lane].push_back({c0, c1});
        queued[lane] += std::max(1.0, pl->c.predicted_us);
        if (alone)
            for (int o = 0; o < NL && status == ADAPT_OK; ++o)
                if (o != lane) status = wait_for(o, lane);
    }
    // join, also after an error: the caller's stream continues after whatever was queued
    for (int l = 0; l < NL; ++l) {
        if (cudaEventRecord(L.join[l], L.s[l]) == cudaSuccess) (void)cudaStreamWaitEvent(user, L.join[l], 0);
    }
    return status;
}

extern "C" adapt_status_t adapt_matmul_repeat(adapt_handle_t plan, int sets, const void* const* A, const void* const* B,
                                              void* const* C, int calls, void* cuda_stream)
{
    if (sets < 1 || calls < 0 || !A || !B || !C) return fail(ADAPT_ERR_INVALID_ARG, "bad set count or null array%s");
    for (int i = 0; i < calls; ++i) {
        const int j = i % sets;
        const adapt_status_t r = adapt_matmul(plan, A[j], B[j], C[j], cuda_stream);
        if (r != ADAPT_OK) return r;
    }
    return ADAPT_OK;
}

namespace {
double now_us()
{
    return std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now().time_since_epoch()).count();
}
}  // namespace

extern "C" adapt_status_t adapt_measure_dispatch(adapt_handle_t plan, const void* A, const void* B, void* C,
                                                 void* cuda_stream, int calls, adapt_dispatch_cost_t* out)
{
    State& S = st();
    if (!plan || !out || calls < 1) return fail(ADAPT_ERR_INVALID_ARG, "null argument%s");
    if (!S.inited) return fail(ADAPT_ERR_NOT_INIT, "adapt_init has not been called%s");
    memset(out, 0, sizeof(*out));
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // warm-up (workspace, tensor maps), with the launches of one call written down for the bare replay
    static thread_local LaunchRecord rec;
    rec.n = 0;
    adapt_status_t r = adapt_matmul(plan, A, B, C, cuda_stream);
    if (r != ADAPT_OK) return r;
    const int64_t l0 = S.launches.load(), e0 = S.map_encodes.load();
    launch_recorder() = &rec;
    r = adapt_matmul(plan, A, B, C, cuda_stream);
    launch_recorder() = nullptr;
    if (r != ADAPT_OK) return r;
    out->launches_per_call = (int32_t)(S.launches.load() - l0);
    CUDA_TRY(cudaStreamSynchronize(stream));
    cudaEvent_t ev0, ev1;
    CUDA_TRY(cudaEventCreate(&ev0));
    CUDA_TRY(cudaEventCreate(&ev1));
    // batches short enough that the launch queue never fills: the host clock then sees host work only
    const int batch = 128;
    double host[3] = {0, 0, 0}, dev_ms[3] = {0, 0, 0};
    for (int mode = 0; mode < 3; ++mode) {          // 0: cached maps, 1: maps encoded on every call, 2: bare launches
        if (mode == 2 && rec.n != out->launches_per_call) { host[2] = -1.0; break; }
        S.map_cache.store(mode == 1 ? 0 : 1);
        const int64_t enc0 = S.map_encodes.load();
        for (int done = 0; done < calls; done += batch) {
            const int n = std::min(batch, calls - done);
            CUDA_TRY(cudaEventRecord(ev0, stream));
            const double t0 = now_us();
            for (int i = 0; i < n; ++i) {
                if (mode < 2) {
                    r = adapt_matmul(plan, A, B, C, cuda_stream);
                    if (r != ADAPT_OK) { S.map_cache.store(1); return r; }
                } else {
                    for (int l = 0; l < rec.n; ++l) CUDA_TRY(launch_replay(rec.launch[l], stream));
                }
            }
            host[mode] += now_us() - t0;
            CUDA_TRY(cudaEventRecord(ev1, stream));
            CUDA_TRY(cudaStreamSynchronize(stream));
            float ms = 0.f;
            CUDA_TRY(cudaEventElapsedTime(&ms, ev0, ev1));
            dev_ms[mode] += ms;
        }
        if (mode == 1) out->maps_per_call = (int32_t)((S.map_encodes.load() - enc0) / calls);
    }
    S.map_cache.store(1);
    (void)e0;
    cudaEventDestroy(ev0);
    cudaEventDestroy(ev1);
    out->host_us_call = host[0] / calls;
    out->host_us_call_map_miss = host[1] / calls;
    out->host_us_bare_launches = host[2] < 0 ? -1.0 : host[2] / calls;
    out->device_us_call = dev_ms[0] * 1e3 / calls;
    out->device_us_call_map_miss = dev_ms[1] * 1e3 / calls;
    out->device_us_bare_launches = host[2] < 0 ? -1.0 : dev_ms[2] * 1e3 / calls;
    return ADAPT_OK;
}

extern "C" adapt_status_t adapt_measure_empty_launch(int launches, int programmatic, void* cuda_stream,
                                                     double* host_us, double* device_us)
{
    if (launches < 1 || !host_us || !device_us) return fail(ADAPT_ERR_INVALID_ARG, "bad argument%s");
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const bool saved = pdl_enabled();
    pdl_enabled() = programmatic != 0;
    cudaEvent_t ev0, ev1;
    CUDA_TRY(cudaEventCreate(&ev0));
    CUDA_TRY(cudaEventCreate(&ev1));
    for (int i = 0; i < 16; ++i) (void)launch_pdl(empty_kernel, dim3(1), dim3(32), 0, stream, 0);
    CUDA_TRY(cudaStreamSynchronize(stream));
    const int batch = 128;
    double host = 0, dev_ms = 0;
    for (int done = 0; done < launches; done += batch) {
        const int n = std::min(batch, launches - done);
        CUDA_TRY(cudaEventRecord(ev0, stream));
        const double t0 = now_us();
        for (int i = 0; i < n; ++i) (void)launch_pdl(empty_kernel, dim3(1), dim3(32), 0, stream, i);
        host += now_us() - t0;
        CUDA_TRY(cudaEventRecord(ev1, stream));
        CUDA_TRY(cudaStreamSynchronize(stream));
        float ms = 0.f;
        CUDA_TRY(cudaEventElapsedTime(&ms, ev0, ev1));
        dev_ms += ms;
    }
    pdl_enabled() = saved;
    cudaEventDestroy(ev0);
    cudaEventDestroy(ev1);
    CUDA_TRY(cudaGetLastError());
    *host_us = host / launches;
    *device_us = dev_ms * 1e3 / launches;
    return ADAPT_OK;
}

extern "C" adapt_status_t adapt_measure_store_rate(void* buffer, int64_t rows, int64_t cols, int mode, int tile_cols,
                                                   int order, int hint, int passes, void* cuda_stream, double* device_us)
{
    State& S = st();
    if (!S.inited) return fail(ADAPT_ERR_NOT_INIT, "adapt_init has not been called%s");
    if (!buffer || !device_us || rows < 1 || cols < 64 || cols % 64 != 0 || mode < 0 || mode > 2 || passes < 1 ||
        tile_cols < 64 || tile_cols > 256 || tile_cols % 64 != 0 || ((uintptr_t)buffer & 31) != 0 || rows > 2147483647ll || cols > 2147483647ll)
        return fail(ADAPT_ERR_INVALID_ARG, "store-rate measurement: rows >= 1, cols a multiple of 64, tile_cols 64..256, a 32-byte aligned buffer%s");
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    CUtensorMap map2d, map3d;
    adapt_status_t r = encode_map(S, &map2d, buffer, 0, cols, rows, cols, 64, 32);
    if (r != ADAPT_OK) return r;
    {
        const cuuint64_t gdim[3] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
        const cuuint64_t gstride[2] = {(cuuint64_t)cols * 2, 128};
        const cuuint32_t box[3] = {64, 32, (cuuint32_t)(tile_cols / 64)};
        const cuuint32_t estr[3] = {1, 1, 1};
        const CUresult cr = S.encode(&map3d, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, buffer, gdim, gstride, box, estr,
                                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (cr != CUDA_SUCCESS) {
            if (mode == 1) return fail(ADAPT_ERR_CUDA, "cuTensorMapEncodeTiled refused the 3-d store map%s");
            map3d = map2d;
        }
    }
    FillParams p;
    p.C = (unsigned short*)buffer; p.rows = (int)rows; p.cols = (int)cols; p.tile_cols = tile_cols; p.order = order; p.hint = hint;
    const void* k = mode == 0 ? (const void*)fill_kernel<0> : mode == 1 ? (const void*)fill_kernel<1> : (const void*)fill_kernel<2>;
    const size_t smem = 8 * 16384 + 1024;
    CUDA_TRY(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    cudaEvent_t ev0, ev1;
    CUDA_TRY(cudaEventCreate(&ev0));
    CUDA_TRY(cudaEventCreate(&ev1));
    for (int i = 0; i < passes + 1; ++i) {
        if (i == 1) CUDA_TRY(cudaEventRecord(ev0, stream));
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3((unsigned)S.machine.n_sm, 1, 1);
        cfg.blockDim = dim3(256, 1, 1);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        void* args[3] = {&map2d, &map3d, &p};
        CUDA_TRY(cudaLaunchKernelExC(&cfg, k, args));
    }
    CUDA_TRY(cudaEventRecord(ev1, stream));
    CUDA_TRY(cudaStreamSynchronize(stream));
    float ms = 0.f;
    CUDA_TRY(cudaEventElapsedTime(&ms, ev0, ev1));
    cudaEventDestroy(ev0);
    cudaEventDestroy(ev1);
    *device_us = (double)ms * 1e3 / passes;
    return ADAPT_OK;
}

extern "C" adapt_status_t adapt_selftest_wait_expiry(uint64_t limit_ns, void* cuda_stream)
{
    State& S = st();
    if (!S.inited) return fail(ADAPT_ERR_NOT_INIT, "adapt_init has not been called%s");
    if (limit_ns > 100000000ull) return fail(ADAPT_ERR_INVALID_ARG, "the self-test's wait limit is at most 0.1 s%s");
    CUDA_TRY(launch_pdl(wait_expiry_kernel, dim3(1), dim3(32), 0, (cudaStream_t)cuda_stream, S.d_status, (unsigned long long)limit_ns));
    S.launches.fetch_add(1, std::memory_order_relaxed);
    CUDA_TRY(cudaGetLastError());
    return ADAPT_OK;
}

#ifdef ADAPT_TRACE_BUILD
// Diagnostic builds only: copy the timestamp trace to the host and clear it.
extern "C" int adapt_debug_trace(unsigned long long* out, int n_words)
{
    State& S = st();
    cudaDeviceSynchronize();
    cudaMemcpy(out, S.d_trace, (size_t)n_words * 8, cudaMemcpyDeviceToHost);
    cudaMemset(S.d_trace, 0, 8 * 60002);
    return 0;
}
#endif

// ---------------------------------------------------------------------------------------------
// allocation-free entry point
// ---------------------------------------------------------------------------------------------
// Scratch for the fp32 split-K partials of adapt_matmul_noalloc.  It lives in the library image:
// every device that loads the library carries it.  In host code the name below is only a handle
// for cudaGetSymbolAddress, never a pointer a kernel may be given.
constexpr size_t kNoAllocScratchBytes = (size_t)4 << 20;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
std::atomic<float*> g_noalloc_ptr[kMaxDevices];      // device address of the scratch, per device
std::mutex g_noalloc_mu;
}  // namespace

extern "C" adapt_status_t adapt_matmul_noalloc(int64_t M, int64_t N, int64_t K, adapt_dtype_t dtype,
                                               adapt_layout_t layoutA, adapt_layout_t layoutB,
                                               const void* A, const void* B, void* C, void* cuda_stream)
{
    if (M < 1 || N < 1 || K < 1) return fail(ADAPT_ERR_INVALID_ARG, "adapt_matmul_noalloc needs M, N, K >= 1%s");
    if (M > 2147483647ll || N > 2147483647ll || K > 2147483647ll) return fail(ADAPT_ERR_UNSUPPORTED, "dimension above 2^31-1%s");
    if (((int)dtype != 0 && (int)dtype != 1) || ((int)layoutA != 0 && (int)layoutA != 1) || ((int)layoutB != 0 && (int)layoutB != 1))
        return fail(ADAPT_ERR_INVALID_ARG, "bad dtype or layout value%s");
    if (!A || !B || !C) return fail(ADAPT_ERR_INVALID_ARG, "null operand%s");
    if (((uintptr_t)A | (uintptr_t)B | (uintptr_t)C) & 1) return fail(ADAPT_ERR_INVALID_ARG, "operands must be 2-byte aligned%s");
    const int64_t Np = partial_pitch(N);
    const int64_t slab = M * Np * 4;                       // bytes of one split's partial
    if (slab <= 0 || 2 * slab > (int64_t)kNoAllocScratchBytes)
        return fail(ADAPT_ERR_UNSUPPORTED,
                    "adapt_matmul_noalloc: output too large for the fixed 4 MiB scratch (needs 2 * M * roundup(N,8) * 4 bytes <= 4 MiB)%s");

    int dev = -1;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(ADAPT_ERR_UNSUPPORTED, "device ordinal out of range%s");
    float* scratch = g_noalloc_ptr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        // set-up, once per device, with that device current: ask the runtime for the DEVICE address
        std::lock_guard<std::mutex> lock(g_noalloc_mu);
        scratch = g_noalloc_ptr[dev].load(std::memory_order_acquire);
        if (!scratch) {
            void* ptr = nullptr;
            cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
            if (e != cudaSuccess || !ptr) return fail(ADAPT_ERR_CUDA, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(e));
            scratch = (float*)ptr;
            g_noalloc_ptr[dev].store(scratch, std::memory_order_release);
        }
    }

    const int64_t kblocks = ceil_div(K, 16);
    int64_t pk = std::min<int64_t>(32, (int64_t)kNoAllocScratchBytes / slab);
    pk = std::min<int64_t>(pk, ceil_div(K, 64));
    if (pk < 1) pk = 1;
    if (pk > kblocks) pk = kblocks;
    const int64_t per = ceil_div(kblocks, pk);
    pk = ceil_div(kblocks, per);                           // no empty split

    cudaStream_t stream = (cudaStream_t)cuda_stream;
    SimtParams p;
    p.M = (int)M; p.N = (int)N; p.K = (int)K;
    if (layoutA == ADAPT_ROW_MAJOR) { p.a_sm = K; p.a_sk = 1; } else { p.a_sm = 1; p.a_sk = M; }
    if (layoutB == ADAPT_ROW_MAJOR) { p.b_sk = N; p.b_sn = 1; } else { p.b_sk = 1; p.b_sn = K; }
    p.P_n = (int)ceil_div(N, 64);
    p.P_k = 2;                                             // any value > 1: the kernel then writes fp32 partials
    p.Np = (int)Np;
    p.kb_per_split = (int)per;
    p.dtype = (int)dtype;
    p.prefetch = 0;
    p.C = (unsigned short*)C;
    p.partial = scratch;
    const int64_t tiles = ceil_div(M, 64) * ceil_div(N, 64);
    dim3 grid((unsigned)tiles, (unsigned)pk, 1);
    CUDA_TRY(launch_pdl(simt_gemm_kernel, grid, dim3(256), 0, stream, (const unsigned short*)A, (const unsigned short*)B, p));
    CUDA_TRY(cudaGetLastError());
    const int64_t work = M * (Np / 4);
    const int blocks = (int)std::min<int64_t>(ceil_div(work, 256), 148 * 8);
    CUDA_TRY(launch_pdl(splitk_reduce_kernel, dim3(blocks), dim3(256), 0, stream, (const float*)scratch, (unsigned short*)C, (int)M, (int)N, (int)Np, (int)pk, (int)dtype, ReduceEpilogue{nullptr, 0, 1.f, 0.f}));
    CUDA_TRY(cudaGetLastError());
    st().launches.fetch_add(2, std::memory_order_relaxed);
    return ADAPT_OK;
}
