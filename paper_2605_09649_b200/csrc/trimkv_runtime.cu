// Host side of the trimkv C ABI: handle, device memory, call-order checks, kernel orchestration.
#include <algorithm>
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "trimkv_internal.cuh"

namespace tkv {
static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
static std::atomic<int> g_test_hooks{0};   // testing aids of the handle-less calls (trimkv_set_test_hooks(NULL, ...))
int global_test_hooks() { return g_test_hooks.load(std::memory_order_relaxed); }
bool first_use_on_device(int slot) {
    constexpr int MAX_DEV = 64, SLOTS = 8;
    static std::atomic<bool> seen[SLOTS][MAX_DEV];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEV || slot < 0 || slot >= SLOTS) return true;
    return !seen[slot][dev].exchange(true);
}
}  // namespace tkv

using namespace tkv;

namespace {

thread_local char g_err[512] = "";

trimkv_status fail(trimkv_status s, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return s;
}

#define CUDA_TRY(expr)                                                                                     \
    do {                                                                                                   \
        cudaError_t e__ = (expr);                                                                          \
        if (e__ != cudaSuccess)                                                                            \
            return fail(e__ == cudaErrorMemoryAllocation ? TRIMKV_E_NOMEM : TRIMKV_E_CUDA, "%s: %s", #expr, \
                        cudaGetErrorString(e__));                                                          \
    } while (0)

constexpr int TC_MIN_ROWS = 256;   // rows of one layer from which the gate's hidden layer runs on tensor cores

int ceil_log2(long long v) {
    int b = 0;
    while ((1LL << b) < v) ++b;
    return b;
}

}  // namespace

namespace tkv {
void set_last_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}
}  // namespace tkv

struct Profiler : public tkv::PhaseMarker {
    bool on = false;
    int only = -1;                                 // >= 0: record this phase alone
    std::vector<cudaEvent_t> pool;                 // reusable events
    size_t used = 0;
    std::vector<std::pair<int, std::pair<cudaEvent_t, cudaEvent_t>>> recs;
    cudaEvent_t open_ev[tkv::PH_COUNT] = {};
    cudaEvent_t get() {
        if (used == pool.size()) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
            pool.push_back(e);
        }
        return pool[used++];
    }
    void mark(int phase, int end, cudaStream_t st) override {
        if (!on || recs.size() >= (1u << 18) || (only >= 0 && phase != only)) return;
        cudaEvent_t e = get();
        if (!e) return;
        cudaEventRecord(e, st);
        if (!end) open_ev[phase] = e;
        else if (open_ev[phase]) { recs.push_back({phase, {open_ev[phase], e}}); open_ev[phase] = nullptr; }
    }
    void clear() { recs.clear(); used = 0; for (auto& e : open_ev) e = nullptr; }
    ~Profiler() override { for (cudaEvent_t e : pool) cudaEventDestroy(e); }
};

struct trimkv {
    trimkv_config cfg;
    Profiler prof;
    int B, L, H, Hq, g, d, D, dg, de, elt;
    long long M, P_seq, maxpp, slots_seq, e_max, n_max;
    int pool_bits;
    long long max_pos;
    CacheView cv;
    SelectBuffers sb;
    AttnBuffers ab;
    int32_t *hole, *mover, *cursor;
    float *W1T, *b1, *W2, *b2, *w_g, *gv, *gs0, *u, *g_lam, *g_c;
    float* st_x = nullptr;                                   // staging of trimkv_decode_step_all_host: x or lambda
    char *st_k = nullptr, *st_v = nullptr, *st_q = nullptr, *st_out = nullptr;
    float *W1hi = nullptr, *W1lo = nullptr, *xhi = nullptr, *xlo = nullptr;   // 3xTF32 operands of the tensor-core gate
    GateTcState* tc = nullptr;
    PrefillTcState* ptc = nullptr;   // tensor-core chunk attention (bf16, d = 128), else null
    float b_g;
    bool shared_set;
    std::vector<char> gate_set;
    std::vector<long long> tokens;   // per layer
    long long entries;               // per sequence (all sequences advance together)
    long long rows_max;
    std::vector<void*> allocs;
    // decode_step_all runs on two streams of its own: `fast` (highest priority) carries K/V append, attention and
    // compaction; `side` (lowest priority) carries the gate and the selection beside the attention kernels
    cudaStream_t fast = nullptr, side = nullptr, side2 = nullptr;   // side2: the selection's sampling, beside the gate
    cudaStream_t side_hi = nullptr;                                 // `side` at the priority of `fast` (gate-heavy steps)
    bool overlap = true;
    int test_hooks = 0;              // TRIMKV_TEST_* switches of this handle
    int prio_hi = 0;                 // the device's highest stream priority
    bool shard = false;              // the handle holds a slice of the layers of sequences sharded over ranks
    char* pool_stage = nullptr;      // device staging of trimkv_get_pool, grown on demand
    size_t pool_stage_bytes = 0;
    cudaEvent_t ev_fork = nullptr, ev_append = nullptr, ev_side = nullptr, ev_done = nullptr, ev_sample = nullptr;
};

namespace {

template <class T>
trimkv_status dev_alloc(trimkv* h, T** p, size_t count, bool zero) {
    void* q = nullptr;
    size_t bytes = std::max<size_t>(count * sizeof(T), 256);
    cudaError_t e = cudaMalloc(&q, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(TRIMKV_E_NOMEM, "cudaMalloc of %zu bytes failed: %s", bytes, cudaGetErrorString(e));
    }
    h->allocs.push_back(q);
    if (zero) {
        e = cudaMemset(q, 0, bytes);
        if (e != cudaSuccess) return fail(TRIMKV_E_CUDA, "cudaMemset: %s", cudaGetErrorString(e));
    }
    *p = reinterpret_cast<T*>(q);
    return TRIMKV_OK;
}

trimkv_status init_cache_state(trimkv* h) {
    // free stacks: pops take the lowest page ids first
    std::vector<int32_t> stack((size_t)h->B * h->P_seq);
    for (int b = 0; b < h->B; ++b)
        for (long long p = 0; p < h->P_seq; ++p) stack[(size_t)b * h->P_seq + p] = (int32_t)(h->P_seq - 1 - p);
    CUDA_TRY(cudaMemcpy(h->cv.free_stack, stack.data(), stack.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
    std::vector<int32_t> cnt(h->B, (int32_t)h->P_seq);
    CUDA_TRY(cudaMemcpy(h->cv.free_count, cnt.data(), cnt.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
    std::vector<int4> own((size_t)h->B * h->P_seq, make_int4(-1, 0, 0, 0));
    CUDA_TRY(cudaMemcpy(h->cv.owner, own.data(), own.size() * sizeof(int4), cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemset(h->cv.len, 0, (size_t)h->B * h->L * h->H * sizeof(int32_t)));
    CUDA_TRY(cudaMemset(h->cv.err, 0, sizeof(int32_t)));
    CUDA_TRY(cudaMemset(h->cv.append_failed, 0, (size_t)h->B * h->L * h->H * sizeof(int32_t)));
    CUDA_TRY(cudaMemset(h->sb.stats, 0, (size_t)h->B * 4 * sizeof(long long)));
    CUDA_TRY(cudaMemset(h->cursor, 0, (size_t)h->B * sizeof(int32_t)));
    CUDA_TRY(cudaMemset(h->ab.pool_done, 0, (size_t)h->B * h->L * h->H * sizeof(int32_t)));
    CUDA_TRY(cudaMemset(h->ab.sched, 0, 2 * sizeof(int32_t)));
    launch_select_state_init(h->sb.sel, h->B, 0);
    CUDA_TRY(cudaDeviceSynchronize());
    std::fill(h->tokens.begin(), h->tokens.end(), 0LL);
    h->entries = 0;
    return TRIMKV_OK;
}

trimkv_status check_handle(trimkv_t* h) { return h ? TRIMKV_OK : fail(TRIMKV_E_ARG, "NULL handle"); }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

trimkv_status device_status(trimkv* h) {
    int32_t code = 0;
    CUDA_TRY(cudaMemcpy(&code, h->cv.err, sizeof(code), cudaMemcpyDeviceToHost));
    if (code != 0) return fail((trimkv_status)code, "device-side error %d latched by a kernel", code);
    return TRIMKV_OK;
}

GateParams gate_params(const trimkv* h) {
    GateParams gp;
    gp.W1T = h->W1T; gp.b1 = h->b1; gp.W2 = h->W2; gp.b2 = h->b2; gp.w_g = h->w_g; gp.v = h->gv; gp.s0 = h->gs0; gp.b_g = h->b_g;
    gp.D = h->D; gp.dg = h->dg; gp.de = h->de; gp.H = h->H; gp.horizon = h->cfg.horizon;
    return gp;
}

// Gate of one layer for `rows` rows: tensor cores when the call is a dense contraction, else the weight-streaming kernels.
void gate_one_layer(trimkv* h, const float* x, int layer, int rows, float* beta, float* lam, float* c, cudaStream_t st) {
    if (h->tc && rows >= TC_MIN_ROWS) {
        launch_gate_gemm_tc(h->tc, x, rows, layer, h->u, h->cv.err, st);
        launch_gate_out(gate_params(h), h->u, 1, layer, 1, rows, beta, lam, c, st);
    } else {
        launch_gate(gate_params(h), x, h->u, layer, 1, rows, beta, lam, c, st);
    }
}

trimkv_status gate_ready(const trimkv* h, int layer0, int nlayers) {
    if (h->D <= 0) return fail(TRIMKV_E_STATE, "handle was created without a gate (hidden = 0)");
    if (!h->shared_set) return fail(TRIMKV_E_STATE, "shared projection not set");
    for (int l = layer0; l < layer0 + nlayers; ++l)
        if (!h->gate_set[l]) return fail(TRIMKV_E_STATE, "gate of layer %d not set", l);
    return TRIMKV_OK;
}

// Entries per sequence to evict now: global budget, or (fixed per-pool budget: every pool holds the same number of
// entries, one per token seen, cut back to the budget at each eviction) the excess of the pools.
long long eviction_due(const trimkv* h) {
    if (h->cfg.per_pool_budget > 0) {
        const long long per_pool = h->entries / ((long long)h->L * h->H);
        return std::max<long long>(0, per_pool - h->cfg.per_pool_budget) * h->L * h->H;
    }
    return h->entries - h->M;
}

// Entries per sequence the cache has room for between two eviction rounds: what survives a round plus one chunk.
long long capacity_entries(const trimkv* h) {
    if (h->shard) return h->n_max;
    const long long LH = (long long)h->L * h->H;
    return (h->cfg.per_pool_budget > 0 ? (long long)h->cfg.per_pool_budget * LH : h->M) + h->e_max;
}

// Selection on `sel_st`, compaction on `st`; when the two differ the caller orders them with events.
trimkv_status select_impl(trimkv* h, long long k, cudaStream_t sel_st) {
    PhaseMarker* pm = h->prof.on ? &h->prof : nullptr;
    if (pm) pm->mark(PH_SELECT, 0, sel_st);
    if (h->cfg.per_pool_budget > 0)
        launch_select_pools(h->cv, h->tokens[0], h->cfg.per_pool_budget, h->cursor, sel_st);
    else
        launch_select_cache(h->cv, h->sb, h->tokens[0], h->entries, k, h->cursor, h->test_hooks & TRIMKV_TEST_DISTRUST_SAMPLE, sel_st);
    if (pm) pm->mark(PH_SELECT, 1, sel_st);
    return TRIMKV_OK;
}

trimkv_status compact_impl(trimkv* h, cudaStream_t st) {
    PhaseMarker* pm = h->prof.on ? &h->prof : nullptr;
    if (pm) pm->mark(PH_COMPACT, 0, st);
    launch_compact(h->cv, h->hole, h->mover, h->cursor, h->e_max, eviction_due(h), st);
    if (pm) pm->mark(PH_COMPACT, 1, st);
    h->entries -= eviction_due(h);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

trimkv_status evict_impl(trimkv* h, cudaStream_t st) {
    if (h->shard) return fail(TRIMKV_E_STATE, "this handle holds a slice of the layers: run the eviction round with the trimkv_shard_* calls");
    const long long t = h->tokens[0];
    for (int l = 1; l < h->L; ++l)
        if (h->tokens[l] != t) return fail(TRIMKV_E_STATE, "layer %d holds %lld tokens, layer 0 holds %lld", l, h->tokens[l], t);
    const long long k = eviction_due(h);
    if (k <= 0) return TRIMKV_OK;
    select_impl(h, k, st);
    return compact_impl(h, st);
}

trimkv_status attention_impl(trimkv* h, int layer0, int nlayers, const void* q, void* out, cudaStream_t st, int reserve_sms = 0) {
    const long long tiles = (h->entries * h->B / 32) * nlayers / h->L + (long long)nlayers * h->B * h->H;
    const long long tiles_upper = h->entries * h->B / 32 + (long long)nlayers * h->B * h->H;
    launch_attention(h->cv, h->ab, layer0, nlayers, h->Hq, h->cfg.kv_dtype == TRIMKV_DTYPE_BF16, tiles, tiles_upper,
                     h->cfg.retention_bias, h->tokens[layer0], reserve_sms, (h->test_hooks & TRIMKV_TEST_ATTENTION_NO_COPY) != 0,
                     q, out, st, h->prof.on ? &h->prof : nullptr);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

}  // namespace

extern "C" {

void trimkv_default_config(trimkv_config* cfg, int64_t budget_entries, int layers, int kv_heads, int head_dim) {
    if (!cfg) return;
    memset(cfg, 0, sizeof(*cfg));
    cfg->budget_entries = budget_entries;
    cfg->layers = layers;
    cfg->kv_heads = kv_heads;
    cfg->q_heads = kv_heads;
    cfg->head_dim = head_dim;
    cfg->hidden = 0;
    cfg->max_batch = 1;
    cfg->page_size = PAGE;
    cfg->gate_hidden = 512;
    cfg->gate_embed = 64;
    cfg->horizon = 2;
    cfg->kv_dtype = TRIMKV_DTYPE_BF16;
    cfg->max_chunk = 512;
    cfg->max_pool_pages = 0;
}

trimkv_t* trimkv_create(int64_t budget_entries, int layers, int kv_heads, int head_dim) {
    trimkv_config cfg;
    trimkv_default_config(&cfg, budget_entries, layers, kv_heads, head_dim);
    trimkv_t* h = nullptr;
    if (trimkv_create_ex(&cfg, &h) != TRIMKV_OK) return nullptr;
    return h;
}

trimkv_status trimkv_create_ex(const trimkv_config* cfg, trimkv_t** out) {
    if (!cfg || !out) return fail(TRIMKV_E_ARG, "NULL argument");
    *out = nullptr;
    if (cfg->budget_entries < 1 || cfg->layers < 1 || cfg->kv_heads < 1 || cfg->head_dim < 8 || cfg->max_batch < 1 ||
        cfg->max_chunk < 1)
        return fail(TRIMKV_E_ARG, "budget, layers, kv_heads, head_dim, max_batch and max_chunk must be positive");
    if (cfg->page_size != PAGE) return fail(TRIMKV_E_UNSUPPORTED, "page_size must be %d", PAGE);
    if (cfg->reserved != 0) return fail(TRIMKV_E_ARG, "reserved must be 0");
    if (cfg->q_heads < cfg->kv_heads || cfg->q_heads % cfg->kv_heads) return fail(TRIMKV_E_ARG, "q_heads must be a multiple of kv_heads");
    if (cfg->kv_dtype != TRIMKV_DTYPE_BF16 && cfg->kv_dtype != TRIMKV_DTYPE_F32) return fail(TRIMKV_E_ARG, "unknown kv_dtype");
    if (cfg->head_dim % 8 || cfg->head_dim > 256) return fail(TRIMKV_E_UNSUPPORTED, "head_dim must be a multiple of 8, at most 256");
    if (cfg->horizon < 0 || cfg->horizon > 64) return fail(TRIMKV_E_ARG, "horizon must be in [0, 64]");
    if (cfg->hidden < 0 || (cfg->hidden > 0 && (cfg->hidden % 4 || cfg->gate_hidden < 4 || cfg->gate_hidden % 4 || cfg->gate_embed < 1)))
        return fail(TRIMKV_E_ARG, "hidden and gate_hidden must be multiples of 4, gate_embed positive");
    if (cfg->hidden > 0 && cfg->gate_hidden > 1536) return fail(TRIMKV_E_UNSUPPORTED, "gate_hidden must be at most 1536");
    if ((long long)cfg->layers * cfg->kv_heads > 65536) return fail(TRIMKV_E_UNSUPPORTED, "layers * kv_heads too large");
    if (cfg->per_pool_budget < 0 || (cfg->per_pool_budget > 0 &&
                                     (long long)cfg->per_pool_budget * cfg->layers * cfg->kv_heads > cfg->budget_entries))
        return fail(TRIMKV_E_ARG, "per_pool_budget * layers * kv_heads must not exceed budget_entries (which sizes the cache)");

    if (cfg->shard_total_layers < 0 || (cfg->shard_total_layers > 0 &&
                                        (cfg->shard_layer0 < 0 || cfg->shard_layer0 + cfg->layers > cfg->shard_total_layers ||
                                         cfg->per_pool_budget > 0)))
        return fail(TRIMKV_E_ARG, "shard_layer0 + layers must lie within shard_total_layers (global budget only)");
    if ((long long)cfg->shard_total_layers * cfg->kv_heads > 65536) return fail(TRIMKV_E_UNSUPPORTED, "layers * kv_heads too large");
    trimkv* h = new (std::nothrow) trimkv();
    if (!h) return fail(TRIMKV_E_NOMEM, "host allocation failed");
    h->cfg = *cfg;
    h->B = cfg->max_batch; h->L = cfg->layers; h->H = cfg->kv_heads; h->Hq = cfg->q_heads; h->g = h->Hq / h->H;
    h->d = cfg->head_dim; h->D = cfg->hidden; h->dg = cfg->gate_hidden; h->de = cfg->gate_embed;
    h->elt = cfg->kv_dtype == TRIMKV_DTYPE_BF16 ? 2 : 4;
    h->M = cfg->budget_entries;
    const long long LH = (long long)h->L * h->H;
    h->shard = cfg->shard_total_layers > 0;
    const long long LH_all = h->shard ? (long long)cfg->shard_total_layers * h->H : LH;   // pools of the whole model
    // a round may evict, on this handle, as many entries as the WHOLE model gained since the last round
    h->e_max = (long long)cfg->max_chunk * LH_all;
    h->n_max = h->M + (long long)cfg->max_chunk * LH;
    h->P_seq = (h->n_max + PAGE - 1) / PAGE + LH + 8;
    h->maxpp = cfg->max_pool_pages > 0 ? std::min<long long>(cfg->max_pool_pages, h->P_seq) : h->P_seq;
    h->slots_seq = h->P_seq * PAGE;
    h->pool_bits = std::max(1, ceil_log2(LH_all));
    h->max_pos = std::min<long long>((1LL << 24) - 1, (1LL << (32 - h->pool_bits)) - 1);
    h->tokens.assign(h->L, 0);
    h->gate_set.assign(h->L, 0);
    h->shared_set = false;
    h->b_g = 0.f;
    h->entries = 0;
    h->W1T = h->b1 = h->W2 = h->b2 = h->w_g = h->gv = h->gs0 = h->u = h->g_lam = h->g_c = nullptr;

    CacheView& cv = h->cv;
    memset(&cv, 0, sizeof(cv));
    cv.P_seq = h->P_seq; cv.maxpp = h->maxpp; cv.B = h->B; cv.L = h->L; cv.H = h->H; cv.d = h->d;
    cv.row_bytes = h->d * h->elt;
    cv.swizzle = (cfg->kv_dtype == TRIMKV_DTYPE_BF16 && cv.row_bytes % 128 == 0) ? 1 : 0;
    cv.pool_bits = h->pool_bits;
    cv.pool_offset = h->shard ? cfg->shard_layer0 * h->H : 0;
    const size_t pools = (size_t)h->B * LH;
    const size_t slots = (size_t)h->B * h->slots_seq;
    trimkv_status s = TRIMKV_OK;
    auto A = [&](trimkv_status r) { if (s == TRIMKV_OK) s = r; };
    A(dev_alloc(h, &cv.kv, slots * 2 * cv.row_bytes, true));
    A(dev_alloc(h, &cv.lam, slots, true));
    A(dev_alloc(h, &cv.c, slots, true));
    A(dev_alloc(h, &cv.pos, slots, true));
    A(dev_alloc(h, &cv.owner, (size_t)h->B * h->P_seq, false));
    A(dev_alloc(h, &cv.block_table, pools * h->maxpp, true));
    A(dev_alloc(h, &cv.len, pools, true));
    A(dev_alloc(h, &cv.free_stack, (size_t)h->B * h->P_seq, false));
    A(dev_alloc(h, &cv.free_count, (size_t)h->B, false));
    A(dev_alloc(h, &cv.evict_mask, (size_t)h->B * h->P_seq, true));
    A(dev_alloc(h, &cv.err, 1, true));
    A(dev_alloc(h, &cv.append_failed, pools, true));
    SelectBuffers& sb = h->sb;
    sb.cand_cap = h->n_max;
    A(dev_alloc(h, &sb.sel, (size_t)h->B, true));
    A(dev_alloc(h, &sb.cand, (size_t)h->B * sb.cand_cap, false));
    A(dev_alloc(h, &sb.stats, (size_t)h->B * 4, true));
    A(dev_alloc(h, &sb.sample, (size_t)h->B * 4096, false));
    A(dev_alloc(h, &h->hole, (size_t)h->B * h->e_max, false));
    A(dev_alloc(h, &h->mover, (size_t)h->B * h->e_max, false));
    A(dev_alloc(h, &h->cursor, (size_t)h->B, true));
    AttnBuffers& ab = h->ab;
    const long long tiles_max = (long long)h->B * (h->n_max / 32 + 2 * LH);
    ab.max_items = std::max<long long>(592LL * 32, tiles_max / 32) + 2 * (long long)pools;
    A(dev_alloc(h, &ab.pool_done, pools, true));
    A(dev_alloc(h, &ab.sched, 2, true));
    A(dev_alloc(h, &ab.part_o, (size_t)ab.max_items * h->g * h->d, false));
    A(dev_alloc(h, &ab.part_ml, (size_t)ab.max_items * h->g * 2, false));
    h->rows_max = std::max<long long>((long long)h->B * cfg->max_chunk, (long long)h->L * h->B);
    A(dev_alloc(h, &h->g_lam, (size_t)h->rows_max * h->H, false));
    A(dev_alloc(h, &h->g_c, (size_t)h->rows_max * h->H, false));
    A(dev_alloc(h, &h->st_x, (size_t)h->L * h->B * std::max(h->D, h->H), false));
    A(dev_alloc(h, &h->st_k, (size_t)h->L * h->B * h->H * h->d * h->elt, false));
    A(dev_alloc(h, &h->st_v, (size_t)h->L * h->B * h->H * h->d * h->elt, false));
    A(dev_alloc(h, &h->st_q, (size_t)h->L * h->B * h->Hq * h->d * h->elt, false));
    A(dev_alloc(h, &h->st_out, (size_t)h->L * h->B * h->Hq * h->d * h->elt, false));
    if (h->D > 0) {
        A(dev_alloc(h, &h->W1T, (size_t)h->L * h->dg * h->D, false));
        A(dev_alloc(h, &h->b1, (size_t)h->L * h->dg, false));
        A(dev_alloc(h, &h->W2, (size_t)h->L * h->H * h->de * h->dg, false));
        A(dev_alloc(h, &h->b2, (size_t)h->L * h->H * h->de, false));
        A(dev_alloc(h, &h->w_g, (size_t)h->de, false));
        A(dev_alloc(h, &h->gv, (size_t)h->L * h->H * h->dg, false));
        A(dev_alloc(h, &h->gs0, (size_t)h->L * h->H, false));
        if (s == TRIMKV_OK && gate_tc_supported(h->D, h->dg) && (long long)h->B * cfg->max_chunk >= TC_MIN_ROWS) {
            A(dev_alloc(h, &h->W1hi, (size_t)h->L * h->dg * h->D, true));
            A(dev_alloc(h, &h->W1lo, (size_t)h->L * h->dg * h->D, true));
            A(dev_alloc(h, &h->xhi, (size_t)h->rows_max * h->D, true));
            A(dev_alloc(h, &h->xlo, (size_t)h->rows_max * h->D, true));
            if (s == TRIMKV_OK) h->tc = gate_tc_create(h->xhi, h->xlo, h->rows_max, h->W1hi, h->W1lo, h->L, h->dg, h->D);
        }
        // scratch of the hidden layer: one slab per input-dimension chunk for the calls the streaming kernel takes (every
        // call without the tensor-core form, else only those below its row threshold and the all-layer decode step)
        const long long rows_stream = h->tc ? std::min<long long>(h->rows_max, std::max<long long>(TC_MIN_ROWS, (long long)h->L * h->B))
                                            : h->rows_max;
        A(dev_alloc(h, &h->u, (size_t)std::max<long long>(h->rows_max, rows_stream * gate_chunks(h->D)) * h->dg, false));
    }
    if (s == TRIMKV_OK) {
        int prio_lo = 0, prio_hi = 0;
        cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);     // numerically lower = higher priority
        h->prio_hi = prio_hi;
        if (cudaStreamCreateWithPriority(&h->side, cudaStreamNonBlocking, prio_lo) != cudaSuccess ||
            cudaStreamCreateWithPriority(&h->fast, cudaStreamNonBlocking, prio_hi) != cudaSuccess ||
            cudaStreamCreateWithPriority(&h->side2, cudaStreamNonBlocking, prio_lo) != cudaSuccess ||
            cudaStreamCreateWithPriority(&h->side_hi, cudaStreamNonBlocking, prio_hi) != cudaSuccess ||
            cudaEventCreateWithFlags(&h->ev_sample, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&h->ev_done, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&h->ev_append, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&h->ev_side, cudaEventDisableTiming) != cudaSuccess)
            s = fail(TRIMKV_E_CUDA, "stream or event creation failed: %s", cudaGetErrorString(cudaGetLastError()));
    }
    if (s == TRIMKV_OK) s = init_cache_state(h);
    if (s == TRIMKV_OK) h->ptc = prefill_tc_create(h->cv, cfg->kv_dtype == TRIMKV_DTYPE_BF16, h->Hq);
    if (s != TRIMKV_OK) {
        char keep[sizeof(g_err)];
        memcpy(keep, g_err, sizeof(keep));
        trimkv_destroy(h);
        memcpy(g_err, keep, sizeof(keep));
        return s;
    }
    *out = h;
    return TRIMKV_OK;
}

void trimkv_destroy(trimkv_t* h) {
    if (!h) return;
    cudaDeviceSynchronize();
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_append) cudaEventDestroy(h->ev_append);
    if (h->ev_side) cudaEventDestroy(h->ev_side);
    if (h->ev_done) cudaEventDestroy(h->ev_done);
    if (h->ev_sample) cudaEventDestroy(h->ev_sample);
    if (h->side2) cudaStreamDestroy(h->side2);
    if (h->side_hi) cudaStreamDestroy(h->side_hi);
    if (h->side) cudaStreamDestroy(h->side);
    if (h->fast) cudaStreamDestroy(h->fast);
    for (void* p : h->allocs) cudaFree(p);
    if (h->pool_stage) cudaFree(h->pool_stage);
    gate_tc_destroy(h->tc);
    prefill_tc_destroy(h->ptc);
    delete h;
}

trimkv_status trimkv_reset(trimkv_t* h) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    CUDA_TRY(cudaDeviceSynchronize());
    return init_cache_state(h);
}

trimkv_status trimkv_set_gate(trimkv_t* h, int layer, const float* W1, const float* b1, const float* W2, const float* b2) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (h->D <= 0) return fail(TRIMKV_E_STATE, "handle was created without a gate (hidden = 0)");
    if (layer < 0 || layer >= h->L || !W1 || !b1 || !W2 || !b2) return fail(TRIMKV_E_ARG, "bad layer or NULL weights");
    CUDA_TRY(cudaDeviceSynchronize());
    launch_gate_transpose(W1, h->W1T + (size_t)layer * h->dg * h->D, h->dg, h->D, 0);     // kept input-dimension major
    CUDA_TRY(cudaMemcpy(h->b1 + (size_t)layer * h->dg, b1, (size_t)h->dg * 4, cudaMemcpyDeviceToDevice));
    CUDA_TRY(cudaMemcpy(h->W2 + (size_t)layer * h->H * h->de * h->dg, W2, (size_t)h->H * h->de * h->dg * 4, cudaMemcpyDeviceToDevice));
    CUDA_TRY(cudaMemcpy(h->b2 + (size_t)layer * h->H * h->de, b2, (size_t)h->H * h->de * 4, cudaMemcpyDeviceToDevice));
    h->gate_set[layer] = 1;
    if (h->tc) launch_split_tf32(W1, h->W1hi + (size_t)layer * h->dg * h->D,
                                 h->W1lo + (size_t)layer * h->dg * h->D, (long long)h->dg * h->D, 0);
    if (h->shared_set) launch_gate_fold(gate_params(h), layer, 1, h->gv, h->gs0, 0);
    CUDA_TRY(cudaDeviceSynchronize());
    return TRIMKV_OK;
}

trimkv_status trimkv_set_shared_projection(trimkv_t* h, const float* w_g, float b_g) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (h->D <= 0) return fail(TRIMKV_E_STATE, "handle was created without a gate (hidden = 0)");
    if (!w_g) return fail(TRIMKV_E_ARG, "NULL w_g");
    CUDA_TRY(cudaDeviceSynchronize());
    CUDA_TRY(cudaMemcpy(h->w_g, w_g, (size_t)h->de * 4, cudaMemcpyDeviceToDevice));
    h->b_g = b_g;
    h->shared_set = true;
    for (int l = 0; l < h->L; ++l)
        if (h->gate_set[l]) launch_gate_fold(gate_params(h), l, 1, h->gv, h->gs0, 0);
    CUDA_TRY(cudaDeviceSynchronize());
    return TRIMKV_OK;
}

trimkv_status trimkv_gate(trimkv_t* h, int layer, int n_new, const float* x, float* beta, float* lambda, float* c,
                          void* stream) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (layer < 0 || layer >= h->L || n_new < 1 || !x || !aligned16(x)) return fail(TRIMKV_E_ARG, "bad layer, n_new or x (x must be 16-byte aligned)");
    if ((long long)h->B * n_new > h->rows_max) return fail(TRIMKV_E_ARG, "n_new exceeds max_chunk");
    if (trimkv_status s = gate_ready(h, layer, 1)) return s;
    gate_one_layer(h, x, layer, h->B * n_new, beta, lambda, c, (cudaStream_t)stream);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

trimkv_status trimkv_append(trimkv_t* h, int layer, int n_new, const float* x, const float* lambda, const float* c,
                            const void* k, const void* v, void* stream) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (layer < 0 || layer >= h->L) return fail(TRIMKV_E_ARG, "layer out of range");
    if (n_new < 1 || n_new > h->cfg.max_chunk) return fail(TRIMKV_E_ARG, "n_new must be in [1, max_chunk]");
    if (!k || !v || !aligned16(k) || !aligned16(v)) return fail(TRIMKV_E_ARG, "k and v must be non-NULL and 16-byte aligned");
    if (!x && !lambda) return fail(TRIMKV_E_ARG, "either x or lambda is required");
    if (h->tokens[layer] + n_new > h->max_pos) return fail(TRIMKV_E_UNSUPPORTED, "position limit %lld reached", h->max_pos);
    if (h->entries + (long long)n_new * h->H > capacity_entries(h))
        return fail(TRIMKV_E_STATE, "the cache holds %lld entries per sequence and has room for %lld: run trimkv_score_and_evict "
                    "before appending more (at most max_chunk tokens per layer between eviction rounds)", h->entries, capacity_entries(h));
    cudaStream_t st = (cudaStream_t)stream;
    const float* lam = lambda;
    const float* cc = c;
    if (x) {
        if (!aligned16(x)) return fail(TRIMKV_E_ARG, "x must be 16-byte aligned");
        if (trimkv_status s = gate_ready(h, layer, 1)) return s;
        if (h->prof.on) h->prof.mark(PH_GATE, 0, st);
        gate_one_layer(h, x, layer, h->B * n_new, nullptr, h->g_lam, h->g_c, st);
        if (h->prof.on) h->prof.mark(PH_GATE, 1, st);
        lam = h->g_lam;
        cc = h->g_c;
    }
    if (h->prof.on) h->prof.mark(PH_APPEND, 0, st);
    launch_append(h->cv, layer, 1, n_new, h->tokens[layer], lam, cc, h->cfg.horizon, k, v, APPEND_KV | APPEND_META, st);
    if (h->prof.on) h->prof.mark(PH_APPEND, 1, st);
    CUDA_TRY(cudaGetLastError());
    h->tokens[layer] += n_new;
    h->entries += (long long)n_new * h->H;
    return TRIMKV_OK;
}

trimkv_status trimkv_score_and_evict(trimkv_t* h, void* stream) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    return evict_impl(h, (cudaStream_t)stream);
}

trimkv_status trimkv_decode_attention(trimkv_t* h, int layer, const void* q, void* out, void* stream) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (layer < 0 || layer >= h->L || !q || !out || !aligned16(q) || !aligned16(out)) return fail(TRIMKV_E_ARG, "bad layer, q or out");
    return attention_impl(h, layer, 1, q, out, (cudaStream_t)stream);
}

trimkv_status trimkv_prefill_attention(trimkv_t* h, int layer, int n_new, const void* q, void* out, void* stream) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (layer < 0 || layer >= h->L || !q || !out || !aligned16(q) || !aligned16(out)) return fail(TRIMKV_E_ARG, "bad layer, q or out");
    if (n_new < 1 || n_new > h->cfg.max_chunk || n_new > h->tokens[layer])
        return fail(TRIMKV_E_ARG, "n_new must be the size of the chunk last appended to this layer");
    if (h->cfg.retention_bias) return fail(TRIMKV_E_UNSUPPORTED, "chunk attention supports the plain softmax only");
    PhaseMarker* pm = h->prof.on ? &h->prof : nullptr;
    cudaStream_t st = (cudaStream_t)stream;
    if (pm) pm->mark(PH_ATTN_MAIN, 0, st);
    launch_prefill_attention(h->cv, layer, n_new, h->Hq, h->cfg.kv_dtype == TRIMKV_DTYPE_BF16, h->ptc, q, out, st);
    if (pm) pm->mark(PH_ATTN_MAIN, 1, st);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

}  // extern "C"

namespace {

// Host-resident arguments of trimkv_decode_step_all_host.  x (or lambda) is copied to a staging buffer of the handle on the
// side stream, ahead of the gate.  K, V, q and the output are each touched exactly once by a kernel (K and V by the
// append, q and the output by the attention kernel): where the caller's buffers are pinned memory that the device can
// address (k_map .. out_map, null otherwise), those kernels can read and write them in place across the bus with no copy
// queued (q and the output always, K and V while they are small); otherwise they go through staging buffers, K, V, q
// ahead of the append, the output after the compaction.
struct HostArgs {
    const void *x, *lambda, *k, *v, *q;
    void* out;
    const void *k_map, *v_map, *q_map;
    void* out_map;
};

// The device's address of a pinned (page-locked, mapped) host buffer; null for any other memory.
void* device_view_of_host(const void* p) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    if (a.type != cudaMemoryTypeHost || a.devicePointer == nullptr) return nullptr;
    return aligned16(a.devicePointer) ? a.devicePointer : nullptr;
}

trimkv_status step_all_impl(trimkv* h, const float* x, const float* lambda, const void* k, const void* v, const void* q,
                            void* out, void* stream, const HostArgs* host) {
    if (h->shard) return fail(TRIMKV_E_STATE, "this handle holds a slice of the layers: use the per-layer calls and the trimkv_shard_* calls");
    const long long t = h->tokens[0];
    for (int l = 1; l < h->L; ++l)
        if (h->tokens[l] != t) return fail(TRIMKV_E_STATE, "layers hold different token counts");
    if (t + 1 > h->max_pos) return fail(TRIMKV_E_UNSUPPORTED, "position limit %lld reached", h->max_pos);
    if (h->entries + (long long)h->L * h->H > capacity_entries(h))
        return fail(TRIMKV_E_STATE, "the cache holds %lld entries per sequence and has room for %lld: run trimkv_score_and_evict first",
                    h->entries, capacity_entries(h));
    cudaStream_t st = (cudaStream_t)stream;
    if (x) {
        if (trimkv_status s = gate_ready(h, 0, h->L)) return s;
    }
    // Two internal streams, forked from and joined back to the caller's stream.  `fast`: K/V append -> attention ->
    // (wait for side) -> compaction.  `side`: gate -> retention terms of the new entries -> score + selection.
    // Attention never reads the retention terms and the selection never reads K/V, so the weight streaming of the gate
    // and the metadata scans run beside the attention kernel, which keeps the memory system busy throughout; compaction
    // moves K/V rows and therefore waits for both.  `fast` has the higher priority so that its few, large CTAs are
    // placed ahead of the many small ones of the side kernels.
    const bool two = h->overlap;                 // off: every phase back to back on the caller's stream
    // The side chain runs below the attention kernel's priority, unless the gate's weight stream is a sizeable part of
    // the step's traffic (above 15 % of the K/V bytes): a starved gate then ends together with the attention kernel and
    // the whole selection would follow it; at equal priority the gate finishes early and the selection hides under the
    // rest of the attention kernel (measured on the named workloads: stress_128k 0.499 -> 0.480 ms per step, qwen_vl_16k
    // 0.169 -> 0.155; llama8b_32k, where the gate is 7 % of the traffic, loses 9 us that way and keeps the low priority).
    const double kv_bytes = (double)(h->entries + (long long)h->L * h->H) * h->B * 2.0 * h->cv.row_bytes;
    const bool gate_heavy = x && (double)h->L * h->D * h->dg * 4.0 > 0.15 * kv_bytes;
    // A caller whose own stream already has the highest priority gets the fast chain on that stream: the two hand-offs
    // between its stream and `fast` (fork and join, a few microseconds each on the critical path) fall away.
    int st_prio = 0;
    const bool st_is_fast = two && st != nullptr &&
                            (st == h->fast || (cudaStreamGetPriority(st, &st_prio) == cudaSuccess && st_prio == h->prio_hi));
    cudaStream_t sd = two ? (gate_heavy ? h->side_hi : h->side) : st, fs = (two && !st_is_fast) ? h->fast : st;
    if (two) {
        CUDA_TRY(cudaEventRecord(h->ev_fork, st));
        if (!st_is_fast) CUDA_TRY(cudaStreamWaitEvent(fs, h->ev_fork, 0));
        CUDA_TRY(cudaStreamWaitEvent(sd, h->ev_fork, 0));
    }
    if (host) {
        const size_t kvb = (size_t)h->L * h->B * h->H * h->d * h->elt, qb = (size_t)h->L * h->B * h->Hq * h->d * h->elt;
        if (h->prof.on) h->prof.mark(PH_H2D, 0, fs);
        // K and V in place only while they are small: the append kernel's 16-byte reads cross the bus at about 12 GB/s
        // (measured: 1 MB in 85 us), a copy engine moves them at 50 GB/s but costs two more calls and a hand-over to the
        // kernel (1 MB: 34 us + 27 us).  q is read by a kernel that runs for the whole step, where the rate does not matter.
        if (host->k_map && host->v_map && 2 * kvb < ((size_t)512 << 10)) {
            k = host->k_map; v = host->v_map;
        } else {
            CUDA_TRY(cudaMemcpyAsync(h->st_k, host->k, kvb, cudaMemcpyHostToDevice, fs));
            CUDA_TRY(cudaMemcpyAsync(h->st_v, host->v, kvb, cudaMemcpyHostToDevice, fs));
        }
        if (host->q_map) q = host->q_map;
        else CUDA_TRY(cudaMemcpyAsync(h->st_q, host->q, qb, cudaMemcpyHostToDevice, fs));
        if (host->out_map) out = host->out_map;
        if (h->prof.on) h->prof.mark(PH_H2D, 1, fs);
        if (h->prof.on) h->prof.mark(PH_H2D_SIDE, 0, sd);
        if (host->x) CUDA_TRY(cudaMemcpyAsync(h->st_x, host->x, (size_t)h->L * h->B * h->D * 4, cudaMemcpyHostToDevice, sd));
        else CUDA_TRY(cudaMemcpyAsync(h->st_x, host->lambda, (size_t)h->L * h->B * h->H * 4, cudaMemcpyHostToDevice, sd));
        if (h->prof.on) h->prof.mark(PH_H2D_SIDE, 1, sd);
    }
    if (h->prof.on) h->prof.mark(PH_APPEND, 0, fs);
    launch_append(h->cv, 0, h->L, 1, t, nullptr, nullptr, h->cfg.horizon, k, v, APPEND_KV, fs);
    if (h->prof.on) h->prof.mark(PH_APPEND, 1, fs);
    if (two) CUDA_TRY(cudaEventRecord(h->ev_append, fs));
    for (int l = 0; l < h->L; ++l) h->tokens[l] += 1;
    h->entries += (long long)h->L * h->H;
    const long long kev = eviction_due(h);
    // Scheduling policy of the overlapped step.  When the K/V stream of the step is short (under ~1 GB, ~150 us), the
    // side chain (gate -> selection) is the critical path: the attention kernel then leaves one SM per sequence to the
    // selection's single-CTA kernels and the sampling runs early on a third stream.  With a long attention kernel the
    // side chain has slack: two SMs are enough for its single-CTA kernels to finish before the attention kernel does
    // (they cannot share an SM with a resident attention CTA and would otherwise run after it), and the third stream
    // is not used (measured: it costs the host-buffer entry point 30 us per step there).
    const bool side_critical = (double)h->entries * h->B * 2.0 * h->cv.row_bytes < 1.0e9;
    const int reserve = (two && kev > 0) ? std::min(h->B, side_critical ? 8 : 2) : 0;
    trimkv_status s = attention_impl(h, 0, h->L, q, out, fs, reserve);

    const float* lam = lambda;
    const float* cc = nullptr;
    if (x) {
        // the hidden layer streams its weights beside the K/V append; the output kernel then writes the retention terms
        // straight into the new entries' slots, which exist once the K/V half of the append has run
        if (h->prof.on) h->prof.mark(PH_GATE, 0, sd);
        launch_gate_hidden(gate_params(h), x, h->u, 0, h->L, h->B, sd);
        if (two) CUDA_TRY(cudaStreamWaitEvent(sd, h->ev_append, 0));
        launch_gate_out(gate_params(h), h->u, gate_chunks(h->D), 0, h->L, h->B, nullptr, nullptr, nullptr, sd, &h->cv);
        if (h->prof.on) h->prof.mark(PH_GATE, 1, sd);
    }
    // The selection's sample and rank bracket need only the page records of this step (final once the K/V half of the
    // append has run), not the new entries' retention terms: they run on a third stream beside the gate.
    const bool early_sample = two && kev > 0 && h->cfg.per_pool_budget == 0 && side_critical;
    if (early_sample) {
        CUDA_TRY(cudaStreamWaitEvent(h->side2, h->ev_append, 0));
        launch_select_cache_sample(h->cv, h->sb, h->tokens[0], h->entries, kev, 1, h->test_hooks & TRIMKV_TEST_DISTRUST_SAMPLE, h->side2);
        // ... and so does the filter pass over every entry but the newest of each pool: only those wait for the gate
        launch_select_cache_filter(h->cv, h->sb, h->tokens[0], 1, h->side2);
        CUDA_TRY(cudaEventRecord(h->ev_sample, h->side2));
    }
    if (!x) {
        if (two) CUDA_TRY(cudaStreamWaitEvent(sd, h->ev_append, 0));
        launch_append(h->cv, 0, h->L, 1, t, lam, cc, h->cfg.horizon, k, v, APPEND_META, sd);
    }
    if (early_sample) {
        CUDA_TRY(cudaStreamWaitEvent(sd, h->ev_sample, 0));
        if (h->prof.on) h->prof.mark(PH_SELECT, 0, sd);
        launch_select_cache_finish(h->cv, h->sb, h->tokens[0], kev, h->cursor, 1, sd);
        if (h->prof.on) h->prof.mark(PH_SELECT, 1, sd);
    } else if (kev > 0) {
        select_impl(h, kev, sd);
    }
    if (two) {
        CUDA_TRY(cudaEventRecord(h->ev_side, sd));
        CUDA_TRY(cudaStreamWaitEvent(fs, h->ev_side, 0));
    }
    if (s == TRIMKV_OK && kev > 0) s = compact_impl(h, fs);
    if (host) {
        if (h->prof.on) h->prof.mark(PH_D2H, 0, fs);
        if (!host->out_map)
            CUDA_TRY(cudaMemcpyAsync(host->out, out, (size_t)h->L * h->B * h->Hq * h->d * h->elt, cudaMemcpyDeviceToHost, fs));
        if (h->prof.on) h->prof.mark(PH_D2H, 1, fs);
    }
    if (two) {
        if (!st_is_fast) {
            CUDA_TRY(cudaEventRecord(h->ev_done, fs));
            CUDA_TRY(cudaStreamWaitEvent(st, h->ev_done, 0));
        }
    }
    if (s != TRIMKV_OK) return s;
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

}  // namespace

extern "C" {

trimkv_status trimkv_decode_step_all(trimkv_t* h, const float* x, const float* lambda, const void* k, const void* v,
                                     const void* q, void* out, void* stream) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (!k || !v || !q || !out || (!x && !lambda)) return fail(TRIMKV_E_ARG, "NULL argument");
    if (!aligned16(k) || !aligned16(v) || !aligned16(q) || !aligned16(out) || (x && !aligned16(x))) return fail(TRIMKV_E_ARG, "buffers must be 16-byte aligned");
    return step_all_impl(h, x, lambda, k, v, q, out, stream, nullptr);
}

trimkv_status trimkv_decode_step_all_host(trimkv_t* h, const float* x_host, const float* lambda_host, const void* k_host,
                                          const void* v_host, const void* q_host, void* out_host, void* stream) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (!k_host || !v_host || !q_host || !out_host || (!x_host && !lambda_host)) return fail(TRIMKV_E_ARG, "NULL argument");
    if (x_host && h->D <= 0) return fail(TRIMKV_E_STATE, "handle was created without a gate (hidden = 0)");
    HostArgs ha{x_host, lambda_host, k_host, v_host, q_host, out_host, nullptr, nullptr, nullptr, nullptr};
    ha.k_map = device_view_of_host(k_host);
    ha.v_map = device_view_of_host(v_host);
    ha.q_map = device_view_of_host(q_host);
    ha.out_map = device_view_of_host(out_host);
    return step_all_impl(h, x_host ? h->st_x : nullptr, x_host ? nullptr : h->st_x, h->st_k, h->st_v, h->st_q, h->st_out,
                         stream, &ha);
}

trimkv_status trimkv_get_lengths(trimkv_t* h, int32_t* out_host) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (!out_host) return fail(TRIMKV_E_ARG, "NULL output");
    CUDA_TRY(cudaDeviceSynchronize());
    CUDA_TRY(cudaMemcpy(out_host, h->cv.len, (size_t)h->B * h->L * h->H * sizeof(int32_t), cudaMemcpyDeviceToHost));
    return device_status(h);
}

trimkv_status trimkv_get_pool(trimkv_t* h, int seq, int layer, int head, int cap, int* n, int32_t* pos_host,
                              float* lambda_host, float* c_host, void* k_host, void* v_host) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (seq < 0 || seq >= h->B || layer < 0 || layer >= h->L || head < 0 || head >= h->H || !n || cap < 0)
        return fail(TRIMKV_E_ARG, "pool index out of range or NULL n");
    CUDA_TRY(cudaDeviceSynchronize());
    const long long pool = ((long long)seq * h->L + layer) * h->H + head;
    int32_t len = 0;
    CUDA_TRY(cudaMemcpy(&len, h->cv.len + pool, sizeof(len), cudaMemcpyDeviceToHost));
    *n = len;
    if (len > cap) return fail(TRIMKV_E_ARG, "pool holds %d entries, capacity %d", len, cap);
    if (len == 0) return device_status(h);
    const size_t rb = (size_t)h->d * h->elt;
    const size_t meta = ((size_t)len * 4 + 255) / 256 * 256;
    const size_t kvb = ((size_t)len * rb + 255) / 256 * 256;
    const size_t need = 3 * meta + 2 * kvb;
    if (need > h->pool_stage_bytes) {                 // the staging buffer only grows; most calls reuse it
        if (h->pool_stage) cudaFree(h->pool_stage);
        h->pool_stage = nullptr;
        h->pool_stage_bytes = 0;
        const size_t want = std::max(need, (size_t)1 << 20);
        CUDA_TRY(cudaMalloc((void**)&h->pool_stage, want));
        h->pool_stage_bytes = want;
    }
    char* tmp = h->pool_stage;
    int32_t* dpos = (int32_t*)tmp;
    float* dlam = (float*)(tmp + meta);
    float* dc = (float*)(tmp + 2 * meta);
    char* dk = tmp + 3 * meta;
    char* dv = dk + kvb;
    launch_gather_pool(h->cv, seq, layer, head, dpos, dlam, dc, k_host ? dk : nullptr, v_host ? dv : nullptr, len, 0);
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess && pos_host) e = cudaMemcpy(pos_host, dpos, (size_t)len * 4, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && lambda_host) e = cudaMemcpy(lambda_host, dlam, (size_t)len * 4, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && c_host) e = cudaMemcpy(c_host, dc, (size_t)len * 4, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && k_host) e = cudaMemcpy(k_host, dk, (size_t)len * rb, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && v_host) e = cudaMemcpy(v_host, dv, (size_t)len * rb, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail(TRIMKV_E_CUDA, "get_pool: %s", cudaGetErrorString(e));
    return device_status(h);
}

trimkv_status trimkv_import_pool(trimkv_t* h, int seq, int layer, int head, int n, const int32_t* pos_host,
                                 const float* lambda_host, const float* c_host, const void* k_host, const void* v_host) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (seq < 0 || seq >= h->B || layer < 0 || layer >= h->L || head < 0 || head >= h->H || n < 0)
        return fail(TRIMKV_E_ARG, "pool index out of range or negative n");
    if (n == 0) return TRIMKV_OK;
    if (!pos_host || !lambda_host || !c_host || !k_host || !v_host) return fail(TRIMKV_E_ARG, "NULL array");
    if ((long long)n > h->n_max) return fail(TRIMKV_E_NOMEM, "%d entries exceed the cache's capacity of %lld per sequence", n, h->n_max);
    for (int i = 0; i < n; ++i)
        if (pos_host[i] < 1 || pos_host[i] > h->max_pos) return fail(TRIMKV_E_ARG, "position %d out of range", pos_host[i]);
    CUDA_TRY(cudaDeviceSynchronize());
    const size_t rb = (size_t)h->d * h->elt;
    const size_t meta = ((size_t)n * 4 + 255) / 256 * 256, kvb = ((size_t)n * rb + 255) / 256 * 256;
    const size_t need = 3 * meta + 2 * kvb;
    if (need > h->pool_stage_bytes) {
        if (h->pool_stage) cudaFree(h->pool_stage);
        h->pool_stage = nullptr;
        h->pool_stage_bytes = 0;
        const size_t want = std::max(need, (size_t)1 << 20);
        CUDA_TRY(cudaMalloc((void**)&h->pool_stage, want));
        h->pool_stage_bytes = want;
    }
    char* tmp = h->pool_stage;
    CUDA_TRY(cudaMemcpy(tmp, pos_host, (size_t)n * 4, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(tmp + meta, lambda_host, (size_t)n * 4, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(tmp + 2 * meta, c_host, (size_t)n * 4, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(tmp + 3 * meta, k_host, (size_t)n * rb, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(tmp + 3 * meta + kvb, v_host, (size_t)n * rb, cudaMemcpyHostToDevice));
    launch_import_pool(h->cv, seq, layer, head, n, (const int32_t*)tmp, (const float*)(tmp + meta), (const float*)(tmp + 2 * meta),
                       tmp + 3 * meta, tmp + 3 * meta + kvb, 0);
    CUDA_TRY(cudaDeviceSynchronize());
    return device_status(h);
}

trimkv_status trimkv_import_finish(trimkv_t* h, int64_t tokens) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (tokens < 0 || tokens > h->max_pos) return fail(TRIMKV_E_ARG, "tokens out of range");
    CUDA_TRY(cudaDeviceSynchronize());
    const size_t LH = (size_t)h->L * h->H;
    std::vector<int32_t> len((size_t)h->B * LH);
    CUDA_TRY(cudaMemcpy(len.data(), h->cv.len, len.size() * sizeof(int32_t), cudaMemcpyDeviceToHost));
    long long first = -1, worst = 0;
    for (int b = 0; b < h->B; ++b) {
        long long e = 0;
        for (size_t p = 0; p < LH; ++p) e += len[(size_t)b * LH + p];
        if (first < 0) first = e;
        if (!h->shard && e != first)
            return fail(TRIMKV_E_STATE, "sequence %d holds %lld entries, sequence 0 holds %lld: all sequences advance in lock step", b, e, first);
        worst = std::max(worst, e);
    }
    if (worst > h->n_max) return fail(TRIMKV_E_NOMEM, "imported entries exceed the cache's capacity");
    h->entries = worst;
    std::fill(h->tokens.begin(), h->tokens.end(), (long long)tokens);
    return device_status(h);
}

trimkv_status trimkv_get_kept(trimkv_t* h, int seq, int layer, int head, int32_t* pos_out_host, int cap, int* n) {
    if (!pos_out_host) return fail(TRIMKV_E_ARG, "NULL output");
    trimkv_status s = trimkv_get_pool(h, seq, layer, head, cap, n, pos_out_host, nullptr, nullptr, nullptr, nullptr);
    if (s == TRIMKV_OK) std::sort(pos_out_host, pos_out_host + *n);
    return s;
}

trimkv_status trimkv_get_select_stats(trimkv_t* h, int64_t* out_host) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (!out_host) return fail(TRIMKV_E_ARG, "NULL output");
    CUDA_TRY(cudaDeviceSynchronize());
    CUDA_TRY(cudaMemcpy(out_host, h->sb.stats, (size_t)h->B * 4 * sizeof(long long), cudaMemcpyDeviceToHost));
    return device_status(h);
}

trimkv_status trimkv_check_invariants(trimkv_t* h) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    CUDA_TRY(cudaDeviceSynchronize());
    std::vector<unsigned> host((size_t)h->B + 1, 0u);
    unsigned* dev = nullptr;
    CUDA_TRY(cudaMalloc((void**)&dev, host.size() * sizeof(unsigned)));
    cudaError_t e = cudaMemset(dev, 0, host.size() * sizeof(unsigned));
    long long tokens = 0;
    for (int l = 0; l < h->L; ++l) tokens = std::max(tokens, h->tokens[l]);
    if (e == cudaSuccess) {
        launch_check(h->cv, tokens, dev, dev + 1, 0);
        e = cudaDeviceSynchronize();
    }
    if (e == cudaSuccess) e = cudaMemcpy(host.data(), dev, host.size() * sizeof(unsigned), cudaMemcpyDeviceToHost);
    std::vector<int32_t> free_count(h->B, 0);
    if (e == cudaSuccess) e = cudaMemcpy(free_count.data(), h->cv.free_count, (size_t)h->B * sizeof(int32_t), cudaMemcpyDeviceToHost);
    cudaFree(dev);
    if (e != cudaSuccess) return fail(TRIMKV_E_CUDA, "check_invariants: %s", cudaGetErrorString(e));
    unsigned viol = host[0];
    for (int b = 0; b < h->B; ++b)
        if ((long long)host[1 + b] + free_count[b] != h->P_seq) viol |= 32;      // pages neither owned nor free, or both
    if (viol) return fail(TRIMKV_E_STATE, "cache bookkeeping violated (rules 0x%x: 1 page id, 2 page record, 4 orphan page, 8 free "
                          "stack, 16 position, 32 page accounting, 64 NaN retention)", viol);
    return device_status(h);
}

trimkv_status trimkv_sync_status(trimkv_t* h) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    CUDA_TRY(cudaDeviceSynchronize());
    return device_status(h);
}

trimkv_status trimkv_profile(trimkv_t* h, int enable) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    CUDA_TRY(cudaDeviceSynchronize());
    h->prof.clear();
    h->prof.on = enable != 0;
    h->prof.only = enable == 2 ? (int)PH_ATTN_MAIN : -1;
    return TRIMKV_OK;
}

trimkv_status trimkv_set_horizon(trimkv_t* h, int horizon, void* stream) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (horizon < 0 || horizon > 64) return fail(TRIMKV_E_ARG, "horizon must be in [0, 64]");
    h->cfg.horizon = horizon;
    launch_rehorizon(h->cv, horizon, (cudaStream_t)stream);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

// ---- one sequence sharded by layer over ranks: the rank-local stages of an eviction round ----------------------------
static trimkv_status shard_ready(trimkv* h) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (!h->shard) return fail(TRIMKV_E_STATE, "the handle was not created with shard_total_layers > 0");
    for (int l = 1; l < h->L; ++l)
        if (h->tokens[l] != h->tokens[0]) return fail(TRIMKV_E_STATE, "layers hold different token counts");
    return TRIMKV_OK;
}

int32_t trimkv_shard_sample_cap(void) { return shard_sample_cap(); }

trimkv_status trimkv_shard_sample(trimkv_t* h, int64_t n_total, int64_t k_evict, uint64_t* keys_out, int32_t* counts_out,
                                  void* stream) {
    if (trimkv_status s = shard_ready(h)) return s;
    if (!keys_out || !counts_out || n_total < 1 || k_evict < 1 || k_evict > n_total) return fail(TRIMKV_E_ARG, "bad argument");
    launch_shard_sample(h->cv, h->sb, h->tokens[0], n_total, (u64*)keys_out, counts_out, (cudaStream_t)stream);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

trimkv_status trimkv_shard_bracket(trimkv_t* h, int world, const uint64_t* gathered_keys, const int32_t* gathered_counts,
                                   int64_t n_total, int64_t k_evict, void* stream) {
    if (trimkv_status s = shard_ready(h)) return s;
    if (world < 1 || !gathered_keys || !gathered_counts || n_total < 1 || k_evict < 1) return fail(TRIMKV_E_ARG, "bad argument");
    launch_shard_bracket(h->cv, h->sb, (const u64*)gathered_keys, gathered_counts, world, n_total, k_evict,
                         h->test_hooks & TRIMKV_TEST_DISTRUST_SAMPLE, (cudaStream_t)stream);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

trimkv_status trimkv_shard_filter(trimkv_t* h, int64_t* n_below_out, int32_t* cand_count_out, void* stream) {
    if (trimkv_status s = shard_ready(h)) return s;
    if (!n_below_out || !cand_count_out) return fail(TRIMKV_E_ARG, "NULL output");
    launch_shard_filter(h->cv, h->sb, h->tokens[0], (long long*)n_below_out, cand_count_out, (cudaStream_t)stream);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

trimkv_status trimkv_shard_candidates(trimkv_t* h, int64_t cap, void* cand_out, void* stream) {
    if (trimkv_status s = shard_ready(h)) return s;
    if (cap < 1 || !cand_out) return fail(TRIMKV_E_ARG, "bad argument");
    launch_shard_export_cands(h->cv, h->sb, cand_out, cap, (cudaStream_t)stream);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

trimkv_status trimkv_shard_resolve(trimkv_t* h, int world, int rank, int64_t cap, const void* gathered_cand,
                                   const int32_t* gathered_counts, const int64_t* n_below_global, int64_t k_evict,
                                   int32_t* resolved_out, void* stream) {
    if (trimkv_status s = shard_ready(h)) return s;
    if (world < 1 || rank < 0 || rank >= world || world > 255 || cap < 1 || !gathered_cand || !gathered_counts || !n_below_global ||
        !resolved_out)
        return fail(TRIMKV_E_ARG, "bad argument");
    launch_shard_resolve(h->cv, h->sb, gathered_cand, gathered_counts, (const long long*)n_below_global, world, rank, cap, k_evict,
                         h->cursor, resolved_out, (cudaStream_t)stream);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

trimkv_status trimkv_shard_hist(trimkv_t* h, const uint64_t* prefix, int top, uint32_t* hist_out, void* stream) {
    if (trimkv_status s = shard_ready(h)) return s;
    if (!prefix || !hist_out || top < 1 || top > 64) return fail(TRIMKV_E_ARG, "bad argument");
    launch_shard_hist(h->cv, h->sb, h->tokens[0], (const u64*)prefix, top, hist_out, (cudaStream_t)stream);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

trimkv_status trimkv_shard_digit(trimkv_t* h, const uint32_t* hist, uint64_t* prefix, int64_t* rank, int top, void* stream) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (!hist || !prefix || !rank || top < 1 || top > 64) return fail(TRIMKV_E_ARG, "bad argument");
    launch_shard_digit(h->B, hist, (u64*)prefix, (long long*)rank, top, (cudaStream_t)stream);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

trimkv_status trimkv_shard_mark(trimkv_t* h, const uint64_t* tau, void* stream) {
    if (trimkv_status s = shard_ready(h)) return s;
    if (!tau) return fail(TRIMKV_E_ARG, "NULL tau");
    launch_shard_mark(h->cv, h->sb, h->tokens[0], (const u64*)tau, h->cursor, (cudaStream_t)stream);
    CUDA_TRY(cudaGetLastError());
    return TRIMKV_OK;
}

trimkv_status trimkv_shard_compact(trimkv_t* h, int64_t* local_entries_out_host, void* stream) {
    if (trimkv_status s = shard_ready(h)) return s;
    cudaStream_t st = (cudaStream_t)stream;
    launch_compact(h->cv, h->hole, h->mover, h->cursor, h->e_max, h->e_max, st);
    CUDA_TRY(cudaGetLastError());
    CUDA_TRY(cudaStreamSynchronize(st));
    const size_t LH = (size_t)h->L * h->H;
    std::vector<int32_t> len((size_t)h->B * LH);
    CUDA_TRY(cudaMemcpy(len.data(), h->cv.len, len.size() * sizeof(int32_t), cudaMemcpyDeviceToHost));
    long long worst = 0;
    for (int b = 0; b < h->B; ++b) {
        long long e = 0;
        for (size_t p = 0; p < LH; ++p) e += len[(size_t)b * LH + p];
        if (local_entries_out_host) local_entries_out_host[b] = e;
        worst = std::max(worst, e);
    }
    h->entries = worst;              // sequences may keep different numbers here: the fullest one bounds the next append
    return device_status(h);
}

trimkv_status trimkv_set_test_hooks(trimkv_t* h, int flags) {
    if (flags & ~(TRIMKV_TEST_DISTRUST_SAMPLE | TRIMKV_TEST_ATTENTION_NO_COPY)) return fail(TRIMKV_E_ARG, "unknown test hook");
    CUDA_TRY(cudaDeviceSynchronize());
    if (h) h->test_hooks = flags;
    else tkv::g_test_hooks.store(flags, std::memory_order_relaxed);
    return TRIMKV_OK;
}

void* trimkv_step_stream(trimkv_t* h) { return h ? (void*)h->fast : nullptr; }

trimkv_status trimkv_set_overlap(trimkv_t* h, int enable) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    CUDA_TRY(cudaDeviceSynchronize());
    h->overlap = enable != 0;
    return TRIMKV_OK;
}

trimkv_status trimkv_profile_read(trimkv_t* h, double* ms_host, int64_t* count_host) {
    if (check_handle(h)) return TRIMKV_E_ARG;
    if (!ms_host || !count_host) return fail(TRIMKV_E_ARG, "NULL output");
    CUDA_TRY(cudaDeviceSynchronize());
    for (int i = 0; i < PH_COUNT; ++i) { ms_host[i] = 0.0; count_host[i] = 0; }
    for (auto& r : h->prof.recs) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, r.second.first, r.second.second) == cudaSuccess) {
            ms_host[r.first] += ms;
            count_host[r.first] += 1;
        }
    }
    h->prof.clear();
    return TRIMKV_OK;
}

const char* trimkv_last_error(void) { return g_err; }

int64_t trimkv_kernel_launches(void) { return (int64_t)tkv::g_launches.load(std::memory_order_relaxed); }

// ---- standalone selection ---------------------------------------------------------------------------
size_t trimkv_select_workspace_bytes(int64_t n) {
    if (n < 0) return 0;
    return flat_select_workspace_bytes(n);
}

trimkv_status trimkv_select_topk(const float* scores, int64_t n, int64_t k_keep, uint64_t* keep_bits, void* workspace,
                                 size_t workspace_bytes, int32_t* status_out, void* stream) {
    if (n < 0 || k_keep < 0 || n > 0xFFFFFFFFLL) return fail(TRIMKV_E_ARG, "n must be in [0, 2^32), k_keep >= 0");
    if (n == 0) return TRIMKV_OK;
    if (!scores || !keep_bits || !workspace || !aligned16(scores) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return fail(TRIMKV_E_ARG, "NULL or misaligned buffer (scores 16 B, workspace 256 B)");
    if (workspace_bytes < trimkv_select_workspace_bytes(n)) return fail(TRIMKV_E_ARG, "workspace too small");
    const cudaError_t e = launch_select_flat(scores, n, k_keep, (u64*)keep_bits, workspace, workspace_bytes, status_out,
                                             tkv::global_test_hooks() & TRIMKV_TEST_DISTRUST_SAMPLE, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(TRIMKV_E_CUDA, "selection launch failed: %s", cudaGetErrorString(e));
    return TRIMKV_OK;
}

}  // extern "C"
