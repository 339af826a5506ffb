// Internal declarations shared by the translation units of the trimkv library.
// Not part of the public ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "trimkv.h"

namespace tkv {

// ------------------------------------------------------------------ constants
constexpr int PAGE = 64;                 // entries per page
typedef unsigned long long u64;

// Per-sequence state of the cache's selection (device resident).
struct SelState {
    u64 cand_lo;       // candidate range [cand_lo, cand_hi]: keys below are evicted, above are kept
    u64 cand_hi;
    long long n_below; // number of keys < cand_lo
    int resolved;      // 1 once the threshold of this call is settled
    int passes;        // keys sampled in this call (reported in the statistics)
    unsigned int cand_count;   // candidates appended by the filter pass
    unsigned int sample_count; // keys drawn by the sampling pass of this call
};

struct Cand {          // one candidate of the exact resolution stage
    u64 key;
    u64 slot;          // slot index inside the sequence (page * 64 + offset) or flat index
};

// Order-preserving map of a float onto uint32 (smaller float -> smaller integer); -0 is folded onto +0.
__device__ __forceinline__ uint32_t orderable_key(float s) {
    s = __fadd_rn(s, 0.0f);
    uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Retention score in log space: S = c + age * lambda with one fp32 multiply and one fp32 add,
// each rounded to nearest even and never contracted into an FMA.
__device__ __forceinline__ float retention_score(float lam, float c, float age) {
    return __fadd_rn(c, __fmul_rn(age, lam));
}

// Eviction-order key: entries with the SMALLEST keys are evicted first.
//   high 32 bits: orderable score; low 32 bits: ~tie, where a larger tie (newer position, then higher
//   layer*H+head) is evicted first among equal scores.
__device__ __forceinline__ u64 make_key(float score, uint32_t tie) {
    return ((u64)orderable_key(score) << 32) | (u64)(~tie);
}

__device__ __forceinline__ u64 compose_key(uint32_t sc, uint32_t tie) { return ((u64)sc << 32) | (u64)(~tie); }

// Float-domain forms of 32-bit key comparisons, for any non-NaN x:
//   x <  key_float_lt(k)  iff  orderable_key(x) <  k        x <= key_float_le(k)  iff  orderable_key(x) <= k
// Keys at or below that of -inf / at or above that of +inf (NaN bit patterns) clamp to -inf / +inf.  No float has the
// key 0x7fffffff (it would be -0, which is folded onto +0): "<" there means "< -0", "<=" means "<= the key before it".
__device__ __forceinline__ float key_float_lt(uint32_t key) {
    if (key <= 0x007fffffu) return __uint_as_float(0xff800000u);         // at or below key(-inf)
    if (key >= 0xff800000u) return __uint_as_float(0x7f800000u);         // at or above key(+inf)
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}
__device__ __forceinline__ float key_float_le(uint32_t key) { return key_float_lt(key == 0x7fffffffu ? 0x7ffffffeu : key); }

__device__ __forceinline__ uint32_t mix32(uint32_t x) {   // integer finaliser: spreads slot indices over 32 bits
    x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
    return x;
}

// c = ln sum_{k<horizon} exp(k * lambda): the beta-only factor of the retention score (horizon 0 = infinite).
__device__ __forceinline__ float horizon_term_f32(float lam, int horizon) {
    if (horizon == 1) return 0.0f;
    if (horizon == 0) return -logf(-expm1f(lam));
    float acc = 1.0f;
    for (int k = 1; k < horizon; ++k) acc += expf((float)k * lam);
    return logf(acc);
}

// ------------------------------------------------------------------ cache geometry
// KV storage: kv[b][page][2][PAGE][row_bytes]; part 0 = K rows, part 1 = V rows of the page.
// bf16 rows whose length is a multiple of 128 bytes are stored with their 16-byte chunks permuted
// inside each 128-byte group: physical chunk = logical chunk ^ (slot_in_page & 7).  A linear bulk copy of
// a page to shared memory is then bank-conflict free for 8-row matrix loads.
struct CacheView {
    char* kv;
    float* lam;
    float* c;
    int32_t* pos;
    int4* owner;           // [B][P_seq] {pool_local or -1, logical page index, live entries in the page, 0}
    int32_t* block_table;  // [B*L*H][maxpp]
    int32_t* len;          // [B*L*H]
    int32_t* free_stack;   // [B][P_seq]
    int32_t* free_count;   // [B]
    u64* evict_mask;       // [B][P_seq]
    int32_t* err;          // latched device status
    int32_t* append_failed; // [B*L*H] 1 if the bookkeeping half of the pool's last append failed (no page), else 0
    long long P_seq;       // pages per sequence
    long long maxpp;       // block-table row length
    int B, L, H, d;
    int row_bytes;         // d * sizeof(element)
    int swizzle;           // 1 if rows are chunk-permuted
    int pool_bits;         // bits that hold layer*H+head in the tie-break word
    int pool_offset;       // added to the local layer*H+head in that word: > 0 when the handle holds a slice of a
                           // sequence's layers (the pool id of the tie-break is the id within the whole model)
};

__device__ __forceinline__ size_t kv_row_offset(const CacheView& cv, int b, long long page, int part, int off) {
    return ((((size_t)b * cv.P_seq + page) * 2 + part) * PAGE + off) * (size_t)cv.row_bytes;
}
__device__ __forceinline__ int phys_chunk(const CacheView& cv, int chunk, int off) {
    return cv.swizzle ? (chunk ^ (off & 7)) : chunk;
}

__device__ __forceinline__ void latch_error(int32_t* err, int code) {
    if (err) atomicCAS(err, 0, code);
}

// ------------------------------------------------------------------ launchers (host)
struct GateParams {
    const float* W1T; // [L][D][dg]  first layer, transposed (input dimension major)
    const float* b1;  // [L][dg]
    const float* W2;  // [L][H][de][dg]
    const float* b2;  // [L][H][de]
    const float* w_g; // [de]
    const float* v;   // [L][H][dg]  second layer folded with the shared readout: W2^T w_g
    const float* s0;  // [L][H]      w_g . b2 + b_g
    float b_g;
    int D, dg, de, H, horizon;
};

// Recomputes v and s0 of layers [layer0, layer0 + nlayers) from W2, b2, w_g, b_g.
void launch_gate_fold(const GateParams& gp, int layer0, int nlayers, float* v, float* s0, cudaStream_t st);

// Number of input-dimension chunks the hidden layer is split into; the scratch of launch_gate holds
// gate_chunks(D) * rows * dg floats per layer.
int gate_chunks(int D);

// W1T[d][j] = W1[j][d] for one layer's first-layer weights W1 [dg][D].
void launch_gate_transpose(const float* W1, float* W1T, int dg, int D, cudaStream_t st);

// rows_per_layer rows of x per layer, layers [layer0, layer0 + nlayers).
void launch_gate(const GateParams& gp, const float* x, float* z_scratch, int layer0, int nlayers, int rows_per_layer,
                 float* beta, float* lam, float* c, cudaStream_t st);

constexpr int APPEND_KV = 1, APPEND_META = 2;   // halves of an append; see append_kernel
constexpr int APPEND_ROWS_ELSEWHERE = 4;        // (internal to launch_append: the K/V rows are copied by a second kernel)
void launch_append(const CacheView& cv, int layer0, int nlayers, int n_new, long long pos0, const float* lam,
                   const float* c, int horizon, const void* k, const void* v, int mode, cudaStream_t st);

// Second half of the gate alone: z_scratch holds nchunk partial pre-activations per (row, hidden unit).
// to_cache != null (decode step, one row per sequence): lambda and c are also written to the newest entry of every pool.
void launch_gate_out(const GateParams& gp, const float* z_scratch, int nchunk, int layer0, int nlayers, int rows_per_layer,
                     float* beta, float* lam, float* c, cudaStream_t st, const CacheView* to_cache = nullptr);
// First half of the gate alone (the hidden layer's partial pre-activations into z_scratch).
void launch_gate_hidden(const GateParams& gp, const float* x, float* z_scratch, int layer0, int nlayers, int rows_per_layer,
                        cudaStream_t st);

// Tensor-core (tcgen05, 3xTF32) form of the hidden layer for calls with many rows of one layer.
struct GateTcState;
bool gate_tc_supported(int D, int dg);
GateTcState* gate_tc_create(float* xhi, float* xlo, long long rows_alloc, float* whi, float* wlo, int L, int dg, int D);
void gate_tc_destroy(GateTcState* s);
void launch_split_tf32(const float* in, float* hi, float* lo, long long n, cudaStream_t st);
void launch_gate_gemm_tc(GateTcState* s, const float* x, int R, int layer, float* z, int32_t* err, cudaStream_t st);

struct SelectBuffers {
    SelState* sel;        // [B]
    Cand* cand;           // [B][cand_cap]
    long long cand_cap;
    long long* stats;     // [B][4]
    u64* sample;          // [B][4096] sampled keys (cache path)
};

// compact_cursor [B]: zeroed by the selection for the compaction that follows.
void launch_select_cache(const CacheView& cv, const SelectBuffers& sb, long long t, long long n_total, long long k_evict,
                         int32_t* compact_cursor, int distrust_sample, cudaStream_t st);
// The same selection in two parts, for callers that run the sampling beside other work: the sample and its rank bracket
// (skip_newest: entries at the tail of every pool whose retention terms are not written yet), then filter and resolution.
void launch_select_cache_sample(const CacheView& cv, const SelectBuffers& sb, long long t, long long n_total,
                                long long k_evict, int skip_newest, int distrust_sample, cudaStream_t st);
void launch_select_cache_rest(const CacheView& cv, const SelectBuffers& sb, long long t, long long k_evict,
                              int32_t* compact_cursor, cudaStream_t st);
// ... or in three parts: the filter pass may leave out the newest entry of every pool as well (skip_newest) and run beside
// the gate; the finish then classifies those entries (newest_left_out) and ranks the candidates.
void launch_select_cache_filter(const CacheView& cv, const SelectBuffers& sb, long long t, int skip_newest, cudaStream_t st);
void launch_select_cache_finish(const CacheView& cv, const SelectBuffers& sb, long long t, long long k_evict,
                                int32_t* compact_cursor, int newest_left_out, cudaStream_t st);
// Rank-local stages of the selection of a sequence whose layers are sharded over ranks (see select.cu).
int shard_sample_cap();
void launch_shard_sample(const CacheView& cv, const SelectBuffers& sb, long long t, long long n_total, u64* keys_out,
                         int32_t* counts_out, cudaStream_t st);
void launch_shard_export_sample(const CacheView& cv, const SelectBuffers& sb, u64* keys_out, int32_t* counts_out, cudaStream_t st);
void launch_shard_bracket(const CacheView& cv, const SelectBuffers& sb, const u64* gkeys, const int32_t* gcounts, int world,
                          long long n_total, long long k_evict, int distrust, cudaStream_t st);
void launch_shard_filter(const CacheView& cv, const SelectBuffers& sb, long long t, long long* n_below_out,
                         int32_t* cand_count_out, cudaStream_t st);
void launch_shard_export_cands(const CacheView& cv, const SelectBuffers& sb, void* out, long long cap, cudaStream_t st);
void launch_shard_resolve(const CacheView& cv, const SelectBuffers& sb, const void* gcand, const int32_t* gcounts,
                          const long long* n_below_global, int world, int rank, long long cap, long long k_evict,
                          int32_t* compact_cursor, int32_t* resolved_out, cudaStream_t st);
void launch_shard_hist(const CacheView& cv, const SelectBuffers& sb, long long t, const u64* prefix, int top, unsigned* hist_out,
                       cudaStream_t st);
void launch_shard_digit(int B, const unsigned* hist, u64* prefix, long long* rank, int top, cudaStream_t st);
void launch_shard_mark(const CacheView& cv, const SelectBuffers& sb, long long t, const u64* tau, int32_t* compact_cursor,
                       cudaStream_t st);
// Fixed per-pool budget: every pool keeps its keep_per_pool best entries (masks as for launch_select_cache).
void launch_select_pools(const CacheView& cv, long long t, int keep_per_pool, int32_t* compact_cursor, cudaStream_t st);
// evictions_per_seq: how many entries the selection just flagged per sequence (sizes the CTAs).
void launch_compact(const CacheView& cv, int32_t* hole, int32_t* mover, int32_t* cursor, long long e_max,
                    long long evictions_per_seq, cudaStream_t st);

// Standalone selection over a flat score array (select_flat.cu).  Workspace layout: 1 KB of state and counters, the
// candidate histogram (in several copies; the exact fallback's histograms reuse the space), the keys ranked exactly,
// then the candidate list.
constexpr int FLAT_HIST_BINS = 4096, FLAT_HIST_REPLICAS = 3, FLAT_X_BINS = 2048, FLAT_X_PASSES = 6, FLAT_CAND2_CAP = 16384;
constexpr size_t FLAT_FIXED_BYTES = 1024 + (size_t)FLAT_HIST_REPLICAS * FLAT_HIST_BINS * 4 + (size_t)FLAT_CAND2_CAP * 8;
constexpr long long flat_select_cand_cap(long long n) { return n / 16 + 16384; }   // keys inside the sampled bracket, with margin
constexpr size_t flat_select_workspace_bytes(long long n) {
    return FLAT_FIXED_BYTES + (size_t)flat_select_cand_cap(n) * 8 + 256;
}
// Keeps the k_keep largest of n scores: keep_bits words are written in full.  status (may be null) is set by the kernels.
cudaError_t launch_select_flat(const float* scores, long long n, long long k_keep, u64* keep_bits, void* workspace,
                               size_t workspace_bytes, int32_t* status, int distrust, cudaStream_t stream);
void launch_select_state_init(SelState* sel, int B, cudaStream_t st);

struct AttnBuffers {
    int32_t* pool_done;    // [pools] items of the pool finished so far in the running call; zero between calls
    int32_t* sched;        // [2] {items handed out beyond the first per warp, warps finished}; zero between calls
    float* part_o;         // [max_items][g][d]
    float* part_ml;        // [max_items][g][2]
    long long max_items;
};

// Optional per-phase timing: mark(phase, 0) before and mark(phase, 1) after a phase's launches.
enum Phase { PH_GATE = 0, PH_APPEND = 1, PH_H2D = 2, PH_ATTN_MAIN = 3, PH_D2H = 4, PH_SELECT = 5,
             PH_COMPACT = 6, PH_H2D_SIDE = 7, PH_COUNT = 8 };
struct PhaseMarker {
    virtual void mark(int phase, int end, cudaStream_t st) = 0;
    virtual ~PhaseMarker() {}
};

// reserve_sms: SMs the persistent kernel leaves to kernels running beside it (0 when it runs alone).
// retention_bias != 0: retention-gated weights beta_i^(t_now - i) e^{z_i} instead of the plain softmax.
void launch_attention(const CacheView& cv, const AttnBuffers& ab, int layer0, int nlayers, int Hq, int is_bf16,
                      long long tiles_estimate, long long tiles_upper, int retention_bias, long long t_now, int reserve_sms,
                      bool test_no_copy, const void* q, void* out, cudaStream_t st, PhaseMarker* pm);

// Causal attention of the chunk of n_new tokens just appended to `layer`; q, out: [B, n_new, Hq, d].
// tc: state of the tensor-core (tcgen05) form, or null; used when the chunk is large enough to fill its tiles.
struct PrefillTcState;
bool prefill_tc_supported(const CacheView& cv, int is_bf16, int Hq);
PrefillTcState* prefill_tc_create(const CacheView& cv, int is_bf16, int Hq);
void prefill_tc_destroy(PrefillTcState* s);
bool prefill_tc_wanted(const CacheView& cv, int n_new, int Hq);
void launch_prefill_attention_tc(const PrefillTcState* s, const CacheView& cv, int layer, int n_new, int Hq, const void* q,
                                 void* out, cudaStream_t st);
void launch_prefill_attention(const CacheView& cv, int layer, int n_new, int Hq, int is_bf16, const PrefillTcState* tc,
                              const void* q, void* out, cudaStream_t st);

// Rewrites c of every stored entry from its lambda for a new horizon.
void launch_rehorizon(const CacheView& cv, int horizon, cudaStream_t st);

// Fills an empty pool from dense device arrays (pos, lambda, c [n]; k, v [n, d] in the KV dtype).
void launch_import_pool(const CacheView& cv, int seq, int layer, int head, int n, const int32_t* pos, const float* lam,
                        const float* c, const void* k, const void* v, cudaStream_t st);

// Bookkeeping self-check (see check_kernel): viol [1] and owned [B] must be zero on entry.
void launch_check(const CacheView& cv, long long tokens, unsigned* viol, unsigned* owned, cudaStream_t st);

void launch_gather_pool(const CacheView& cv, int seq, int layer, int head, int32_t* pos, float* lam, float* c, void* k,
                        void* v, int n, cudaStream_t st);

void count_launch(int n = 1);

// ---- programmatic dependent launch: a chain of short kernels in one stream overlaps each kernel's launch latency and
// prologue with the tail of the kernel before it.  A kernel launched by launch_dependent() may start while its predecessor
// in the stream still runs; it must call grid_dependency_wait() before it touches anything a predecessor reads or writes
// (the wait returns once every earlier grid of the stream has completed and its writes are visible).  A predecessor lets
// the next kernel's CTAs be placed by calling grid_dependents_may_launch() in every CTA (or by exiting); that call says
// nothing about memory.  Both are no-ops in a kernel launched the ordinary way.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependents_may_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem_bytes, cudaStream_t stream,
                                    Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// TRIMKV_TEST_* switches of the handle-less calls.
int global_test_hooks();

// True the first time it is called for (slot, current device): kernels with more than 48 KB of dynamic shared memory
// need their opt-in attribute set once per device, not once per process.
bool first_use_on_device(int slot);

// Sets the calling thread's message returned by trimkv_last_error (printf format).
void set_last_error(const char* fmt, ...);

}  // namespace tkv
