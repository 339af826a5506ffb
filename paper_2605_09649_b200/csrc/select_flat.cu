// Standalone global selection over a flat array of fp32 scores (Sec. 4.2's ranking alone): keep the k largest of n
// scores, ties keeping the lower index.  Every score maps to the unique 64-bit key  orderable(score) || ~index, whose
// integer order is the eviction order, so the result equals a full sort and no float is compared after key construction.
//
// One pass over the scores:
//   0. flat_gather_kernel: a stratified sample of the scores (one hashed position per stratum), as keys.
//   1. flat_bracket_kernel (one CTA): ranks the sample and
//      brackets the k-th smallest key between two sample keys, several standard deviations of the sample rank apart;
//      the bracket's midpoint (`mid`) serves as a first estimate of the threshold.  (1b, largest arrays only:
//      flat_refine_kernel narrows the bracket with a 32 times larger sample gathered by many CTAs.)
//   2. flat_main_kernel (whole GPU, reads the scores once): writes the keep bits against `mid`, counts the keys below
//      the bracket, appends the keys inside it to a candidate list and bins them (shared-memory histogram of 4096 equal
//      bins over the bracket); the last CTA finds the bin of the k-th key: a fine bracket with a few thousand keys.
//   3. flat_cand_kernel (reads the candidate list, a few percent of n): flips the keep bits of candidates on the wrong
//      side of `mid`, collects the keys of the fine bracket; its last CTA ranks those exactly (radix select on the
//      differing bits) and settles their bits.
//   4. flat_exact_kernel (cooperative launch; returns at once unless needed): the exact fallback.  If the fine bracket
//      was too crowded, an exact radix select over the candidate list; if the sampled bracket missed the k-th key or the
//      candidate list overflowed, an exact radix select over all scores.  The result never depends on the sample.
#include <algorithm>

#include "async_copy.cuh"
#include "trimkv_internal.cuh"

namespace tkv {

namespace {

constexpr int FB = FLAT_HIST_BINS;          // bins of the candidate histogram
constexpr int HREP = FLAT_HIST_REPLICAS;    // copies of it in global memory: CTAs merge into copy (CTA % HREP), which keeps
                                            // the number of atomics that meet on one address small
constexpr int FB_BITS = 12;
constexpr int XB_BITS = 11, XB = FLAT_X_BINS;    // digit of the exact fallback's radix select
constexpr int X_PASSES = FLAT_X_PASSES;     // 64 bits in digits of 11 (the last one 9)
constexpr int CAND2_CAP = FLAT_CAND2_CAP;   // keys the last CTA of flat_cand_kernel ranks exactly
static_assert(FB == 1 << FB_BITS && XB == 1 << XB_BITS && X_PASSES * XB_BITS >= 64, "digit layout");
constexpr int MODE_DONE = 0, MODE_EXACT_LIST = 1, MODE_EXACT_ALL = 2;
constexpr unsigned BARRIER_SPIN_LIMIT = 1u << 22;

// Selection state, at the start of the workspace (256 bytes reserved).
struct FlatState {
    u64 lo, hi, mid;                 // bracket [lo, hi] of the k-th smallest key; first estimate of the threshold
    u64 bin_base;                    // histogram: bin(key) = clamp((key - bin_base) >> shift, 0, FB - 1)
    u64 lo2, hi2;                    // fine bracket: the histogram bin of the k-th key
    unsigned long long n_below;      // keys below lo (counted by the main pass)
    long long r2;                    // rank of the k-th key inside [lo2, hi2], 1-based
    long long r1;                    // rank of the k-th key inside [lo, hi], 1-based (exact fallback over the list)
    unsigned cand_count, cand2_count;
    int shift;                       // histogram bin width = 2^shift keys
    int mode;                        // MODE_*
    unsigned done_main, done_cand;   // CTA tickets
    unsigned bar_count, bar_abort;   // grid barrier of the exact fallback
    int ns;                          // keys sampled
    unsigned done_refine;            // CTA ticket of the refinement round
    unsigned long long below_s;      // refinement round: its sample keys below lo
    u64 e_hi;                        // upper end of the histogram's range (= hi unless hi is open)
    // float-domain forms of the bracket for the main pass
    float lo_f, hi_f;                // x < lo_f: score word below lo's; x > hi_f: above hi's
    float mid_lt;                    // x < mid_lt  iff  score word < mid's
    float ctr, hw;                   // finite bracket: score word within [lo's, hi's] implies !(|x - ctr| > hw)
    int finite;                      // form of the main pass's tests.  0: two compares per score with lo_f and hi_f;
                                     // 1: both ends finite: one subtraction + one compare (ctr, hw); 2: as 1 with hw and
                                     // |mid_lt| at least 2^-100: the arithmetic form is exact (see flat_main_body)
};
static_assert(sizeof(FlatState) <= 256, "FlatState must fit the reserved header");

__device__ __forceinline__ u64 flat_key(float x, uint32_t idx) { return compose_key(orderable_key(x), idx); }
__device__ __forceinline__ int flat_bin(u64 key, u64 base, int shift) {
    if (key < base) return 0;
    const u64 b = (key - base) >> shift;
    return b > (u64)(FB - 1) ? FB - 1 : (int)b;
}

// Publishes a bracket [lo, hi] (thread 0 of whichever kernel determined it): the histogram range [e_lo, e_hi] (the
// bracket itself, or a finite stand-in for an open end), the first estimate `mid` of the threshold, and the float-domain
// forms the main pass compares scores with.
__device__ void flat_publish(FlatState* st, u64 lo, u64 hi, u64 e_lo, u64 e_hi, u64 mid) {
    const u64 span = e_hi - e_lo;
    const int bits = span ? 64 - __clzll((long long)span) : 0;
    if (mid < lo) mid = lo;
    if (mid > hi) mid = hi;
    st->lo = lo; st->hi = hi; st->mid = mid;
    st->bin_base = e_lo;
    st->e_hi = e_hi;
    st->shift = bits > FB_BITS ? bits - FB_BITS : 0;
    const float lo_f = key_float_lt((uint32_t)(lo >> 32)), hi_f = key_float_le((uint32_t)(hi >> 32));
    st->lo_f = lo_f; st->hi_f = hi_f;
    st->mid_lt = key_float_lt((uint32_t)(mid >> 32));
    const bool fin = isfinite(lo_f) && isfinite(hi_f) && lo_f <= hi_f;
    float ctr = 0.f, hw = 0.f;
    if (fin) {
        ctr = (float)(0.5 * (double)lo_f + 0.5 * (double)hi_f);
        const double h = fmax((double)ctr - (double)lo_f, (double)hi_f - (double)ctr);
        hw = (float)(h * (1.0 + 1e-6));
        hw = nextafterf(nextafterf(hw, INFINITY), INFINITY);   // rounding of x - ctr and of hw itself: stay on the safe side
    }
    const float mid_lt = st->mid_lt;
    const bool fin1 = fin && isfinite(hw);
    const bool mid_ok = isfinite(mid_lt) && fabsf(mid_lt) >= 0x1p-100f;
    int form = fin1 ? 1 : 0;
    if (fin1 && mid_ok && hw >= 0x1p-100f) form = 2;
    st->ctr = ctr; st->hw = hw;
    st->finite = form;
}

// ------------------------------------------------------------------ 0. sample gather
// One thread per sample: a hashed position inside its stratum, the score there, its key.  Spread over many SMs because
// the reads are scattered over the whole array (one CTA needs 8 us for 8192 of them); the same launch clears what the later
// kernels accumulate into.  cap: the most samples (4096 or 8192); the strata are as wide as that needs.
__global__ void __launch_bounds__(256)
flat_gather_kernel(const float* __restrict__ s, long long n, int cap, u64* __restrict__ samples, uint32_t* __restrict__ hist,
                   int32_t* __restrict__ status) {
    grid_dependents_may_launch();
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    for (int i = j; i < FB * (HREP + 1); i += gridDim.x * blockDim.x) hist[i] = 0u;   // + the refinement round's histogram
    if (j == 0 && status) *status = 0;
    const long long stride = (n + cap - 1) / cap;          // stratum width; 1 when every score is sampled
    const int ns = (int)((n + stride - 1) / stride);
    if (j >= ns) return;
    const long long base = (long long)j * stride;
    const uint32_t width = (uint32_t)min(stride, n - base);
    const uint32_t idx = (uint32_t)base + (width > 1u ? mix32((uint32_t)j * 0x9E3779B1u + 0x7F4A7C15u) % width : 0u);
    samples[j] = flat_key(__ldg(s + idx), idx);
}

// ------------------------------------------------------------------ 1. sample bracket
// PER keys per thread in registers (1024 threads): 4096 or 16384 samples.  The lower and the upper end of the bracket
// are found by ONE radix descent over the sample: while the two ranks fall into the same bin one histogram serves both;
// after they part each key still matches at most one of the two prefixes, so a sweep costs the same.
template <int PER>
__global__ void __launch_bounds__(1024)
flat_bracket_kernel(const u64* __restrict__ samples, long long n, long long k_evict, FlatState* __restrict__ st,
                    long long* __restrict__ stats, float sigmas, int distrust) {
    constexpr int DB = 11, NBIN = 1 << DB, CAP = 1024 * PER;
    __shared__ unsigned hAB[NBIN];          // low half-word: keys under the lower end's prefix; high: the upper end's
    __shared__ unsigned wtot[32];
    __shared__ u64 s_or[32], s_and[32], s_min[32], s_max[32];
    __shared__ int s_digit[2];
    __shared__ long long s_r[2];
    __shared__ unsigned s_cnt[2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    grid_dependents_may_launch();
    grid_dependency_wait();                                // the samples come from the kernel before

    const long long stride = (n + CAP - 1) / CAP;          // stratum width; 1 when every score is sampled
    const int ns = (int)((n + stride - 1) / stride);
    u64 key[PER];
    u64 vor = 0ull, vand = ~0ull, kmin = ~0ull, kmax = 0ull;
#pragma unroll
    for (int i = 0; i < PER; ++i) key[i] = tid + i * 1024 < ns ? samples[tid + i * 1024] : ~0ull;   // all loads in flight at once
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        if (tid + i * 1024 < ns) {
            vor |= key[i];
            vand &= key[i];
            kmin = key[i] < kmin ? key[i] : kmin;
            kmax = key[i] > kmax ? key[i] : kmax;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        vor |= __shfl_xor_sync(0xffffffffu, vor, o);
        vand &= __shfl_xor_sync(0xffffffffu, vand, o);
        const u64 a = __shfl_xor_sync(0xffffffffu, kmin, o), b = __shfl_xor_sync(0xffffffffu, kmax, o);
        kmin = a < kmin ? a : kmin;
        kmax = b > kmax ? b : kmax;
    }
    if (lane == 0) { s_or[warp] = vor; s_and[warp] = vand; s_min[warp] = kmin; s_max[warp] = kmax; }
    __syncthreads();
    if (warp == 0) {                                       // one warp combines the 32 partial results and publishes them
        vor = s_or[lane]; vand = s_and[lane]; kmin = s_min[lane]; kmax = s_max[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            vor |= __shfl_xor_sync(0xffffffffu, vor, o);
            vand &= __shfl_xor_sync(0xffffffffu, vand, o);
            const u64 a = __shfl_xor_sync(0xffffffffu, kmin, o), b = __shfl_xor_sync(0xffffffffu, kmax, o);
            kmin = a < kmin ? a : kmin;
            kmax = b > kmax ? b : kmax;
        }
        if (lane == 0) { s_or[0] = vor; s_and[0] = vand; s_min[0] = kmin; s_max[0] = kmax; }
    }
    __syncthreads();
    vor = s_or[0]; vand = s_and[0]; kmin = s_min[0]; kmax = s_max[0];
    const u64 diff = vor ^ vand;
    const int top0 = diff ? 64 - __clzll((long long)diff) : 0;   // low bits in which the sample keys differ

    // bins of rank rA among the low half-word counts and of rank rB among the high ones (or the low ones too, while
    // both ends follow the same prefix), from one block-wide scan of the packed histogram (sample size < 65536)
    auto find2 = [&](long long rA, bool wantA, long long rB, bool wantB, bool split) {
        const unsigned h0 = hAB[2 * tid], h1 = hAB[2 * tid + 1];
        unsigned incl = h0 + h1;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) wtot[warp] = incl;
        __syncthreads();
        unsigned off = 0;
        for (int w = 0; w < warp; ++w) off += wtot[w];
        const unsigned excl = off + incl - (h0 + h1);
        auto pick = [&](long long r, unsigned sh16, int which) {
            const long long e = (excl >> sh16) & 0xffffu, a = (h0 >> sh16) & 0xffffu, b = (h1 >> sh16) & 0xffffu;
            if (r > e && r <= e + a) { s_digit[which] = 2 * tid; s_r[which] = r - e; s_cnt[which] = (unsigned)a; }
            else if (r > e + a && r <= e + a + b) { s_digit[which] = 2 * tid + 1; s_r[which] = r - e - a; s_cnt[which] = (unsigned)b; }
        };
        if (wantA) pick(rA, 0u, 0);
        if (wantB) pick(rB, split ? 16u : 0u, 1);
        __syncthreads();
    };

    u64 lo = 0ull, hi = ~0ull;
    if (distrust) {
        lo = hi = ~0ull;                    // testing aid: a bracket that cannot hold the k-th key
    } else {
        long long rA, rB;                   // sample ranks (1-based) whose keys bound the bracket
        if (stride == 1) {                  // every key was sampled: the k-th smallest is known exactly
            rA = rB = k_evict;
        } else {
            const float q = (float)((double)k_evict / (double)n);
            const float mu = q * (float)ns;                            // expected sample rank of the k-th key
            const float dev = sigmas * sqrtf(mu * (1.0f - q)) + 8.0f;  // binomial bound (strata only narrow it), with slack
            rA = (long long)floorf(mu - dev);
            rB = (long long)ceilf(mu + dev) + 1;
        }
        const bool openA = rA < 1, openB = rB > ns;  // an end outside the sample stays open (0 / ~0)
        bool actA = !openA, actB = !openB;
        if (actA) rA = min(rA, (long long)ns);
        if (actB) rB = max(rB, 1LL);
        // the descent stops at a bin with at most ns / 1024 sample keys (exact mode: at most two)
        const unsigned few = stride == 1 ? 2u : (unsigned)max(2, ns >> 10);
        u64 pA = top0 >= 64 ? 0ull : (vor >> top0), pB = pA;
        int top = top0, topA = top0, topB = top0;
        while (top > 0 && (actA || actB)) {
            const int dbits = top < DB ? top : DB;
            const int sh = top - dbits;
            const bool split = actA && actB && pA != pB;
            hAB[tid] = 0u; hAB[tid + 1024] = 0u;
            __syncthreads();
            const u64 p1 = actA ? pA : pB;                       // prefix counted in hA (serves both ends while they agree)
#pragma unroll
            for (int i = 0; i < PER; ++i) {
                if (tid + i * 1024 < ns) {
                    const u64 kp = top >= 64 ? 0ull : (key[i] >> top);
                    const unsigned dg = (unsigned)((key[i] >> sh) & ((1u << dbits) - 1u));
                    if (kp == p1) atomicAdd(&hAB[dg], 1u);
                    else if (split && kp == pB) atomicAdd(&hAB[dg], 0x10000u);
                }
            }
            __syncthreads();
            find2(rA, actA, rB, actB, split);
            if (actA) {
                pA = (top >= 64 ? 0ull : (pA << dbits)) | (u64)s_digit[0];
                rA = s_r[0];
                topA = sh;
                if (s_cnt[0] <= few) actA = false;               // sparse bin: its outer edge only widens the bracket a little
            }
            if (actB) {
                pB = (top >= 64 ? 0ull : (pB << dbits)) | (u64)s_digit[1];
                rB = s_r[1];
                topB = sh;
                if (s_cnt[1] <= few) actB = false;
            }
            top = sh;
            __syncthreads();
        }
        if (!openA) lo = topA == 0 ? pA : (pA << topA);
        if (!openB) hi = topB == 0 ? pB : ((pB << topB) | ((1ull << topB) - 1ull));
    }
    if (tid == 0) {
        // histogram range: the bracket itself; an open end is replaced by the sample's extreme key plus half the range
        u64 e_lo = lo, e_hi = hi;
        if (!distrust && ns > 0) {
            if (lo == 0ull && kmin <= hi) { const u64 pad = (hi - kmin) / 2 + 1; e_lo = kmin > pad ? kmin - pad : 0ull; }
            if (hi == ~0ull && kmax >= lo) { const u64 pad = (kmax - e_lo) / 2 + 1; e_hi = (~0ull - kmax) > pad ? kmax + pad : ~0ull; }
        }
        flat_publish(st, lo, hi, e_lo, e_hi, e_lo + (e_hi - e_lo) / 2);
        st->lo2 = 0ull; st->hi2 = 0ull;
        st->n_below = 0ull;
        st->r1 = 0; st->r2 = 0;
        st->cand_count = 0u; st->cand2_count = 0u;
        st->mode = MODE_DONE;
        st->done_main = 0u; st->done_cand = 0u; st->done_refine = 0u;
        st->below_s = 0ull;
        st->bar_count = 0u; st->bar_abort = 0u;
        st->ns = ns;
        stats[0] = 0; stats[1] = 0; stats[2] = 0; stats[3] = ns;
    }
}

// ------------------------------------------------------------------ 1b. refinement round (largest arrays only)
// The bracket's width, and with it the candidate list, shrinks with the square root of the sample size, but one CTA
// cannot gather more than some ten thousand scattered scores in reasonable time.  For the largest arrays a second round
// spreads a 16 times larger sample over many CTAs: every sample key inside the first bracket is binned with the first
// bracket's histogram layout, keys below it are counted, and the last CTA reads the narrower bracket off the bins that
// hold the sample ranks several standard deviations around the expected one.  Any outcome is a valid bracket or the
// first one unchanged; the exact stages after it check whatever they are given.
constexpr int REFINE_CTAS = 128, REFINE_THREADS = 256, REFINE_PER = 8;     // 2^18 samples
__global__ void __launch_bounds__(REFINE_THREADS)
flat_refine_kernel(const float* __restrict__ s, long long n, long long k_evict, FlatState* __restrict__ st,
                   uint32_t* __restrict__ hist2, long long* __restrict__ stats, float sigmas) {
    __shared__ uint32_t sh[FB];
    __shared__ unsigned long long wt[REFINE_THREADS / 32];
    __shared__ int s_bin[3];
    __shared__ int s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr long long CAP = (long long)REFINE_CTAS * REFINE_THREADS * REFINE_PER;
    grid_dependents_may_launch();
    grid_dependency_wait();                                // the first bracket comes from the kernel before
    const u64 lo = st->lo, hi = st->hi, bin_base = st->bin_base;
    const int shift = st->shift;
    for (int i = tid; i < FB; i += REFINE_THREADS) sh[i] = 0u;
    __syncthreads();
    const long long stride = (n + CAP - 1) / CAP;
    const long long ns2 = (n + stride - 1) / stride;
    uint32_t sidx[REFINE_PER];
    float sval[REFINE_PER];
    const long long j0 = ((long long)blockIdx.x * REFINE_PER) * REFINE_THREADS + tid;
#pragma unroll
    for (int i = 0; i < REFINE_PER; ++i) {
        const long long j = j0 + (long long)i * REFINE_THREADS;
        sidx[i] = 0u;
        if (j < ns2) {
            const long long base = j * stride;
            const uint32_t width = (uint32_t)min(stride, n - base);
            sidx[i] = (uint32_t)base + (width > 1u ? mix32((uint32_t)j * 0x85EBCA77u + 0x2545F491u) % width : 0u);
        }
    }
#pragma unroll
    for (int i = 0; i < REFINE_PER; ++i) sval[i] = (j0 + (long long)i * REFINE_THREADS < ns2) ? __ldg(s + sidx[i]) : 0.0f;
    unsigned below = 0;
#pragma unroll
    for (int i = 0; i < REFINE_PER; ++i) {
        if (j0 + (long long)i * REFINE_THREADS < ns2) {
            const u64 key = flat_key(sval[i], sidx[i]);
            if (key < lo) ++below;
            else if (key <= hi) atomicAdd(&sh[flat_bin(key, bin_base, shift)], 1u);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) below += __shfl_xor_sync(0xffffffffu, below, o);
    if (lane == 0 && below) atomicAdd(&st->below_s, (unsigned long long)below);
    __syncthreads();
    for (int i = tid; i < FB; i += REFINE_THREADS) {
        const uint32_t v = sh[i];
        if (v) atomicAdd(hist2 + i, v);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(&st->done_refine, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // ---- last CTA: sample ranks -> bins -> narrower bracket
    constexpr int PERT = FB / REFINE_THREADS;
    unsigned v[PERT];
    unsigned long long local = 0;
#pragma unroll
    for (int i = 0; i < PERT; ++i) { v[i] = __ldcg(hist2 + tid * PERT + i); local += v[i]; }
    unsigned long long incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (tid < 3) s_bin[tid] = -1;
    if (lane == 31) wt[warp] = incl;
    __syncthreads();
    unsigned long long off = 0, total = 0;
#pragma unroll
    for (int w = 0; w < REFINE_THREADS / 32; ++w) { if (w < warp) off += wt[w]; total += wt[w]; }
    const long long below_s = (long long)*((volatile unsigned long long*)&st->below_s);
    const float q = (float)((double)k_evict / (double)n);
    const float mu = q * (float)ns2;
    const float dev = sigmas * sqrtf(mu * (1.0f - q)) + 8.0f;
    // ranks among the sample keys inside the first bracket (1-based)
    const long long r[3] = {(long long)floorf(mu - dev) - below_s, (long long)ceilf(mu + dev) + 1 - below_s,
                            (long long)llrintf(mu) - below_s};
    const unsigned long long excl = off + incl - local;
#pragma unroll
    for (int w = 0; w < 3; ++w) {
        unsigned long long cum = excl;
#pragma unroll
        for (int i = 0; i < PERT; ++i) {
            if (r[w] >= 1 && (unsigned long long)r[w] > cum && (unsigned long long)r[w] <= cum + v[i]) s_bin[w] = tid * PERT + i;
            cum += v[i];
        }
    }
    __syncthreads();
    if (tid == 0) {
        const u64 e_hi0 = st->e_hi;
        auto lower_edge = [&](int b) -> u64 { return b <= 0 ? lo : bin_base + ((u64)b << shift); };
        auto upper_edge = [&](int b) -> u64 {
            if (b >= FB - 1) return hi;
            const u64 e = bin_base + ((u64)(b + 1) << shift) - 1ull;
            return (e >= bin_base && e < hi) ? e : hi;
        };
        // an end whose rank fell outside the first bracket's sample keys stays where it was
        u64 nlo = lo, nhi = hi;
        if (s_bin[0] >= 0) nlo = lower_edge(s_bin[0]);
        if (s_bin[1] >= 0) nhi = upper_edge(s_bin[1]);
        const bool sane = nlo <= nhi && r[0] <= (long long)total && r[1] >= 1;
        if (sane && (nlo != lo || nhi != hi)) {
            const u64 e_lo = nlo == lo ? bin_base : nlo;          // an end that stays open keeps its stand-in
            const u64 e_hi = nhi == hi ? e_hi0 : nhi;
            const u64 mid = s_bin[2] >= 0 ? lower_edge(s_bin[2]) : e_lo + (e_hi - e_lo) / 2;
            flat_publish(st, nlo, nhi, e_lo, e_hi, mid);
        }
        stats[3] = (long long)ns2;
    }
}

// ------------------------------------------------------------------ 2. the pass over the scores
constexpr int FBUF = 128;         // candidate keys a warp stages before it takes a slice of the global list
constexpr int FJ = 16;            // ballots per warp trip: a warp takes 32 * FJ = 512 consecutive scores
constexpr int MAIN_WARPS = 24;
constexpr int MAIN_THREADS = MAIN_WARPS * 32;

// Appends the warp's staged keys to the candidate list (one atomic per flush).  Keys beyond the list's capacity are
// dropped; the count still includes them, which tells the last CTA that the list overflowed.
__device__ __noinline__ void flat_flush(const u64* wb, int nbuf, FlatState* st, u64* cand, long long cap) {
    const int lane = threadIdx.x & 31;
    unsigned base = 0;
    if (lane == 0) base = atomicAdd(&st->cand_count, (unsigned)nbuf);
    base = __shfl_sync(0xffffffffu, base, 0);
    for (int i = lane; i < nbuf; i += 32)
        if ((long long)base + i < cap) cand[(long long)base + i] = wb[i];
    __syncwarp();
}

// Last CTA of the main pass: the histogram bin that holds the k-th smallest key becomes the fine bracket.
__device__ void flat_pick_bin(FlatState* st, const uint32_t* hist, long long k_evict, long long cand_cap, long long* stats) {
    __shared__ unsigned long long wt[MAIN_WARPS];
    __shared__ int s_bin;
    __shared__ unsigned long long s_before;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int PICK_THREADS = 512, PERT = FB / PICK_THREADS;          // the first 512 threads hold eight bins each
    static_assert(MAIN_THREADS >= PICK_THREADS, "the scan needs 512 threads");
    unsigned v[PERT];
    unsigned long long local = 0;
    {
        // every load is issued before the first sum: one round trip to L2, not one per copy and bin
        uint4 part[HREP][PERT / 4];
        const int t = tid < PICK_THREADS ? tid : 0;
#pragma unroll
        for (int r = 0; r < HREP; ++r)
#pragma unroll
            for (int q = 0; q < PERT / 4; ++q) part[r][q] = __ldcg(reinterpret_cast<const uint4*>(hist + r * FB + t * PERT) + q);
#pragma unroll
        for (int q = 0; q < PERT / 4; ++q) {
            uint4 a = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int r = 0; r < HREP; ++r) { a.x += part[r][q].x; a.y += part[r][q].y; a.z += part[r][q].z; a.w += part[r][q].w; }
            v[4 * q] = a.x; v[4 * q + 1] = a.y; v[4 * q + 2] = a.z; v[4 * q + 3] = a.w;
        }
#pragma unroll
        for (int i = 0; i < PERT; ++i) {
            if (tid >= PICK_THREADS) v[i] = 0u;
            local += v[i];
        }
    }
    unsigned long long incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (tid == 0) s_bin = -1;
    if (lane == 31) wt[warp] = incl;
    __syncthreads();
    unsigned long long off = 0, total = 0;
#pragma unroll
    for (int w = 0; w < MAIN_WARPS; ++w) { if (w < warp) off += wt[w]; total += wt[w]; }
    const unsigned long long n_below = *((volatile unsigned long long*)&st->n_below);
    const long long r1 = k_evict - (long long)n_below;               // rank of the k-th key among the candidates
    const unsigned long long excl = off + incl - local;
    if (r1 >= 1 && (unsigned long long)r1 > excl && (unsigned long long)r1 <= excl + local) {
        unsigned long long cum = excl;
#pragma unroll
        for (int i = 0; i < PERT; ++i) {
            if (tid < PICK_THREADS && (unsigned long long)r1 > cum && (unsigned long long)r1 <= cum + v[i]) { s_bin = tid * PERT + i; s_before = cum; }
            cum += v[i];
        }
    }
    __syncthreads();
    if (tid == 0) {
        const unsigned cc = *((volatile unsigned*)&st->cand_count);
        st->r1 = r1;
        if (s_bin < 0 || (long long)cc > cand_cap || (unsigned long long)cc != total) {
            st->mode = MODE_EXACT_ALL;                                  // bracket missed the k-th key, or the list overflowed
        } else {
            const int shift = st->shift;
            const u64 base = st->bin_base, lo = st->lo, hi = st->hi;
            u64 lo2 = lo, hi2 = hi;                                     // the end bins also take what lies beyond the binned range
            if (s_bin > 0) lo2 = base + ((u64)s_bin << shift);
            if (s_bin < FB - 1) {
                const u64 e = base + ((u64)(s_bin + 1) << shift) - 1ull;
                if (e >= base && e < hi) hi2 = e;
            }
            if (lo2 < lo) lo2 = lo;
            st->lo2 = lo2;
            st->hi2 = hi2;
            st->r2 = r1 - (long long)s_before;
        }
        stats[1] = (long long)cc;
    }
}

// Each warp streams its 512-score trips from HBM through a ring of its own in shared memory: lane 0 issues one bulk
// asynchronous copy (2 KB) per trip, RING - 1 trips ahead, completing on an mbarrier; the warp reads a trip's scores from
// shared memory (lane l takes scores 32 j + l: conflict-free, and ballot j is then 32 consecutive keep bits).
// FINITE: both ends of the bracket are finite floats, so one subtraction and one compare tell (conservatively) whether a
// score's word can lie inside the bracket; otherwise two compares do.  Per score the common path is: that test, the
// compare with `mid` that gives the keep bit, a ballot.  Scores that may be inside are handled after the trip, each lane
// walking through its own (a few percent of the scores): exact 64-bit classification, candidate list, histogram, and
// the rare keep bit that the exact comparison decides differently.
constexpr int RING = 3;
constexpr int TRIP = 32 * FJ;                    // scores per trip
constexpr int MAIN_SMEM_HIST = FB * 4;
constexpr int MAIN_SMEM_RING = MAIN_WARPS * RING * TRIP * 4;
constexpr int MAIN_SMEM_STAGE = MAIN_WARPS * FBUF * 8;
constexpr int MAIN_SMEM_ELIST = MAIN_WARPS * TRIP * 2;           // per warp: positions of the trip's scores that may be inside
constexpr int MAIN_SMEM_WORDS = MAIN_WARPS * FJ * 4;             // per warp: the trip's 16 ballots
constexpr int MAIN_OFF_RING = MAIN_SMEM_HIST;
constexpr int MAIN_OFF_STAGE = MAIN_OFF_RING + MAIN_SMEM_RING;
constexpr int MAIN_OFF_ELIST = MAIN_OFF_STAGE + MAIN_SMEM_STAGE;
constexpr int MAIN_OFF_WORDS = MAIN_OFF_ELIST + MAIN_SMEM_ELIST;
constexpr int MAIN_OFF_BARS = MAIN_OFF_WORDS + MAIN_SMEM_WORDS;
constexpr int MAIN_OFF_CNT = MAIN_OFF_BARS + MAIN_WARPS * RING * 8;
constexpr int MAIN_SMEM_BYTES = MAIN_OFF_CNT + MAIN_WARPS * 4 + 32;

struct MainSmem {          // one warp's views of the CTA's dynamic shared memory
    uint32_t* sh;          // candidate histogram (shared by the CTA)
    float* ring;
    uint64_t* bars;
    u64* wb;               // staged candidate keys
    unsigned short* elist;
    uint32_t* words;
    unsigned* ecount;
};

template <int FORM>
__device__ __forceinline__ void flat_main_body(const float* __restrict__ s, long long n, FlatState* __restrict__ st,
                                               u64* __restrict__ cand, long long cand_cap, u64* __restrict__ keep_bits,
                                               int32_t* __restrict__ status, const MainSmem& sm) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const u64 lo = st->lo, hi = st->hi, mid = st->mid, bin_base = st->bin_base;
    const int shift = st->shift;
    const float lo_f = st->lo_f, hi_f = st->hi_f, mid_lt = st->mid_lt, ctr = st->ctr, hw = st->hw;
    const long long words = (n + 63) / 64;
    const long long nfull = n / TRIP;                            // full trips: streamed through the ring
    const long long W = (long long)gridDim.x * MAIN_WARPS;
    const long long c0 = (long long)blockIdx.x * MAIN_WARPS + warp;
    const int my_trips = c0 < nfull ? (int)((nfull - c0 + W - 1) / W) : 0;        // at most 2^23: indices are 32 bits wide
    const bool lane0 = lane == 0;
    int nbuf = 0;                                // warp-uniform fill of the staging buffer
    unsigned ev_fast = 0;                        // lanes < 8: scores of their words with the keep bit clear
    int adj = 0;                                 // per lane: (inside scores below lo) - (inside scores with the keep bit clear)
    bool bad = false, failed = false;

    constexpr bool FINITE = FORM >= 1;
    auto inside_of = [&](float xv) -> bool {
        if (FINITE) return !(fabsf(xv - ctr) > hw);                  // true for NaN as well: it is reported below
        return !(xv < lo_f) && !(xv > hi_f);
    };
    // lane 0 keeps the copy it issues next (RING - 1 trips ahead of the trip being read).  The stage a copy refills was
    // read one trip earlier, and the warp barrier that ends a trip orders those reads before the copy is issued.
    const float* src_next = s + c0 * TRIP;
    const long long src_step = W * TRIP;
    int issue_stg = 0, issued = 0;
    auto issue = [&]() {
        if (lane0 && issued < my_trips) {
            mbar_expect_tx(sm.bars + issue_stg, TRIP * 4);
            bulk_g2s(sm.ring + issue_stg * TRIP, src_next, TRIP * 4, sm.bars + issue_stg);
            src_next += src_step;
            issue_stg = issue_stg == RING - 1 ? 0 : issue_stg + 1;
            ++issued;
        }
    };
    // After a trip's keep words are written: the scores that may be inside.  Every lane lists the positions of its own;
    // the warp then classifies the listed scores exactly, 32 at a time.  xs: the trip's scores in shared memory (null for
    // the ragged last trip, which re-reads them from global memory).
    // exact classification of one score that may be inside; returns true if it is a candidate (key: its key)
    auto classify = [&](float xv, uint32_t idx, u64& key) -> bool {
        bad |= xv != xv;
        key = flat_key(xv, idx);
        const bool fast_ev = xv < mid_lt;
        const bool ev = key < mid;
        adj += (key < lo ? 1 : 0) - (fast_ev ? 1 : 0);
        const bool cnd = key >= lo && key <= hi;
        if (cnd) atomicAdd(&sm.sh[flat_bin(key, bin_base, shift)], 1u);
        if (ev != fast_ev) {                                     // equal score words, the index decides: settle the bit now
            unsigned long long* wp = reinterpret_cast<unsigned long long*>(keep_bits + (idx >> 6));
            if (ev) atomicAnd(wp, ~(1ull << (idx & 63))); else atomicOr(wp, 1ull << (idx & 63));
        }
        return cnd;
    };
    // consec: bit j of m is the lane's score 16 lane + j of the trip (arithmetic form); otherwise score 32 j + lane
    auto handle_inside = [&](unsigned m, long long base, const float* xs, bool consec) {
        const int tot_in = __reduce_add_sync(0xffffffffu, __popc(m));
        if (!tot_in) return;
        if (tot_in <= 8) {
            // a handful: every lane that has some takes its own, one per round (rounds = the most any lane has, mostly one)
            if (nbuf + tot_in > FBUF) {
                flat_flush(sm.wb, nbuf, st, cand, cand_cap);
                nbuf = 0;
            }
            __syncwarp();                                        // the trip's keep words are written
            while (__any_sync(0xffffffffu, m != 0u)) {
                bool cnd = false;
                u64 key = 0ull;
                if (m) {
                    const int j = __ffs(m) - 1;
                    const int p = consec ? 16 * lane + j : 32 * j + lane;
                    m &= m - 1;
                    cnd = classify(xs ? xs[p] : __ldg(s + base + p), (uint32_t)base + (uint32_t)p, key);
                }
                const unsigned cdb = __ballot_sync(0xffffffffu, cnd);
                if (cnd) sm.wb[nbuf + __popc(cdb & ((1u << lane) - 1u))] = key;
                nbuf += __popc(cdb);
            }
            __syncwarp();
            return;
        }
        if (lane0) *sm.ecount = 0u;
        __syncwarp();
        if (m) {
            unsigned pos = atomicAdd(sm.ecount, (unsigned)__popc(m));
            while (m) {
                const int j = __ffs(m) - 1;
                m &= m - 1;
                sm.elist[pos++] = (unsigned short)(consec ? 16 * lane + j : 32 * j + lane);
            }
        }
        __syncwarp();
        const int tot = (int)*((volatile unsigned*)sm.ecount);
        for (int e0 = 0; e0 < tot; e0 += 32) {
            if (nbuf + 32 > FBUF) {                              // room for this batch (warp-uniform)
                flat_flush(sm.wb, nbuf, st, cand, cand_cap);
                nbuf = 0;
            }
            const int e = e0 + lane;
            bool cnd = false;
            u64 key = 0ull;
            if (e < tot) {
                const int p = sm.elist[e];
                cnd = classify(xs ? xs[p] : __ldg(s + base + p), (uint32_t)base + (uint32_t)p, key);
            }
            const unsigned cdb = __ballot_sync(0xffffffffu, cnd);
            if (cnd) sm.wb[nbuf + __popc(cdb & ((1u << lane) - 1u))] = key;
            nbuf += __popc(cdb);
        }
        __syncwarp();
    };
    // the 16 ballots of a trip sit in shared memory (written by lane 0); lanes 0..7 turn them into keep words
    // (full: a whole trip of 512 scores, every word inside the array)
    auto write_words = [&](long long word0, int live_scores, bool full) {
        __syncwarp();
        if (lane < FJ / 2 && (full || word0 + lane < words)) {
            const u64 wv = *reinterpret_cast<const u64*>(sm.words + 2 * lane);
            keep_bits[word0 + lane] = wv;
            const int lb = full ? 64 : min(64, max(0, live_scores - 64 * lane));
            ev_fast += (unsigned)(lb - __popcll(wv));
        }
    };

    for (int i = 0; i < RING - 1; ++i) issue();
    long long c = c0;
    int t = 0, stg = 0;
    uint32_t phase = 0;
    // arithmetic form: the four 16-byte loads of a lane, as byte offsets into a stage.  Chunk it of the lane is read as
    // chunk it ^ r4 with r4 = (lane / 2) & 3, so that the eight lanes served together touch all banks
    const int r4 = (lane >> 1) & 3;
    const uint32_t off0 = (uint32_t)(lane * 64 + (r4 << 4));
    u64* kw = keep_bits + c0 * (FJ / 2) + lane;                  // lanes 0..7: the keep word of the current trip
    const long long kw_step = W * (FJ / 2);
    for (; t < my_trips; ++t, c += W, kw += kw_step) {
        issue();
        if (!mbar_wait_bounded(sm.bars + stg, phase)) { failed = true; break; }
        const float* xs = sm.ring + stg * TRIP;
        unsigned m = 0u;                                         // this lane's scores of the trip that may be inside
        if (FORM == 2) {
            // Arithmetic form: lane l takes the 16 CONSECUTIVE scores 16 l .. 16 l + 15, so its 16 keep bits are a
            // quarter of a keep word as they stand, and no ballot is needed.  The two tests run on the FMA pipe:
            //   evicted  <=>  x < mid_lt          <=>  saturate((mid_lt - x) * 2^126) = 1
            //   outside  <=>  |x - ctr| > hw      <=>  saturate((|x - ctr| - hw) * 2^126) = 1
            // (a difference of two distinct floats is never zero; with |mid_lt| and hw at least 2^-100 a positive one is
            // at least 2^-124, so the product saturates to exactly 1; a negative one, zero or NaN gives exactly 0, and a
            // NaN score is thereby kept and listed as possibly inside, as in the compare form.)  The bits are collected
            // as a binary number in a float (16 bits: exact).
            const char* xb = reinterpret_cast<const char*>(xs);
            float4 v[4];
#pragma unroll
            for (int it = 0; it < 4; ++it) v[it] = *reinterpret_cast<const float4*>(xb + (off0 ^ (uint32_t)(it << 4)));
            float acc_e = 0.f, acc_o = 0.f;
#pragma unroll
            for (int it = 3; it >= 0; --it) {
                const float xe[4] = {v[it].x, v[it].y, v[it].z, v[it].w};
#pragma unroll
                for (int e = 3; e >= 0; --e) {
                    acc_e = fmaf(acc_e, 2.0f, __saturatef((mid_lt - xe[e]) * 0x1p126f));
                    acc_o = fmaf(acc_o, 2.0f, __saturatef((fabsf(xe[e] - ctr) - hw) * 0x1p126f));
                }
            }
            // local nibble `it` holds the scores of nibble it ^ r4: swap nibbles within bytes if r4 & 1, bytes if r4 & 2
            // (both 16-bit masks at once, one in each half of a word)
            unsigned eo = (unsigned)acc_e | ((unsigned)acc_o << 16);
            if (r4 & 1) eo = ((eo & 0x0F0F0F0Fu) << 4) | ((eo >> 4) & 0x0F0F0F0Fu);
            if (r4 & 2) eo = __byte_perm(eo, 0u, 0x2301);
            const unsigned keep16 = ~eo & 0xFFFFu;
            m = ~eo >> 16;
            ev_fast += 16u - (unsigned)__popc(keep16);
            reinterpret_cast<unsigned short*>(sm.words)[lane] = (unsigned short)keep16;
            __syncwarp();
            if (lane < FJ / 2) *kw = *reinterpret_cast<const u64*>(sm.words + 2 * lane);
        } else {
            float x[FJ];                                         // all 16 loads first: none waits behind a store
#pragma unroll
            for (int j = 0; j < FJ; ++j) x[j] = xs[32 * j + lane];
            unsigned kb[FJ];
#pragma unroll
            for (int j = 0; j < FJ; ++j) {
                if (inside_of(x[j])) m |= 1u << j;
                kb[j] = __ballot_sync(0xffffffffu, !(x[j] < mid_lt));
            }
            if (lane0) {
#pragma unroll
                for (int j = 0; j < FJ; j += 4) *reinterpret_cast<uint4*>(sm.words + j) = make_uint4(kb[j], kb[j + 1], kb[j + 2], kb[j + 3]);
            }
            write_words(c * (FJ / 2), TRIP, true);
        }
        handle_inside(m, c * TRIP, xs, FORM == 2);
        __syncwarp();                                            // every lane is done with this stage before it is refilled
        if (stg == RING - 1) { stg = 0; phase ^= 1u; } else ++stg;
    }
    if (failed) {                                                // a wait gave up: report, and let the copies in flight land
        latch_error(status, TRIMKV_E_TIMEOUT);
        for (int u = t; u < my_trips && u < t + RING; ++u)                  // trips issued and not yet waited for
            mbar_wait_bounded(sm.bars + u % RING, (uint32_t)((u / RING) & 1));
    }
    // the ragged last trip (fewer than 512 scores), by the warp whose turn it would be: plain loads
    if (nfull * TRIP < n && c0 == nfull % W) {
        const long long base = nfull * TRIP, rem = n - base;
        unsigned m = 0u;
#pragma unroll 1
        for (int j = 0; j < FJ; ++j) {
            const bool live = 32 * j + lane < rem;
            const float xv = live ? __ldg(s + base + 32 * j + lane) : 0.0f;
            if (live && inside_of(xv)) m |= 1u << j;
            const unsigned kb = __ballot_sync(0xffffffffu, live && !(xv < mid_lt));
            if (lane0) sm.words[j] = kb;
        }
        write_words(nfull * (FJ / 2), (int)rem, false);
        handle_inside(m, base, nullptr, false);
    }
    if (nbuf > 0) flat_flush(sm.wb, nbuf, st, cand, cand_cap);
    if (bad) latch_error(status, TRIMKV_E_NONFINITE);
    // keys below lo = (scores whose keep bit the fast compare cleared) corrected by the scores classified exactly
    long long nb = (long long)ev_fast + (long long)adj;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) nb += __shfl_xor_sync(0xffffffffu, nb, o);
    if (lane0 && nb) atomicAdd(&st->n_below, (unsigned long long)nb);
}

__global__ void __launch_bounds__(MAIN_THREADS, 1)
flat_main_kernel(const float* __restrict__ s, long long n, long long k_evict, FlatState* __restrict__ st,
                 uint32_t* __restrict__ hist, u64* __restrict__ cand, long long cand_cap, u64* __restrict__ keep_bits,
                 long long* __restrict__ stats, int32_t* __restrict__ status) {
    extern __shared__ __align__(128) unsigned char fm_smem[];
    __shared__ int s_last;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    MainSmem sm;
    sm.sh = reinterpret_cast<uint32_t*>(fm_smem);
    sm.ring = reinterpret_cast<float*>(fm_smem + MAIN_OFF_RING) + (size_t)warp * RING * TRIP;
    sm.wb = reinterpret_cast<u64*>(fm_smem + MAIN_OFF_STAGE) + (size_t)warp * FBUF;
    sm.elist = reinterpret_cast<unsigned short*>(fm_smem + MAIN_OFF_ELIST) + (size_t)warp * TRIP;
    sm.words = reinterpret_cast<uint32_t*>(fm_smem + MAIN_OFF_WORDS) + warp * FJ;
    sm.bars = reinterpret_cast<uint64_t*>(fm_smem + MAIN_OFF_BARS) + warp * RING;
    sm.ecount = reinterpret_cast<unsigned*>(fm_smem + MAIN_OFF_CNT) + warp;
    uint32_t* sh = sm.sh;
    for (int i = threadIdx.x; i < FB; i += MAIN_THREADS) sh[i] = 0u;
    if (lane == 0) {
        *sm.ecount = 0u;
        for (int i = 0; i < RING; ++i) mbar_init(sm.bars + i, 1);
    }
    fence_proxy_async_smem();
    grid_dependents_may_launch();
    grid_dependency_wait();                                // shared memory is set up; the bracket comes from the kernel before
    __syncthreads();
    const int form = st->finite;
    if (blockIdx.x == 0 && threadIdx.x == 0) stats[4] = form;
    if (form == 2) flat_main_body<2>(s, n, st, cand, cand_cap, keep_bits, status, sm);
    else if (form == 1) flat_main_body<1>(s, n, st, cand, cand_cap, keep_bits, status, sm);
    else flat_main_body<0>(s, n, st, cand, cand_cap, keep_bits, status, sm);
    __syncthreads();
    uint32_t* hrep = hist + (size_t)(blockIdx.x % HREP) * FB;
    for (int i = threadIdx.x; i < FB; i += MAIN_THREADS) {
        const uint32_t v = sh[i];
        if (v) atomicAdd(hrep + i, v);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(&st->done_main, 1u) == gridDim.x - 1);
    __syncthreads();
    if (s_last) {
        __threadfence();
        flat_pick_bin(st, hist, k_evict, cand_cap, stats);
    }
}

// ------------------------------------------------------------------ 3. the pass over the candidate list
__device__ __forceinline__ void set_keep(u64* keep_bits, u64 key, bool keep) {
    const uint32_t idx = ~(uint32_t)key;                     // the key's low word is ~index
    if (keep) atomicOr(reinterpret_cast<unsigned long long*>(keep_bits + (idx >> 6)), 1ull << (idx & 63));
    else atomicAnd(reinterpret_cast<unsigned long long*>(keep_bits + (idx >> 6)), ~(1ull << (idx & 63)));
}

// Last CTA (1024 threads): the r2-th smallest key of the fine bracket is the threshold tau; every key up to tau is
// evicted.  The main pass set each candidate's bit by comparing with `mid`; only bits that tau decides otherwise flip.
__device__ void flat_resolve(FlatState* st, const u64* cand2, u64* keep_bits, long long* stats) {
    constexpr int DB = 11, NBIN = 1 << DB, PER = CAND2_CAP / 1024;
    __shared__ unsigned hist[NBIN];
    __shared__ unsigned wtot[32];
    __shared__ u64 s_or[32], s_and[32];
    __shared__ u64 s_prefix;
    __shared__ long long s_r;
    __shared__ int s_found;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long C = (long long)*((volatile unsigned*)&st->cand2_count);
    long long r = st->r2;
    const u64 mid = st->mid;
    if (C > CAND2_CAP) {                                      // too crowded a bin (heavy clustering): exact select over the list
        if (tid == 0) { st->mode = MODE_EXACT_LIST; stats[2] = C; }
        return;
    }
    if (r < 1 || r > C) {                                     // cannot happen with consistent counts: redo everything exactly
        if (tid == 0) { st->mode = MODE_EXACT_ALL; stats[2] = C; }
        return;
    }
    if (C <= 512) {
        // the usual case, a few hundred keys: every thread that holds a key counts the keys below its own (the keys are
        // unique, so the thread whose count is r - 1 holds the threshold): C broadcast reads per key holder, cheaper than
        // several radix sweeps of the whole CTA up to about this size
        __shared__ u64 skeys[512];
        __shared__ u64 s_tau;
        const bool have = tid < C;
        const u64 mine = have ? __ldcg(cand2 + tid) : 0ull;
        if (have) skeys[tid] = mine;
        __syncthreads();
        int below = 0;
        if (have) {                                            // whole warps beyond the list skip the loop
#pragma unroll 8
            for (int j = 0; j < (int)C; ++j) below += skeys[j] < mine ? 1 : 0;
        }
        if (have && below == (int)r - 1) s_tau = mine;
        __syncthreads();
        const u64 tau = s_tau;
        if (have) {
            const bool keep = mine > tau;
            if (keep != (mine >= mid)) set_keep(keep_bits, mine, keep);
        }
        if (tid == 0) stats[2] = C;
        return;
    }
    u64 kr[PER];
    u64 vor = 0ull, vand = ~0ull;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const long long idx = tid + (long long)i * 1024;
        kr[i] = idx < C ? __ldcg(cand2 + idx) : 0ull;
        if (idx < C) { vor |= kr[i]; vand &= kr[i]; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        vor |= __shfl_xor_sync(0xffffffffu, vor, o);
        vand &= __shfl_xor_sync(0xffffffffu, vand, o);
    }
    if (lane == 0) { s_or[warp] = vor; s_and[warp] = vand; }
    __syncthreads();
    vor = 0ull; vand = ~0ull;
    for (int w = 0; w < 32; ++w) { vor |= s_or[w]; vand &= s_and[w]; }
    const u64 diff = vor ^ vand;
    int top = diff ? 64 - __clzll((long long)diff) : 0;
    u64 prefix = top >= 64 ? 0ull : (vor >> top);
    while (top > 0) {
        const int dbits = top < DB ? top : DB;
        const int sh = top - dbits;
        hist[tid] = 0u;
        hist[tid + 1024] = 0u;
        if (tid == 0) s_found = 0;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            if (tid + (long long)i * 1024 < C) {
                const bool match = top >= 64 ? true : ((kr[i] >> top) == prefix);
                if (match) atomicAdd(&hist[(unsigned)((kr[i] >> sh) & ((1u << dbits) - 1u))], 1u);
            }
        }
        __syncthreads();
        const unsigned h0 = hist[2 * tid], h1 = hist[2 * tid + 1];
        unsigned incl = h0 + h1;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) wtot[warp] = incl;
        __syncthreads();
        unsigned off = 0;
        for (int w = 0; w < warp; ++w) off += wtot[w];
        const long long excl = (long long)off + incl - (h0 + h1);
        if (r > excl && r <= excl + h0) {
            s_prefix = (top >= 64 ? 0ull : (prefix << dbits)) | (u64)(2 * tid);
            s_r = r - excl;
            s_found = 1;
        } else if (r > excl + h0 && r <= excl + h0 + h1) {
            s_prefix = (top >= 64 ? 0ull : (prefix << dbits)) | (u64)(2 * tid + 1);
            s_r = r - excl - h0;
            s_found = 1;
        }
        __syncthreads();
        if (!s_found) {                                       // cannot happen: the counts cover all C keys
            if (tid == 0) st->mode = MODE_EXACT_ALL;
            return;
        }
        prefix = s_prefix;
        r = s_r;
        top = sh;
        __syncthreads();
    }
    const u64 tau = prefix;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        if (tid + (long long)i * 1024 < C) {
            const bool keep = kr[i] > tau;
            if (keep != (kr[i] >= mid)) set_keep(keep_bits, kr[i], keep);
        }
    }
    if (tid == 0) stats[2] = C;
}

__global__ void __launch_bounds__(1024)
flat_cand_kernel(FlatState* __restrict__ st, const u64* __restrict__ cand, u64* __restrict__ cand2,
                 u64* __restrict__ keep_bits, long long* __restrict__ stats) {
    __shared__ int s_last;
    grid_dependency_wait();                                   // the list and its bin come from the kernel before
    if (st->mode != MODE_DONE) return;                        // the exact fallback over all scores takes over
    const int lane = threadIdx.x & 31;
    const long long C1 = (long long)st->cand_count;
    const u64 lo2 = st->lo2, hi2 = st->hi2, mid = st->mid;
    // eight keys per thread and trip are requested before any is used (the list is read once, from L2 or HBM)
    constexpr int U = 8;
    const long long T = (long long)gridDim.x * blockDim.x;
    const long long trips = (C1 + T * U - 1) / (T * U);       // warp-uniform trip count
    long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    for (long long t = 0; t < trips; ++t, i0 += T * U) {
        u64 keys[U];
#pragma unroll
        for (int u = 0; u < U; ++u) keys[u] = (i0 + u * T < C1) ? __ldcs(cand + i0 + u * T) : 0ull;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const u64 key = keys[u];
            bool fine = false;
            if (i0 + u * T < C1) {
                if (key < lo2) { if (key >= mid) set_keep(keep_bits, key, false); }       // below the threshold: evicted
                else if (key > hi2) { if (key < mid) set_keep(keep_bits, key, true); }    // above it: kept
                else fine = true;
            }
            const unsigned fb = __ballot_sync(0xffffffffu, fine);
            if (fb) {
                unsigned base = 0;
                if (lane == 0) base = atomicAdd(&st->cand2_count, (unsigned)__popc(fb));
                base = __shfl_sync(0xffffffffu, base, 0);
                const unsigned w = base + __popc(fb & ((1u << lane) - 1u));
                if (fine && w < (unsigned)CAND2_CAP) cand2[w] = key;
            }
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(&st->done_cand, 1u) == gridDim.x - 1);
    __syncthreads();
    if (s_last) {
        __threadfence();
        flat_resolve(st, cand2, keep_bits, stats);
    }
}

// ------------------------------------------------------------------ 4. exact fallback (cooperative launch)
// Grid-wide barrier for a kernel whose CTAs are all resident (cooperative launch).  The wait is bounded: a CTA that
// gives up raises the abort flag, which releases the others, and the status word reports TRIMKV_E_TIMEOUT.
__device__ bool grid_barrier(FlatState* st, unsigned& epoch, int32_t* status) {
    __shared__ int s_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        bool ok = true;
        __threadfence();
        epoch += 1;
        const unsigned target = epoch * gridDim.x;
        atomicAdd(&st->bar_count, 1u);
        unsigned it = 0;
        while (*((volatile unsigned*)&st->bar_count) < target) {
            if (*((volatile unsigned*)&st->bar_abort)) { ok = false; break; }
            if (++it > BARRIER_SPIN_LIMIT) {
                atomicExch(&st->bar_abort, 1u);
                latch_error(status, TRIMKV_E_TIMEOUT);
                ok = false;
                break;
            }
            __nanosleep(100);
        }
        __threadfence();
        s_ok = ok ? 1 : 0;
    }
    __syncthreads();
    return s_ok != 0;
}

// Exact radix select (digits of 11 bits from the top) over the candidate list (MODE_EXACT_LIST) or over all scores
// (MODE_EXACT_ALL), then every bit it decides is written.  ghist: X_PASSES histograms of XB bins.
__global__ void __launch_bounds__(256)
flat_exact_kernel(const float* __restrict__ s, long long n, long long k_evict, FlatState* __restrict__ st,
                  const u64* __restrict__ cand, uint32_t* __restrict__ ghist, u64* __restrict__ keep_bits,
                  long long* __restrict__ stats, int32_t* __restrict__ status) {
    __shared__ unsigned sh[XB];
    __shared__ unsigned wt[8];
    __shared__ int s_digit;
    __shared__ long long s_rnew;
    const int mode = st->mode;
    if (mode == MODE_DONE) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool list = mode == MODE_EXACT_LIST;
    const long long N = list ? (long long)st->cand_count : n;
    long long r = list ? st->r1 : k_evict;                    // the r-th smallest key of the source is the threshold
    const long long T = (long long)gridDim.x * blockDim.x;
    const long long g0 = (long long)blockIdx.x * blockDim.x + tid;
    unsigned epoch = 0;
    for (long long i = g0; i < (long long)X_PASSES * XB; i += T) ghist[i] = 0u;
    if (!grid_barrier(st, epoch, status)) return;
    auto key_at = [&](long long i) -> u64 { return list ? __ldg(cand + i) : flat_key(__ldg(s + i), (uint32_t)i); };
    u64 prefix = 0ull;
    int top = 64;
    for (int pass = 0; pass < X_PASSES; ++pass) {
        const int dbits = top < XB_BITS ? top : XB_BITS;
        const int shf = top - dbits;
        for (int i = tid; i < XB; i += 256) sh[i] = 0u;
        __syncthreads();
        for (long long i = g0; i < N; i += T) {
            const u64 key = key_at(i);
            if (top >= 64 || (key >> top) == prefix) atomicAdd(&sh[(unsigned)((key >> shf) & ((1u << dbits) - 1u))], 1u);
        }
        __syncthreads();
        uint32_t* gh = ghist + (size_t)pass * XB;
        for (int i = tid; i < XB; i += 256) {
            const unsigned v = sh[i];
            if (v) atomicAdd(gh + i, v);
        }
        if (!grid_barrier(st, epoch, status)) return;
        // every CTA finds the digit of the r-th key from the merged histogram (8 consecutive bins per thread)
        unsigned v[8];
        unsigned local = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { v[i] = __ldcg(gh + tid * 8 + i); local += v[i]; }
        unsigned incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (tid == 0) s_digit = -1;
        if (lane == 31) wt[warp] = incl;
        __syncthreads();
        long long off = 0;
        for (int w = 0; w < warp; ++w) off += wt[w];
        long long cum = off + incl - local;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (r > cum && r <= cum + (long long)v[i]) { s_digit = tid * 8 + i; s_rnew = r - cum; }
            cum += v[i];
        }
        __syncthreads();
        if (s_digit < 0) {                                    // cannot happen: the counts cover all N keys
            if (tid == 0 && blockIdx.x == 0) latch_error(status, TRIMKV_E_STATE);
            return;
        }
        prefix = (top >= 64 ? 0ull : (prefix << dbits)) | (u64)s_digit;
        r = s_rnew;
        top = shf;
        __syncthreads();
    }
    const u64 tau = prefix;                                   // every key up to tau is evicted
    if (list) {
        for (long long i = g0; i < N; i += T) {
            const u64 key = __ldg(cand + i);
            set_keep(keep_bits, key, key > tau);
        }
    } else {
        const long long words = (n + 63) / 64;
        const long long nchunk = (n + 32 * FJ - 1) / (32 * FJ);
        for (long long c = (long long)blockIdx.x * 8 + warp; c < nchunk; c += (long long)gridDim.x * 8) {
            const long long base = c * (32 * FJ);
            u64 wv = 0ull;
#pragma unroll 1
            for (int j = 0; j < FJ; ++j) {
                const long long idx = base + 32 * j + lane;
                const bool keep = idx < n && flat_key(__ldg(s + idx), (uint32_t)idx) > tau;
                const unsigned kb = __ballot_sync(0xffffffffu, keep);
                if (lane == (j >> 1)) wv |= (u64)kb << (32 * (j & 1));
            }
            const long long wi = c * (FJ / 2) + lane;
            if (lane < FJ / 2 && wi < words) keep_bits[wi] = wv;
        }
    }
    if (blockIdx.x == 0 && tid == 0) stats[0] = mode;
}

// keep_bits for the cases that need no ranking: everything kept, or nothing.
__global__ void flat_fill_kernel(u64* __restrict__ keep_bits, long long n, int keep_all, int32_t* __restrict__ status) {
    const long long words = (n + 63) / 64;
    if (blockIdx.x == 0 && threadIdx.x == 0 && status) *status = 0;
    for (long long w = blockIdx.x * (long long)blockDim.x + threadIdx.x; w < words; w += (long long)gridDim.x * blockDim.x) {
        const long long rem = n - w * 64;
        const u64 valid = rem >= 64 ? ~0ull : ((1ull << rem) - 1ull);
        keep_bits[w] = keep_all ? valid : 0ull;
    }
}

}  // namespace

// ------------------------------------------------------------------ host side
cudaError_t launch_select_flat(const float* scores, long long n, long long k_keep, u64* keep_bits, void* workspace,
                               size_t workspace_bytes, int32_t* status, int distrust, cudaStream_t stream) {
    const long long k_evict = n - std::min<long long>(k_keep, n);
    if (k_evict == 0 || k_evict == n) {
        const long long words = (n + 63) / 64;
        const int grid = (int)std::max<long long>(1, std::min<long long>((words + 255) / 256, 1184));
        flat_fill_kernel<<<grid, 256, 0, stream>>>(keep_bits, n, k_evict == 0, status);
        count_launch();
        return cudaGetLastError();
    }
    char* ws = (char*)workspace;
    FlatState* st = (FlatState*)ws;
    long long* stats = (long long*)(ws + 512);
    uint32_t* hist = (uint32_t*)(ws + 1024);
    uint32_t* ghist = hist;                  // the exact fallback's histograms reuse the space: the candidate histogram is
                                             // dead once the main pass has picked its bin
    u64* cand2 = (u64*)(hist + (size_t)HREP * FB);
    static_assert(X_PASSES * XB <= HREP * FB, "fallback histograms must fit the candidate histogram's space");
    u64* cand = cand2 + CAND2_CAP;
    const long long cand_cap = (long long)((workspace_bytes - FLAT_FIXED_BYTES) / sizeof(u64));
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    // A miss of the sampled bracket costs the exact fallback over all scores (about seven passes), so the margin is wide
    // enough to make it a once-in-tens-of-thousands event, no wider: the bracket's width is what the main pass writes out.
    const float sigmas = 4.0f;
    // 8192 samples keep the bracket under 5 % of the scores (the candidate list has room for 6 %).  Where that is still
    // millions of keys (the largest arrays, threshold away from the ends), a second, 32 times larger sample gathered by
    // many CTAs narrows it about fivefold: the list's traffic and the bits settled later shrink with it.
    int launches = 4;
    {
        const double q = (double)k_evict / (double)n;
        const double width = 2.0 * (sigmas * std::sqrt(q * (1.0 - q) / 8192.0) + 9.0 / 8192.0);
        const bool refine = !distrust && n >= (1LL << 26) && width * (double)n > 2.0e6;
        // where the refinement follows, the first bracket only has to hold the threshold: half the samples do
        u64* samples = cand2 + FB / 2;          // behind the refinement round's histogram, which shares the space of cand2
        const int cap = refine ? 4096 : 8192;
        flat_gather_kernel<<<cap / 256, 256, 0, stream>>>(scores, n, cap, samples, hist, status);
        // every kernel after the first is a dependent launch: it is placed and set up while its predecessor finishes
        if (refine) launch_dependent(flat_bracket_kernel<4>, dim3(1), dim3(1024), 0, stream, samples, n, k_evict, st, stats, sigmas, distrust);
        else launch_dependent(flat_bracket_kernel<8>, dim3(1), dim3(1024), 0, stream, samples, n, k_evict, st, stats, sigmas, distrust);
        ++launches;
        if (refine) {
            launch_dependent(flat_refine_kernel, dim3(REFINE_CTAS), dim3(REFINE_THREADS), 0, stream, scores, n, k_evict, st,
                             hist + (size_t)HREP * FB, stats, sigmas);
            ++launches;
        }
    }
    const long long nchunk = (n + 32 * FJ - 1) / (32 * FJ);
    const int grid2 = (int)std::max<long long>(1, std::min<long long>((nchunk + MAIN_WARPS - 1) / MAIN_WARPS, (long long)sms));
    if (first_use_on_device(2)) cudaFuncSetAttribute(flat_main_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MAIN_SMEM_BYTES);
    launch_dependent(flat_main_kernel, dim3(grid2), dim3(MAIN_THREADS), MAIN_SMEM_BYTES, stream, scores, n, k_evict, st, hist, cand,
                     cand_cap, keep_bits, stats, status);
    const long long expect = n / 24 + 1024;                    // candidates the pass over the list should be sized for
    const int grid3 = (int)std::max<long long>(1, std::min<long long>((expect + 8191) / 8192, (long long)sms));
    launch_dependent(flat_cand_kernel, dim3(grid3), dim3(1024), 0, stream, st, cand, cand2, keep_bits, stats);
    // exact fallback: all CTAs resident at once (cooperative launch), so that its grid barrier is safe
    static int blocks_per_sm[64] = {};
    if (dev >= 0 && dev < 64 && blocks_per_sm[dev] == 0) {
        int nb = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, flat_exact_kernel, 256, 0) != cudaSuccess || nb < 1) nb = 1;
        blocks_per_sm[dev] = std::min(nb, 4);
    }
    const int gridx = sms * ((dev >= 0 && dev < 64) ? blocks_per_sm[dev] : 1);
    const u64* cand_c = cand;
    void* args[] = {(void*)&scores, (void*)&n, (void*)&k_evict, (void*)&st, (void*)&cand_c, (void*)&ghist, (void*)&keep_bits,
                    (void*)&stats, (void*)&status};
    cudaError_t e = cudaLaunchCooperativeKernel((void*)flat_exact_kernel, dim3(gridx), dim3(256), args, 0, stream);
    count_launch(launches);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace tkv
