// Global selection (Sec. 4.2): per sequence, evict the k entries with the lowest retention score
// S = (t + 1 - i) * lambda + c  (log of Eq. (global_score)) under the total order
// (score, then newer position first, then higher layer, then higher head are evicted first).
//
// Every entry maps to a unique 64-bit key whose integer order is the eviction order, so the result is identical
// to a full sort and no floating-point value is compared after key construction.
//
// Cache path (one pass over the metadata): a Bernoulli sample of the sequence's keys brackets the k-th smallest
// key; one filter pass counts the keys below the bracket (marking them in per-page 64-bit eviction masks built with
// warp votes) and collects the keys inside it; one CTA per sequence verifies the bracket and ranks the collected
// keys exactly (radix select on the differing bits).  A bracket that missed (probability below 1e-9) is redone
// exactly by a single-CTA radix select over the whole sequence.
// Flat-array path (standalone selection over fp32 scores): shared-memory histogram passes (4094 equal-width bins,
// first centred on a small sample, then narrowed to the bin that holds the k-th key), filter, exact ranking.
// Fixed per-pool budgets: one CTA per pool ranks that pool's keys exactly.
#include <algorithm>

#include "trimkv_internal.cuh"

namespace tkv {

namespace {

// ------------------------------------------------------------------ key sources
// A source presents its entries as pages of 64; a half-warp reads one page, 4 consecutive entries per lane.
struct CacheSrc {
    static constexpr bool FLAT = false;
    CacheView cv;
    long long t1;   // t + 1
    __device__ long long pages() const { return cv.P_seq; }
    // {pool, logical page, live entries, -}; pool < 0: the page is free
    __device__ int4 info(int b, long long p) const { return __ldg(cv.owner + (size_t)b * cv.P_seq + p); }
    // returns the valid-entry bits (4) of this lane; sc = orderable score (high key word), tie = ~low key word
    __device__ unsigned load4(int b, long long p, int e0, const int4& inf, uint32_t (&sc)[4], uint32_t (&tie)[4]) const {
        if (inf.x < 0 || e0 >= inf.z) return 0u;
        const size_t s = ((size_t)b * cv.P_seq + p) * PAGE + e0;
        const float4 lm = *reinterpret_cast<const float4*>(cv.lam + s);
        const float4 cc = *reinterpret_cast<const float4*>(cv.c + s);
        const int4 ps = *reinterpret_cast<const int4*>(cv.pos + s);
        const float l4[4] = {lm.x, lm.y, lm.z, lm.w};
        const float c4[4] = {cc.x, cc.y, cc.z, cc.w};
        const int p4[4] = {ps.x, ps.y, ps.z, ps.w};
        const int t1i = (int)t1;
        unsigned vm = 0;
        bool bad = false;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float S = retention_score(l4[j], c4[j], (float)(t1i - p4[j]));
            bad |= (S != S) && (e0 + j < inf.z);
            sc[j] = orderable_key(S);
            tie[j] = ((uint32_t)p4[j] << cv.pool_bits) | (uint32_t)inf.x;
            if (e0 + j < inf.z) vm |= 1u << j;
        }
        if (bad) latch_error(cv.err, TRIMKV_E_NONFINITE);
        return vm;
    }
};

struct ArraySrc {
    static constexpr bool FLAT = true;
    const float* s;
    long long n;
    int32_t* err;
    __device__ long long pages() const { return (n + PAGE - 1) / PAGE; }
    __device__ int4 info(int, long long) const { return make_int4(0, 0, PAGE, 0); }
    __device__ unsigned load4(int, long long p, int e0, const int4&, uint32_t (&sc)[4], uint32_t (&tie)[4]) const {
        const long long i0 = p * PAGE + e0;
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        unsigned vm = 0;
        if (i0 + 3 < n) {
            const float4 f = *reinterpret_cast<const float4*>(s + i0);
            v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
            vm = 0xFu;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (i0 + j < n) { v[j] = s[i0 + j]; vm |= 1u << j; }
        }
        bool bad = false;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            bad |= (v[j] != v[j]) && (vm & (1u << j));
            sc[j] = orderable_key(v[j]);
            tie[j] = (uint32_t)(i0 + j);
        }
        if (bad) latch_error(err, TRIMKV_E_NONFINITE);
        return vm;
    }
};

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

// ------------------------------------------------------------------ threshold search (one CTA, 256 threads)
__device__ void threshold_scan(SelState* st, uint32_t* hist_b, long long k, long long n_total, bool last_pass,
                               unsigned cand_target) {
    __shared__ u64 warp_tot[8];
    __shared__ int s_bin;
    __shared__ u64 s_below;
    __shared__ unsigned s_cnt;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int PER = NB / 256;
    uint32_t v[PER];
    u64 local = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int bin = tid * PER + i;
        v[i] = (bin < NB - 1) ? __ldcg(hist_b + bin) : 0u;
        local += v[i];
    }
    u64 incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const u64 t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (tid == 0) s_bin = -1;
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    u64 off = 0, total = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
        const u64 t = warp_tot[w];
        if (w < warp) off += t;
        total += t;
    }
    const u64 excl = off + incl - local;
    const u64 kk = (u64)k;
    if (kk > excl && kk <= excl + local) {
        u64 cum = excl;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            if (kk > cum && kk <= cum + v[i]) { s_bin = tid * PER + i; s_below = cum; s_cnt = v[i]; }
            cum += v[i];
        }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < PER; ++i) hist_b[tid * PER + i] = 0u;     // clean for the next pass / call
    if (tid == 0) {
        const u64 lo = st->lo;
        const int shift = st->shift;
        u64 c_lo, c_hi, below, cnt;
        if (s_bin == 0) {                       // k-th key lies below the binned range
            c_lo = 0; c_hi = lo - 1; below = 0; cnt = s_cnt;
        } else if (s_bin > 0) {
            c_lo = lo + ((u64)(s_bin - 1) << shift);
            const u64 width_m1 = (shift >= 64) ? ~0ull : ((1ull << shift) - 1ull);
            c_hi = (c_lo + width_m1 < c_lo) ? ~0ull : c_lo + width_m1;
            below = s_below; cnt = s_cnt;
        } else {                                // above the binned range
            c_lo = lo + ((u64)REG_BINS << shift);
            c_hi = ~0ull; below = total; cnt = (u64)n_total - total;
        }
        const u64 kmin = __ldcg(&st->kmin), kmax = __ldcg(&st->kmax);   // written by other CTAs' atomics
        if (c_lo < kmin) c_lo = kmin;           // no key lies in [c_lo, kmin): the count below is unchanged
        if (c_hi > kmax) c_hi = kmax;
        st->cand_lo = c_lo;
        st->cand_hi = c_hi;
        st->n_below = (long long)below;
        st->cand_expected = (unsigned)(cnt > 0xffffffffull ? 0xffffffffull : cnt);
        st->passes += 1;
        if (cnt <= (u64)cand_target || c_lo >= c_hi || last_pass) {
            st->resolved = 1;
        } else {
            u64 nlo = c_lo;
            int bits = 64 - __clzll((long long)(c_hi - nlo));
            int nshift = bits > ZOOM_BITS ? bits - ZOOM_BITS : 0;
            if (nshift >= 32) {                 // bins then depend on the score word alone: start them on a score boundary
                nlo &= ~0xffffffffull;
                bits = 64 - __clzll((long long)(c_hi - nlo));
                nshift = bits > ZOOM_BITS ? bits - ZOOM_BITS : 0;
            }
            st->lo = nlo;
            st->shift = nshift;
        }
        st->kmin = ~0ull;
        st->kmax = 0ull;
    }
}

// ------------------------------------------------------------------ pass 1..n: histogram
template <class Src>
__global__ void __launch_bounds__(256)
hist_kernel(Src src, SelState* __restrict__ sel, uint32_t* __restrict__ hist, unsigned int* __restrict__ done,
            long long k, long long n_total, int last_pass, unsigned cand_target) {
    __shared__ uint32_t sh[NB];
    __shared__ u64 s_min[8], s_max[8];
    __shared__ int s_last;
    const int b = blockIdx.y;
    SelState* st = sel + b;
    if (st->resolved) return;
    const u64 lo = st->lo;
    const int shift = st->shift;
    for (int i = threadIdx.x; i < NB; i += blockDim.x) sh[i] = 0u;
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane >> 4, e0 = (lane & 15) * 4;
    const long long P = src.pages();
    const long long chunk = (P + gridDim.x - 1) / gridDim.x;
    const long long p0 = (long long)blockIdx.x * chunk;
    const long long p1 = min(P, p0 + chunk);

    u64 kmin = ~0ull, kmax = 0ull;
    unsigned under = 0;
    int cur_bin = -1;
    unsigned cur_cnt = 0;
    auto tally = [&](const uint32_t (&sc)[4], const uint32_t (&tie)[4], unsigned vm) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (vm & (1u << j)) {
                const u64 key = compose_key(sc[j], tie[j]);
                kmin = key < kmin ? key : kmin;
                kmax = key > kmax ? key : kmax;
                const int bin = bin_of(key, lo, shift);
                if (bin == 0) {
                    ++under;
                } else if (bin < NB - 1) {
                    if (bin == cur_bin) {
                        ++cur_cnt;
                    } else {
                        if (cur_cnt) atomicAdd(&sh[cur_bin], cur_cnt);
                        cur_bin = bin;
                        cur_cnt = 1;
                    }
                }
            }
        }
    };
    bool fast_done = false;
    if constexpr (Src::FLAT) {
        // Flat arrays, bins at least one score step wide and starting on a score boundary: the bin of a key depends on
        // its 32-bit score word alone.  Grid-stride over 16-byte groups, four groups in flight per thread.
        if (shift >= 32 && (lo & 0xffffffffull) == 0ull) {
            const uint32_t lo32 = (uint32_t)(lo >> 32);
            const int sh32 = shift - 32;
            // Most scores fall outside the binned range (it brackets the k-th key): two float compares settle those.
            const u64 end64 = (u64)lo32 + ((u64)REG_BINS << sh32) - 1ull;
            const float lo_f = key_float_lt(lo32);
            const float hi_f = end64 >= 0xffffffffull ? __uint_as_float(0x7f800000u) : key_float_le((uint32_t)end64);
            float fmin_ = __uint_as_float(0x7f800000u), fmax_ = __uint_as_float(0xff800000u);
            bool bad = false;
            // Straight-line per score (no divergent branches: with a sixth of the scores inside the range nearly every
            // warp would run both sides of one anyway): the in-range work is predicated.
            auto one = [&](float x) {
                bad |= (x != x);
                fmin_ = fminf(fmin_, x);
                fmax_ = fmaxf(fmax_, x);
                const bool below = x < lo_f;
                under += below ? 1u : 0u;
                const uint32_t sc = orderable_key(x);
                const uint32_t bi = (sc - lo32) >> sh32;
                if (!below && x <= hi_f && bi < (uint32_t)REG_BINS) atomicAdd(&sh[bi + 1], 1u);
            };
            const long long n4 = src.n >> 2;
            const float4* s4 = reinterpret_cast<const float4*>(src.s);
            const long long T = (long long)gridDim.x * blockDim.x;
            long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
            for (; i + 3 * T < n4; i += 4 * T) {                         // four 16-byte groups in flight per thread
                float4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) v[u] = __ldg(s4 + i + u * T);
#pragma unroll
                for (int u = 0; u < 4; ++u) { one(v[u].x); one(v[u].y); one(v[u].z); one(v[u].w); }
            }
            for (; i < n4; i += T) {
                const float4 v = __ldg(s4 + i);
                one(v.x); one(v.y); one(v.z); one(v.w);
            }
            if (blockIdx.x == 0 && threadIdx.x < (int)(src.n & 3)) one(src.s[(n4 << 2) + threadIdx.x]);
            if (bad) latch_error(src.err, TRIMKV_E_NONFINITE);
            if (fmin_ <= fmax_) {
                kmin = (u64)orderable_key(fmin_) << 32;
                kmax = ((u64)orderable_key(fmax_) << 32) | 0xffffffffull;
            }
            fast_done = true;
        }
    }
    // Each half-warp takes two pages per trip; the page records of the next trip are fetched one trip ahead,
    // so the metadata loads of a trip depend on nothing that is still in flight.
    const long long stride = (long long)(blockDim.x >> 5) * 4;
    long long pp = fast_done ? p1 : p0 + warp * 4;
    int4 infA = make_int4(-1, 0, 0, 0), infB = infA;
    if (pp + sub < p1) infA = src.info(b, pp + sub);
    if (pp + 2 + sub < p1) infB = src.info(b, pp + 2 + sub);
    for (; pp < p1; pp += stride) {
        const long long pgA = pp + sub, pgB = pp + 2 + sub, nx = pp + stride;
        int4 nA = make_int4(-1, 0, 0, 0), nB = nA;
        if (nx + sub < p1) nA = src.info(b, nx + sub);
        if (nx + 2 + sub < p1) nB = src.info(b, nx + 2 + sub);
        uint32_t scA[4], scB[4], tiA[4], tiB[4];
        unsigned vmA = 0, vmB = 0;
        if (pgA < p1) vmA = src.load4(b, pgA, e0, infA, scA, tiA);
        if (pgB < p1) vmB = src.load4(b, pgB, e0, infB, scB, tiB);
        tally(scA, tiA, vmA);
        tally(scB, tiB, vmB);
        infA = nA;
        infB = nB;
    }
    if (cur_cnt) atomicAdd(&sh[cur_bin], cur_cnt);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        under += __shfl_xor_sync(0xffffffffu, under, o);
        const u64 a = __shfl_xor_sync(0xffffffffu, kmin, o);
        const u64 c = __shfl_xor_sync(0xffffffffu, kmax, o);
        kmin = a < kmin ? a : kmin;
        kmax = c > kmax ? c : kmax;
    }
    if (lane == 0) {
        if (under) atomicAdd(&sh[0], under);
        s_min[warp] = kmin;
        s_max[warp] = kmax;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) {
            kmin = s_min[w] < kmin ? s_min[w] : kmin;
            kmax = s_max[w] > kmax ? s_max[w] : kmax;
        }
        if (kmin <= kmax) {
            atomicMin(&st->kmin, kmin);
            atomicMax(&st->kmax, kmax);
        }
    }
    uint32_t* hb = hist + (size_t)b * NB;
    for (int i = threadIdx.x; i < NB - 1; i += blockDim.x) {
        const uint32_t v = sh[i];
        if (v) atomicAdd(hb + i, v);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned ticket = atomicAdd(done + b, 1u);
        s_last = (ticket == gridDim.x - 1);
        if (s_last) done[b] = 0u;
    }
    __syncthreads();
    if (s_last) {
        __threadfence();
        threshold_scan(st, hb, k, n_total, last_pass != 0, cand_target);
    }
}

// ------------------------------------------------------------------ filter: evict masks + candidates
// COUNT_BELOW: also count the keys below the candidate range into st->n_below (the sample-bracket path, where
// that count is not known beforehand).
template <class Src, bool COUNT_BELOW>
__global__ void __launch_bounds__(256)
filter_kernel(Src src, SelState* __restrict__ sel, Cand* __restrict__ cand, long long cand_cap,
              u64* __restrict__ evict_mask, long long mask_stride, int32_t* err) {
    const int b = blockIdx.y;
    SelState* st = sel + b;
    unsigned below = 0;
    const u64 c_lo = st->cand_lo, c_hi = st->cand_hi;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane >> 4, l16 = lane & 15, e0 = l16 * 4;
    const long long P = src.pages();
    const long long chunk = (P + gridDim.x - 1) / gridDim.x;
    const long long p0 = (long long)blockIdx.x * chunk;
    const long long p1 = min(P, p0 + chunk);
    Cand* cb = cand + (size_t)b * cand_cap;

    const uint32_t lo32 = (uint32_t)(c_lo >> 32), hi32 = (uint32_t)(c_hi >> 32);
    auto emit = [&](long long page, const int4& inf, const uint32_t (&sc)[4], const uint32_t (&tie)[4], unsigned vm) {
        // called by all lanes.  Most entries score above the range: one 32-bit compare settles them.
        unsigned ev = 0, cd = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if ((vm & (1u << j)) && sc[j] <= hi32) {
                if (sc[j] < lo32) {
                    ev |= 1u << j;
                } else {
                    const u64 key = compose_key(sc[j], tie[j]);
                    if (key < c_lo) ev |= 1u << j;
                    else if (key <= c_hi) cd |= 1u << j;
                }
            }
        }
        if (__ballot_sync(0xffffffffu, (ev | cd) != 0u) == 0u) {      // nothing evicted, no candidate: clear masks
            if (l16 == 0 && page < p1 && inf.x >= 0) evict_mask[(size_t)b * mask_stride + page] = 0ull;
            return;
        }
        if (COUNT_BELOW) below += __popc(ev);
        // candidates: warp-aggregated append
        const unsigned any = __ballot_sync(0xffffffffu, cd != 0u);
        if (any) {
            const int nc = __popc(cd);
            int incl = nc;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            const int tot = __shfl_sync(0xffffffffu, incl, 31);
            unsigned base = 0;
            if (lane == 0) base = atomicAdd(&st->cand_count, (unsigned)tot);
            base = __shfl_sync(0xffffffffu, base, 0);
            long long w = (long long)base + incl - nc;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (cd & (1u << j)) {
                    if (w < cand_cap) {
                        Cand cnd;
                        cnd.key = compose_key(sc[j], tie[j]);
                        cnd.slot = (u64)(page * PAGE + e0 + j);
                        cb[w] = cnd;
                    } else {
                        latch_error(err, TRIMKV_E_NOMEM);
                    }
                    ++w;
                }
            }
        }
        // 64-bit eviction mask of the page: lanes 0-7 of the half-warp build the low word, 8-15 the high word
        const unsigned nib = ev << (4 * (l16 & 7));
        unsigned wlo = (l16 < 8) ? nib : 0u, whi = (l16 >= 8) ? nib : 0u;
#pragma unroll
        for (int o = 1; o < 16; o <<= 1) {
            wlo |= __shfl_xor_sync(0xffffffffu, wlo, o);
            whi |= __shfl_xor_sync(0xffffffffu, whi, o);
        }
        if (l16 == 0 && page < p1 && inf.x >= 0) evict_mask[(size_t)b * mask_stride + page] = ((u64)whi << 32) | (u64)wlo;
    };
    // Pages are visited from the end of the CTA's range backwards: the histogram pass went forwards, so the
    // most recently read metadata (the likeliest to still sit in L2) comes first.  Warp-uniform trip count.
    const long long stride = (long long)(blockDim.x >> 5) * 4;
    long long pp = p0 + warp * 4;
    const long long span = p1 - p0;
    auto page_of = [&](long long q) { return p0 + (span - 1 - (q - p0)); };   // reversed index
    int4 infA = make_int4(-1, 0, 0, 0), infB = infA;
    if (pp + sub < p1) infA = src.info(b, page_of(pp + sub));
    if (pp + 2 + sub < p1) infB = src.info(b, page_of(pp + 2 + sub));
    for (; pp < p1; pp += stride) {
        const long long qA = pp + sub, qB = pp + 2 + sub, nx = pp + stride;
        int4 nA = make_int4(-1, 0, 0, 0), nB = nA;
        if (nx + sub < p1) nA = src.info(b, page_of(nx + sub));
        if (nx + 2 + sub < p1) nB = src.info(b, page_of(nx + 2 + sub));
        const long long pgA = qA < p1 ? page_of(qA) : p1, pgB = qB < p1 ? page_of(qB) : p1;
        uint32_t scA[4], scB[4], tiA[4], tiB[4];
        unsigned vmA = 0, vmB = 0;
        if (pgA < p1) vmA = src.load4(b, pgA, e0, infA, scA, tiA);
        if (pgB < p1) vmB = src.load4(b, pgB, e0, infB, scB, tiB);
        emit(pgA, infA, scA, tiA, vmA);
        emit(pgB, infB, scB, tiB, vmB);
        infA = nA;
        infB = nB;
    }
    if (COUNT_BELOW) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) below += __shfl_xor_sync(0xffffffffu, below, o);
        if (lane == 0 && below) atomicAdd(reinterpret_cast<unsigned long long*>(&st->n_below), (unsigned long long)below);
    }
}



// Filter pass for flat arrays.  A warp takes 512 consecutive scores per trip; lane l reads elements 32 j + l, so the
// ballot over the lanes for a given j is already 32 consecutive bits of the eviction mask.
constexpr int FBUF = 64;                                 // candidates a warp stages before it takes a slice of the global list

// Appends the warp's staged candidates to the global list (one atomic per flush).
__device__ __noinline__ void flat_flush(Cand* wb, int nbuf, SelState* st, Cand* cb, long long cand_cap, int32_t* err) {
    const int lane = threadIdx.x & 31;
    unsigned wbase = 0;
    if (lane == 0) wbase = atomicAdd(&st->cand_count, (unsigned)nbuf);
    wbase = __shfl_sync(0xffffffffu, wbase, 0);
    for (int i = lane; i < nbuf; i += 32) {
        if ((long long)wbase + i < cand_cap) cb[(long long)wbase + i] = wb[i];
        else latch_error(err, TRIMKV_E_NOMEM);
    }
    __syncwarp();
}

// Stages the candidates of one ballot (cdb: lanes whose score at flat index idx is a candidate); returns the new fill.
__device__ __noinline__ int flat_stage(Cand* wb, int nbuf, unsigned cdb, float x, long long idx, SelState* st, Cand* cb,
                                       long long cand_cap, int32_t* err) {
    const int lane = threadIdx.x & 31;
    const int cnt = __popc(cdb);
    if (nbuf + cnt > FBUF) {
        flat_flush(wb, nbuf, st, cb, cand_cap, err);
        nbuf = 0;
    }
    if (cdb & (1u << lane)) {
        Cand cnd;
        cnd.key = compose_key(orderable_key(x), (uint32_t)idx);
        cnd.slot = (u64)idx;
        wb[nbuf + __popc(cdb & ((1u << lane) - 1u))] = cnd;
    }
    __syncwarp();
    return nbuf + cnt;
}

// WHOLE: the candidate range is made of whole score values (its ends carry no index tie-break), the usual case after
// histogram passes over score words: two float compares decide an entry (a NaN is neither evicted nor a candidate; the
// histogram pass has flagged it).  Otherwise the 64-bit keys are compared.
template <bool WHOLE>
__device__ __forceinline__ void flat_filter_body(const float* __restrict__ s, long long n, SelState* __restrict__ st,
                                                 Cand* __restrict__ cb, long long cand_cap, u64* __restrict__ evict_mask,
                                                 int32_t* err, Cand* wb) {
    constexpr int J = 16;
    const u64 c_lo = st->cand_lo, c_hi = st->cand_hi;
    const uint32_t lo32 = (uint32_t)(c_lo >> 32), hi32 = (uint32_t)(c_hi >> 32);
    const float lo_f = key_float_lt(lo32), hi_f = key_float_le(hi32);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long words = (n + 63) / 64;
    const long long nchunk = (n + 32 * J - 1) / (32 * J);
    const long long W = (long long)gridDim.x * (blockDim.x >> 5);
    int nbuf = 0;                                        // warp-uniform
    auto decide = [&](float x, long long idx, bool& ev, bool& cd) {
        if (WHOLE) {
            ev = x < lo_f;
            cd = !ev && x <= hi_f;
        } else {
            const uint32_t sc = orderable_key(x);
            // one 32-bit compare settles an entry unless its score word equals that of a range end
            ev = sc < lo32;
            cd = !ev && sc <= hi32;
            if (cd && (sc == lo32 || sc == hi32)) {
                const u64 key = compose_key(sc, (uint32_t)idx);
                ev = key < c_lo;
                cd = !ev && key <= c_hi;
            }
        }
    };
    for (long long c = (long long)blockIdx.x * (blockDim.x >> 5) + warp; c < nchunk; c += W) {
        const long long base = c * (32 * J);
        const long long rem = n - base;                  // elements left from the start of this chunk
        const float* p = s + base + lane;
        float x[J];
        unsigned evb[J];
        if (rem >= 32 * J) {
#pragma unroll
            for (int j = 0; j < J; ++j) x[j] = __ldg(p + 32 * j);
#pragma unroll
            for (int j = 0; j < J; ++j) {
                bool ev, cd;
                decide(x[j], base + 32 * j + lane, ev, cd);
                evb[j] = __ballot_sync(0xffffffffu, ev);
                const unsigned cdb = __ballot_sync(0xffffffffu, cd);
                if (cdb) nbuf = flat_stage(wb, nbuf, cdb, x[j], base + 32 * j + lane, st, cb, cand_cap, err);
            }
        } else {                                         // the ragged last chunk
#pragma unroll 1
            for (int j = 0; j < J; ++j) {
                const bool live = 32 * j + lane < rem;
                const float xv = live ? __ldg(p + 32 * j) : 0.0f;
                bool ev, cd;
                decide(xv, base + 32 * j + lane, ev, cd);
                ev = ev && live;
                cd = cd && live;
                const unsigned e = __ballot_sync(0xffffffffu, ev);
#pragma unroll
                for (int q = 0; q < J; ++q)
                    if (q == j) evb[q] = e;
                const unsigned cdb = __ballot_sync(0xffffffffu, cd);
                if (cdb) nbuf = flat_stage(wb, nbuf, cdb, xv, base + 32 * j + lane, st, cb, cand_cap, err);
            }
        }
        if (lane < J / 2) {
            // word `lane` of this chunk = ballots 2 * lane (low half) and 2 * lane + 1 (high half)
            u64 wv = 0ull;
#pragma unroll
            for (int j = 0; j < J / 2; ++j)
                if (lane == j) wv = (u64)evb[2 * j] | ((u64)evb[2 * j + 1] << 32);
            const long long wi = c * (J / 2) + lane;
            if (wi < words) evict_mask[wi] = wv;
        }
    }
    if (nbuf > 0) flat_flush(wb, nbuf, st, cb, cand_cap, err);
}

__global__ void __launch_bounds__(256, 4)                // the grid is sized for four CTAs per SM
flat_filter_kernel(const float* __restrict__ s, long long n, SelState* __restrict__ st, Cand* __restrict__ cb,
                   long long cand_cap, u64* __restrict__ evict_mask, int32_t* err) {
    // Candidates go through a per-warp buffer so that the single global counter sees one atomic per ~50 candidates
    // (a quarter of a million same-address atomics would serialise the whole pass).
    __shared__ Cand sbuf[8][FBUF];
    Cand* wb = sbuf[threadIdx.x >> 5];
    const u64 c_lo = st->cand_lo, c_hi = st->cand_hi;
    if ((c_lo & 0xffffffffull) == 0ull && (c_hi & 0xffffffffull) == 0xffffffffull)
        flat_filter_body<true>(s, n, st, cb, cand_cap, evict_mask, err, wb);
    else
        flat_filter_body<false>(s, n, st, cb, cand_cap, evict_mask, err, wb);
}

// ------------------------------------------------------------------ sample bracket (cache path)
// One full pass suffices when a candidate range that surely holds the k-th smallest key is known beforehand.
// A Bernoulli sample of the sequence's keys (a hash of the slot decides, about SAMPLE_MEAN keys) is sorted by one
// CTA; the sample keys at ranks k*p -+ a margin of several standard deviations bound the range.  The filter pass
// then counts the keys below the range, and the exact ranking verifies that the k-th key lay inside; if it did
// not (probability below 1e-9 per call), a single-CTA exact selection redoes the sequence.
constexpr int SAMPLE_CAP = 4096;
constexpr int SAMPLE_MEAN = 3072;

__device__ __forceinline__ uint32_t mix32(uint32_t x) {   // integer finaliser: spreads slot indices over 32 bits
    x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
    return x;
}

// Bernoulli sample of the live slots with probability p each.  sub = 0: every live slot is taken (small sequences).
// Otherwise a thread owns a block of `sub` consecutive slots of a page (sub a power of two, sub * p <= 1/2): it takes
// the block with probability sub * p (thresh / 2^32) and then one slot of it uniformly; a slot beyond the page's fill
// is simply not sampled, so every live slot has probability p.
__global__ void __launch_bounds__(256)
sample_kernel(CacheSrc src, SelState* __restrict__ sel, u64* __restrict__ sample, int sub, uint32_t thresh,
              uint32_t seed, int skip_newest) {
    const int b = blockIdx.y;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int per_page = sub > 0 ? PAGE / sub : 1;
    const long long page = gid / per_page;
    if (page >= src.cv.P_seq) return;
    const int4 inf = src.info(b, page);
    if (inf.x < 0) return;
    SelState* st = sel + b;
    const CacheView& cv = src.cv;
    // skip_newest > 0: the last skip_newest entries of every pool have no retention terms yet (their gate is still
    // running); they are left out of the sample, which only has to be representative
    const int live = skip_newest > 0 ? cv.len[(size_t)b * cv.L * cv.H + inf.x] - skip_newest : 0x7fffffff;
    auto take = [&](int off) {
        if (inf.y * PAGE + off >= live) return;
        const size_t s = ((size_t)b * cv.P_seq + page) * PAGE + off;
        const int pos = cv.pos[s];
        const float S = retention_score(cv.lam[s], cv.c[s], (float)(src.t1 - (long long)pos));
        const uint32_t tie = ((uint32_t)pos << cv.pool_bits) | (uint32_t)inf.x;
        const unsigned w = atomicAdd(&st->sample_count, 1u);
        if (w < SAMPLE_CAP) sample[(size_t)b * SAMPLE_CAP + w] = make_key(S, tie);
    };
    if (sub == 0) {
        for (int off = 0; off < inf.z; ++off) take(off);
        return;
    }
    const int blk = (int)(gid % per_page);
    if (blk * sub >= inf.z) return;
    const uint32_t base = (uint32_t)gid * 0x9E3779B1u + seed + (uint32_t)b * 0x85EBCA77u;
    if (mix32(base) < thresh) {
        const int off = blk * sub + (int)(mix32(base ^ 0x68E31DA4u) & (uint32_t)(sub - 1));
        if (off < inf.z) take(off);
    }
}

// One CTA per sequence: ranks the sample by radix descent (each thread keeps its sample keys in registers) and
// sets the candidate range [cand_lo, cand_hi].  The descent stops early once the bin that holds the wanted rank is
// nearly empty and then takes the bin's outer edge, which only widens the range.
__global__ void __launch_bounds__(1024)
bracket_kernel(SelState* __restrict__ sel, const u64* __restrict__ sample, long long k_evict, long long n_total,
               int distrust, float sigmas) {
    constexpr int DB = 11, NBIN = 1 << DB, PER = SAMPLE_CAP / 1024;
    __shared__ unsigned hist[NBIN];
    __shared__ unsigned wtot[32];
    __shared__ u64 s_or[32], s_and[32];
    __shared__ u64 s_prefix;
    __shared__ long long s_r;
    __shared__ unsigned s_cnt;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    SelState* st = sel + b;
    const unsigned raw = st->sample_count;
    const int ns = (int)min(raw, (unsigned)SAMPLE_CAP);
    u64 key[PER];
    u64 vor = 0ull, vand = ~0ull;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int idx = tid + i * 1024;
        key[i] = idx < ns ? sample[(size_t)b * SAMPLE_CAP + idx] : ~0ull;
        if (idx < ns) { vor |= key[i]; vand &= key[i]; }
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
    const int top0 = (ns > 0 && diff) ? 64 - __clzll((long long)diff) : 0;   // low bits in which the sample keys differ

    // Key bound for sample rank r (1-based, 1 <= r <= ns): the lower (upper = false) or upper edge of the finest
    // bin the descent reaches; exact when the descent runs to the last bit.
    auto bound_of_rank = [&](long long r, bool upper) -> u64 {
        int top = top0;
        u64 prefix = top >= 64 ? 0ull : (vor >> top);
        while (top > 0) {
            const int dbits = top < DB ? top : DB;
            const int sh = top - dbits;
            hist[tid] = 0u;
            hist[tid + 1024] = 0u;
            __syncthreads();
#pragma unroll
            for (int i = 0; i < PER; ++i) {
                const bool live = tid + i * 1024 < ns;
                const bool match = live && (top >= 64 ? true : ((key[i] >> top) == prefix));
                if (match) atomicAdd(&hist[(unsigned)((key[i] >> sh) & ((1u << dbits) - 1u))], 1u);
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
                s_cnt = h0;
            } else if (r > excl + h0 && r <= excl + h0 + h1) {
                s_prefix = (top >= 64 ? 0ull : (prefix << dbits)) | (u64)(2 * tid + 1);
                s_r = r - excl - h0;
                s_cnt = h1;
            }
            __syncthreads();
            prefix = s_prefix;
            r = s_r;
            top = sh;
            const unsigned cnt = s_cnt;
            __syncthreads();
            if (cnt <= 2u) break;
        }
        if (top == 0) return prefix;
        return upper ? ((prefix << top) | ((1ull << top) - 1ull)) : (prefix << top);
    };

    u64 lo = 0ull, hi = ~0ull;
    if (ns > 0 && !distrust) {
        long long r_lo, r_hi;
        if ((long long)raw == n_total) {              // every key was sampled: the k-th smallest is known exactly
            r_lo = r_hi = k_evict;
        } else {
            const double mu = (double)k_evict * (double)ns / (double)n_total;   // expected sample rank of the k-th key
            const double dev = (double)sigmas * sqrt(mu) + 8.0;  // margin in standard deviations of the sample rank
            r_lo = (long long)floor(mu - dev);
            r_hi = (long long)ceil(mu + dev) + 1;
        }
        if (r_lo >= 1) lo = bound_of_rank(min(r_lo, (long long)ns), false);
        if (r_hi <= ns) hi = bound_of_rank(max(r_hi, 1LL), true);
    } else if (distrust) {
        lo = hi = ~0ull;        // test hook: a range that cannot hold the k-th key, so that the exact redo runs
    }
    if (tid == 0) {
        st->cand_lo = lo;
        st->cand_hi = hi;
        st->n_below = 0;
        st->cand_count = 0;
        st->cand_expected = 0;
        st->resolved = 0;
        st->passes = ns;
    }
}

// ------------------------------------------------------------------ exact ranking of the candidates
// One CTA per sequence.  STRICT (histogram path): the candidate range is known to hold the k-th key; any
// inconsistency is an internal error.  Otherwise (sample-bracket path): an inconsistent count means the range
// missed; resolved stays 0 and the exact redo kernel takes over.
template <bool STRICT>
__global__ void __launch_bounds__(1024)
resolve_kernel(SelState* __restrict__ sel, Cand* __restrict__ cand, long long cand_cap, u64* __restrict__ evict_mask,
               long long mask_stride, long long k_evict, unsigned next_aim, long long* __restrict__ stats,
               int32_t* __restrict__ cursor, int32_t* err) {
    constexpr int DB = 11, NBIN = 1 << DB;
    __shared__ unsigned hist[NBIN];
    __shared__ unsigned wtot[32];
    __shared__ u64 s_or[32], s_and[32];
    __shared__ u64 s_prefix;
    __shared__ long long s_r;
    __shared__ int s_found;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    SelState* st = sel + b;
    const Cand* cb = cand + (size_t)b * cand_cap;
    const long long craw = (long long)st->cand_count;
    const long long C = min(craw, cand_cap);
    long long r = k_evict - st->n_below;
    const bool ok = r >= 0 && r <= C && craw <= cand_cap && (!STRICT || (long long)st->cand_expected == craw);
    const int sample_n = st->passes;
    if (!ok) {
        if (STRICT) {
            if (tid == 0) latch_error(err, TRIMKV_E_STATE);
            r = r < 0 ? 0 : (r > C ? C : r);
        } else {
            if (tid == 0) {
                st->resolved = 0;
                st->sample_count = 0;
                if (stats) { stats[b * 4 + 0] = 1; stats[b * 4 + 1] = C; stats[b * 4 + 2] = k_evict; stats[b * 4 + 3] = sample_n; }
                if (cursor) cursor[b] = 0;
            }
            return;
        }
    }
    u64 tau = 0ull;
    if (r > 0) {
        // Candidate keys are kept in registers when they fit (the usual case); otherwise each sweep re-reads them.
        constexpr int PER = 8;
        const bool inreg = C <= (long long)PER * 1024;
        u64 kr[PER];
        if (inreg) {
#pragma unroll
            for (int i = 0; i < PER; ++i) {
                const long long idx = tid + (long long)i * 1024;
                kr[i] = idx < C ? cb[idx].key : 0ull;
            }
        }
        // bits in which the candidate keys differ
        u64 vor = 0ull, vand = ~0ull;
        if (inreg) {
#pragma unroll
            for (int i = 0; i < PER; ++i)
                if (tid + (long long)i * 1024 < C) { vor |= kr[i]; vand &= kr[i]; }
        } else {
            for (long long i = tid; i < C; i += blockDim.x) {
                const u64 key = cb[i].key;
                vor |= key;
                vand &= key;
            }
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
        int top = diff ? 64 - __clzll((long long)diff) : 0;    // number of low bits that differ
        u64 prefix = top >= 64 ? 0ull : (vor >> top);
        while (top > 0) {
            const int dbits = top < DB ? top : DB;
            const int sh = top - dbits;
            hist[tid] = 0u;
            hist[tid + 1024] = 0u;
            if (tid == 0) s_found = 0;
            __syncthreads();
            auto count = [&](u64 key) {
                const bool match = top >= 64 ? true : ((key >> top) == prefix);
                if (match) atomicAdd(&hist[(unsigned)((key >> sh) & ((1u << dbits) - 1u))], 1u);
            };
            if (inreg) {
#pragma unroll
                for (int i = 0; i < PER; ++i)
                    if (tid + (long long)i * 1024 < C) count(kr[i]);
            } else {
                for (long long i = tid; i < C; i += blockDim.x) count(cb[i].key);
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
                s_found = (int)h0;
            } else if (r > excl + h0 && r <= excl + h0 + h1) {
                s_prefix = (top >= 64 ? 0ull : (prefix << dbits)) | (u64)(2 * tid + 1);
                s_r = r - excl - h0;
                s_found = (int)h1;
            }
            __syncthreads();
            const int found = s_found;
            if (!found) {                            // cannot happen with consistent counts
                if (tid == 0) latch_error(err, TRIMKV_E_STATE);
                break;
            }
            prefix = s_prefix;
            r = s_r;
            top = sh;
            __syncthreads();
            if (found == 1 && top > 0) {             // one key left under this prefix: it is the r-th smallest
                auto pick = [&](u64 key) { if ((key >> top) == prefix) s_prefix = key; };
                if (inreg) {
#pragma unroll
                    for (int i = 0; i < PER; ++i)
                        if (tid + (long long)i * 1024 < C) pick(kr[i]);
                } else {
                    for (long long i = tid; i < C; i += blockDim.x) pick(cb[i].key);
                }
                __syncthreads();
                prefix = s_prefix;
                top = 0;
            }
        }
        tau = prefix;   // the r-th smallest candidate key: everything <= tau is evicted
        for (long long i = tid; i < C; i += blockDim.x) {
            const Cand cnd = cb[i];
            if (cnd.key <= tau)
                atomicOr(evict_mask + (size_t)b * mask_stride + (cnd.slot >> 6), 1ull << (cnd.slot & 63));
        }
    } else {
        tau = st->cand_lo;
    }
    __syncthreads();
    if (tid == 0) {
        if (stats) {
            stats[b * 4 + 0] = STRICT ? st->passes : 0;
            stats[b * 4 + 1] = C;
            stats[b * 4 + 2] = k_evict;
            stats[b * 4 + 3] = STRICT ? st->shift : sample_n;
        }
        if (STRICT) {
            // centre the next call's first histogram on this threshold; aim for ~next_aim candidates
            int shift = st->shift;
            const int want = 31 - __clz((int)max(next_aim, 1u));
            const int have = 31 - __clz((int)max((unsigned)min(C, 0x7fffffffLL), 1u));
            shift += want - have;
            shift = shift < 0 ? 0 : (shift > INIT_SHIFT ? INIT_SHIFT : shift);
            const u64 half = (u64)(REG_BINS / 2) << shift;
            st->lo = tau > half ? tau - half : 0ull;
            st->shift = shift;
            st->resolved = 0;
            st->passes = 0;
        } else {
            st->resolved = 1;
        }
        st->cand_count = 0;
        st->sample_count = 0;
        st->kmin = ~0ull;
        st->kmax = 0ull;
        if (cursor) cursor[b] = 0;
    }
}

// Exact redo for a sequence whose sample bracket missed: one CTA radix-selects the k-th smallest key over all of
// the sequence's entries (DB bits per sweep) and rewrites every eviction mask.  Slow and rare.
__global__ void __launch_bounds__(1024)
redo_kernel(CacheSrc src, SelState* __restrict__ sel, u64* __restrict__ evict_mask, long long mask_stride,
            long long k_evict, int32_t* err) {
    constexpr int DB = 11, NBIN = 1 << DB;
    __shared__ unsigned hist[NBIN];
    __shared__ unsigned wtot[32];
    __shared__ u64 s_prefix;
    __shared__ long long s_r;
    __shared__ int s_found;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    SelState* st = sel + b;
    if (st->resolved) return;
    const int sub = lane >> 4, l16 = lane & 15, e0 = l16 * 4;
    const long long P = src.pages();
    u64 prefix = 0ull;
    long long r = k_evict;
    int top = 64;
    while (top > 0) {
        const int dbits = top < DB ? top : DB;
        const int sh = top - dbits;
        hist[tid] = 0u;
        hist[tid + 1024] = 0u;
        if (tid == 0) s_found = 0;
        __syncthreads();
        for (long long pp = warp * 2; pp < P; pp += 64) {
            const long long page = pp + sub;
            if (page < P) {
                const int4 inf = src.info(b, page);
                uint32_t sc[4], tie[4];
                const unsigned vm = src.load4(b, page, e0, inf, sc, tie);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (vm & (1u << j)) {
                        const u64 key = compose_key(sc[j], tie[j]);
                        const bool match = top >= 64 ? true : ((key >> top) == prefix);
                        if (match) atomicAdd(&hist[(unsigned)((key >> sh) & ((1u << dbits) - 1u))], 1u);
                    }
                }
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
        if (!s_found) {
            if (tid == 0) latch_error(err, TRIMKV_E_STATE);
            return;
        }
        prefix = s_prefix;
        r = s_r;
        top = sh;
        __syncthreads();
    }
    const u64 tau = prefix;
    for (long long pp = warp * 2; pp < P; pp += 64) {          // warp-uniform trip count
        const long long page = pp + sub;
        int4 inf = make_int4(-1, 0, 0, 0);
        uint32_t sc[4], tie[4];
        unsigned vm = 0;
        if (page < P) {
            inf = src.info(b, page);
            vm = src.load4(b, page, e0, inf, sc, tie);
        }
        unsigned ev = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if ((vm & (1u << j)) && compose_key(sc[j], tie[j]) <= tau) ev |= 1u << j;
        const unsigned nib = ev << (4 * (l16 & 7));
        unsigned wlo = (l16 < 8) ? nib : 0u, whi = (l16 >= 8) ? nib : 0u;
#pragma unroll
        for (int o = 1; o < 16; o <<= 1) {
            wlo |= __shfl_xor_sync(0xffffffffu, wlo, o);
            whi |= __shfl_xor_sync(0xffffffffu, whi, o);
        }
        if (l16 == 0 && page < P && inf.x >= 0) evict_mask[(size_t)b * mask_stride + page] = ((u64)whi << 32) | (u64)wlo;
    }
    if (tid == 0) st->resolved = 1;
}

// Flat arrays: centres the first histogram pass on the threshold.  4096 evenly spaced scores are sampled and ranked by
// bracket_kernel exactly as for the cache path; the bracket of the k-th key (a tenth of the key range or less) becomes
// the binned range of the first pass, whose bins are then fine enough to settle the selection at once.  Any range is
// correct: keys outside it fall into the catch-all bins and cost a further pass at worst.
__global__ void __launch_bounds__(1024)
flat_sample_kernel(const float* __restrict__ s, long long n, SelState* __restrict__ st, u64* __restrict__ sample) {
    const int gid = blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= SAMPLE_CAP) return;
    const long long step = n / SAMPLE_CAP > 0 ? n / SAMPLE_CAP : 1;
    const long long idx = (long long)gid * step;
    if (idx >= n) return;
    const float x = s[idx];
    if (x != x) return;                                   // NaN is reported by the histogram pass
    const unsigned w = atomicAdd(&st->sample_count, 1u);
    const u64 key = compose_key(orderable_key(x), (uint32_t)idx);
    if (w < SAMPLE_CAP) sample[w] = key;
    atomicMin(&st->kmin, key);                            // smallest sampled key: lower end when the bracket has none
}

__global__ void flat_range_kernel(SelState* __restrict__ st) {
    u64 c_lo = st->cand_lo;
    const u64 c_hi = st->cand_hi, smin = st->kmin;
    st->passes = 0;
    st->sample_count = 0;
    st->kmin = ~0ull;                                     // as the histogram pass expects it
    if (c_lo == 0ull && smin < c_hi) {                    // bracket open below: start a little under the sampled minimum
        const u64 pad = (c_hi - smin) / 8 + 1;
        c_lo = smin > pad ? smin - pad : 0ull;
    }
    if (c_hi <= c_lo) return;                             // keep the full-range default
    u64 lo = c_lo;
    int bits = 64 - __clzll((long long)(c_hi - lo));
    int shift = bits > ZOOM_BITS ? bits - ZOOM_BITS : 0;
    if (shift >= 32) {                                    // bins depend on the score word alone: start on a score boundary
        lo &= ~0xffffffffull;
        bits = 64 - __clzll((long long)(c_hi - lo));
        shift = bits > ZOOM_BITS ? bits - ZOOM_BITS : 0;
    }
    st->lo = lo;
    st->shift = shift;
}

// ------------------------------------------------------------------ fixed per-pool budget (TrimKV arm)
// One CTA per pool: the pool keeps its `keep` best entries on its own.  The keys of the pool (up to 8192; longer pools
// re-read their metadata every sweep) sit in registers; a radix descent over the bits in which they differ finds the
// k-th smallest key exactly, then every entry with a key up to it is flagged in its page's eviction mask.
__global__ void __launch_bounds__(256)
pool_select_kernel(CacheView cv, long long t1, int keep) {
    constexpr int DB = 9, NBIN = 1 << DB, PER = 32;
    __shared__ unsigned hist[NBIN];
    __shared__ unsigned wtot[8];
    __shared__ u64 s_or[8], s_and[8];
    __shared__ u64 s_prefix;
    __shared__ long long s_r;
    __shared__ int s_found;
    const long long pool = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = (int)(pool / ((long long)cv.L * cv.H));
    const int pool_local = (int)(pool % ((long long)cv.L * cv.H));
    const int n = cv.len[pool];
    const int32_t* bt = cv.block_table + pool * cv.maxpp;
    u64* masks = cv.evict_mask + (size_t)b * cv.P_seq;
    const int np = (n + PAGE - 1) / PAGE;
    for (int lp = tid; lp < np; lp += blockDim.x) masks[bt[lp]] = 0ull;
    if (n <= keep) return;
    long long r = n - keep;                                      // evict the r smallest keys
    const int t1i = (int)t1;
    auto key_of = [&](int idx) -> u64 {
        const size_t slot = ((size_t)b * cv.P_seq + bt[idx / PAGE]) * PAGE + idx % PAGE;
        const int pos = cv.pos[slot];
        const float S = retention_score(cv.lam[slot], cv.c[slot], (float)(t1i - pos));
        if (S != S) latch_error(cv.err, TRIMKV_E_NONFINITE);
        return make_key(S, ((uint32_t)pos << cv.pool_bits) | (uint32_t)pool_local);
    };
    const bool inreg = n <= PER * 256;
    u64 kr[PER];
    u64 vor = 0ull, vand = ~0ull;
    if (inreg) {
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int idx = tid + i * 256;
            kr[i] = 0ull;
            if (idx < n) { kr[i] = key_of(idx); vor |= kr[i]; vand &= kr[i]; }
        }
    } else {
        for (int idx = tid; idx < n; idx += 256) { const u64 k = key_of(idx); vor |= k; vand &= k; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        vor |= __shfl_xor_sync(0xffffffffu, vor, o);
        vand &= __shfl_xor_sync(0xffffffffu, vand, o);
    }
    if (lane == 0) { s_or[warp] = vor; s_and[warp] = vand; }
    __syncthreads();
    vor = 0ull; vand = ~0ull;
    for (int w = 0; w < 8; ++w) { vor |= s_or[w]; vand &= s_and[w]; }
    const u64 diff = vor ^ vand;
    int top = diff ? 64 - __clzll((long long)diff) : 0;
    u64 prefix = top >= 64 ? 0ull : (vor >> top);
    while (top > 0) {
        const int dbits = top < DB ? top : DB;
        const int sh = top - dbits;
        hist[tid] = 0u;
        hist[tid + 256] = 0u;
        if (tid == 0) s_found = 0;
        __syncthreads();
        auto count = [&](u64 key) {
            const bool match = top >= 64 ? true : ((key >> top) == prefix);
            if (match) atomicAdd(&hist[(unsigned)((key >> sh) & ((1u << dbits) - 1u))], 1u);
        };
        if (inreg) {
#pragma unroll
            for (int i = 0; i < PER; ++i)
                if (tid + i * 256 < n) count(kr[i]);
        } else {
            for (int idx = tid; idx < n; idx += 256) count(key_of(idx));
        }
        __syncthreads();
        const unsigned h0 = hist[2 * tid], h1 = hist[2 * tid + 1];
        unsigned incl = h0 + h1;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned tt = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += tt;
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
        if (!s_found) {                                          // cannot happen: the counts cover all n keys
            if (tid == 0) latch_error(cv.err, TRIMKV_E_STATE);
            return;
        }
        prefix = s_prefix;
        r = s_r;
        top = sh;
        __syncthreads();
    }
    const u64 tau = prefix;                                      // the r-th smallest key of the pool
    auto flag = [&](int idx, u64 key) {
        if (key <= tau) atomicOr(masks + bt[idx / PAGE], 1ull << (idx % PAGE));
    };
    if (inreg) {
#pragma unroll
        for (int i = 0; i < PER; ++i)
            if (tid + i * 256 < n) flag(tid + i * 256, kr[i]);
    } else {
        for (int idx = tid; idx < n; idx += 256) flag(idx, key_of(idx));
    }
}

__global__ void state_init_kernel(SelState* sel, int B) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    SelState s;
    s.lo = 0ull; s.kmin = ~0ull; s.kmax = 0ull; s.cand_lo = 0ull; s.cand_hi = 0ull; s.n_below = 0;
    s.shift = INIT_SHIFT; s.resolved = 0; s.passes = 0; s.cand_count = 0; s.cand_expected = 0; s.sample_count = 0;
    sel[b] = s;
}

__global__ void invert_mask_kernel(const u64* __restrict__ ev, u64* __restrict__ keep, long long n) {
    const long long words = (n + 63) / 64;
    for (long long w = blockIdx.x * (long long)blockDim.x + threadIdx.x; w < words;
         w += (long long)gridDim.x * blockDim.x) {
        const long long rem = n - w * 64;
        const u64 valid = rem >= 64 ? ~0ull : ((1ull << rem) - 1ull);
        keep[w] = ~ev[w] & valid;
    }
}

int grid_x_for(long long pages, int B) {
    long long g = (pages + 31) / 32;              // at least ~32 pages per CTA
    long long cap = (592 + B - 1) / B;            // ~4 CTAs per SM over the whole grid
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

// Histogram path (flat arrays): up to max_passes histogram passes, filter, exact resolve.
void run_select_flat(const ArraySrc& src, const SelectBuffers& sb, long long k_evict, int max_passes, unsigned cand_target,
                     u64* evict_mask, int32_t* err, cudaStream_t st) {
    const long long pages = (src.n + PAGE - 1) / PAGE;
    dim3 grid(grid_x_for(pages, 1), 1);
    for (int p = 0; p < max_passes; ++p)
        hist_kernel<ArraySrc><<<grid, 256, 0, st>>>(src, sb.sel, sb.hist, sb.done, k_evict, src.n, p == max_passes - 1,
                                                    cand_target);
    flat_filter_kernel<<<grid, 256, 0, st>>>(src.s, src.n, sb.sel, sb.cand, sb.cand_cap, evict_mask, err);
    resolve_kernel<true><<<1, 1024, 0, st>>>(sb.sel, sb.cand, sb.cand_cap, evict_mask, pages, k_evict,
                                             max(cand_target / 8u, 1u), sb.stats, nullptr, err);
    count_launch(max_passes + 2);
}

}  // namespace

void launch_select_state_init(SelState* sel, int B, cudaStream_t st) {
    state_init_kernel<<<(B + 127) / 128, 128, 0, st>>>(sel, B);
    count_launch();
}

void launch_select_cache_sample(const CacheView& cv, const SelectBuffers& sb, long long t, long long n_total,
                                long long k_evict, int skip_newest, int distrust_sample, cudaStream_t st) {
    CacheSrc src;
    src.cv = cv;
    src.t1 = t + 1;
    int sub = 0;                                         // 0: sample every key
    uint32_t thresh = 0xffffffffu;
    if (n_total > SAMPLE_MEAN) {
        const double p = (double)SAMPLE_MEAN / (double)n_total;
        sub = PAGE;
        while (sub > 1 && p * sub > 0.5) sub >>= 1;
        thresh = (uint32_t)(4294967296.0 * std::min(p * sub, 0.999999));
    }
    const uint32_t seed = (uint32_t)t * 0x9E3779B1u + 0x1234567u;
    const long long threads = cv.P_seq * (sub > 0 ? PAGE / sub : 1);
    dim3 gs((unsigned)((threads + 255) / 256), cv.B);
    sample_kernel<<<gs, 256, 0, st>>>(src, sb.sel, sb.sample, sub, thresh, seed, skip_newest);
    // 7 sigma: a miss costs the single-CTA exact redo of the whole sequence, so it must be next to impossible
    bracket_kernel<<<cv.B, 1024, 0, st>>>(sb.sel, sb.sample, k_evict, n_total, distrust_sample, 7.0f);
    count_launch(2);
}

void launch_select_cache_rest(const CacheView& cv, const SelectBuffers& sb, long long t, long long k_evict,
                              int32_t* compact_cursor, cudaStream_t st) {
    CacheSrc src;
    src.cv = cv;
    src.t1 = t + 1;
    dim3 grid(grid_x_for(cv.P_seq, cv.B), cv.B);
    filter_kernel<CacheSrc, true><<<grid, 256, 0, st>>>(src, sb.sel, sb.cand, sb.cand_cap, cv.evict_mask, cv.P_seq, cv.err);
    resolve_kernel<false><<<cv.B, 1024, 0, st>>>(sb.sel, sb.cand, sb.cand_cap, cv.evict_mask, cv.P_seq, k_evict, 0u,
                                                 sb.stats, compact_cursor, cv.err);
    redo_kernel<<<cv.B, 1024, 0, st>>>(src, sb.sel, cv.evict_mask, cv.P_seq, k_evict, cv.err);
    count_launch(3);
}

void launch_select_cache(const CacheView& cv, const SelectBuffers& sb, long long t, long long n_total,
                         long long k_evict, int32_t* compact_cursor, int distrust_sample, cudaStream_t st) {
    launch_select_cache_sample(cv, sb, t, n_total, k_evict, 0, distrust_sample, st);
    launch_select_cache_rest(cv, sb, t, k_evict, compact_cursor, st);
}

void launch_select_pools(const CacheView& cv, long long t, int keep_per_pool, int32_t* compact_cursor, cudaStream_t st) {
    const long long pools = (long long)cv.B * cv.L * cv.H;
    cudaMemsetAsync(compact_cursor, 0, (size_t)cv.B * sizeof(int32_t), st);
    pool_select_kernel<<<(unsigned)pools, 256, 0, st>>>(cv, t + 1, keep_per_pool);
    count_launch();
}

void launch_select_array(const float* scores, long long n, long long k_evict, u64* evict_mask, const SelectBuffers& sb,
                         int32_t* err, cudaStream_t st) {
    ArraySrc src;
    src.s = scores;
    src.n = n;
    src.err = err;
    u64* sample = reinterpret_cast<u64*>(sb.cand);        // the candidate buffer is idle until the filter pass
    flat_sample_kernel<<<SAMPLE_CAP / 1024, 1024, 0, st>>>(scores, n, sb.sel, sample);
    // 4 sigma: here a miss (6e-5 per call) only costs one more histogram pass, and the narrower range keeps the
    // candidate list of the last bin within what the resolution holds in registers
    bracket_kernel<<<1, 1024, 0, st>>>(sb.sel, sample, k_evict, n, 0, 4.0f);
    flat_range_kernel<<<1, 1, 0, st>>>(sb.sel);
    count_launch(3);
    run_select_flat(src, sb, k_evict, 7, (unsigned)sb.cand_cap, evict_mask, err, st);
}

void launch_invert_mask(const u64* evict_mask, u64* keep_bits, long long n, cudaStream_t st) {
    const long long words = (n + 63) / 64;
    int grid = (int)((words + 255) / 256);
    if (grid > 1184) grid = 1184;
    if (grid < 1) grid = 1;
    invert_mask_kernel<<<grid, 256, 0, st>>>(evict_mask, keep_bits, n);
    count_launch();
}

}  // namespace tkv
