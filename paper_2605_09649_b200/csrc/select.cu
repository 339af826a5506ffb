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
// (The standalone selection over a flat score array lives in select_flat.cu.)
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
    int skip_newest = 0;   // > 0: leave out the last skip_newest entries of every pool (their retention terms are not written yet)
    __device__ long long pages() const { return cv.P_seq; }
    // {pool, logical page, live entries, -}; pool < 0: the page is free
    __device__ int4 info(int b, long long p) const { return __ldg(cv.owner + (size_t)b * cv.P_seq + p); }
    // returns the valid-entry bits (4) of this lane; sc = orderable score (high key word), tie = ~low key word
    __device__ unsigned load4(int b, long long p, int e0, const int4& inf, uint32_t (&sc)[4], uint32_t (&tie)[4]) const {
        int live = inf.z;                                 // entries of this page that take part
        if (skip_newest > 0 && inf.x >= 0) {
            const int rest = cv.len[(size_t)b * cv.L * cv.H + inf.x] - skip_newest - inf.y * PAGE;   // entries left for this page
            live = rest < live ? (rest > 0 ? rest : 0) : live;
        }
        if (inf.x < 0 || e0 >= live) return 0u;
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
            bad |= (S != S) && (e0 + j < live);
            sc[j] = orderable_key(S);
            tie[j] = ((uint32_t)p4[j] << cv.pool_bits) | (uint32_t)(inf.x + cv.pool_offset);
            if (e0 + j < live) vm |= 1u << j;
        }
        if (bad) latch_error(cv.err, TRIMKV_E_NONFINITE);
        return vm;
    }
};

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
    // Pages are visited from the end of the CTA's range backwards (warp-uniform trip count).
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



// The newest entry of every pool, classified after a filter pass that left it out (its retention terms arrived later):
// one thread per pool; flagged, listed or left alone exactly as the filter pass would have done.
__global__ void filter_newest_kernel(CacheSrc src, SelState* __restrict__ sel, Cand* __restrict__ cand, long long cand_cap,
                                     u64* __restrict__ evict_mask, long long mask_stride, int32_t* err) {
    const CacheView& cv = src.cv;
    const int LH = cv.L * cv.H;
    const int gid = blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= cv.B * LH) return;
    const int b = gid / LH, pool_local = gid % LH;
    const int n = cv.len[gid];
    if (n <= 0) return;
    const int idx = n - 1;
    const int page = cv.block_table[(size_t)gid * cv.maxpp + idx / PAGE];
    const int off = idx % PAGE;
    const size_t slot = ((size_t)b * cv.P_seq + page) * PAGE + off;
    const int pos = cv.pos[slot];
    const float S = retention_score(cv.lam[slot], cv.c[slot], (float)(src.t1 - (long long)pos));
    if (S != S) latch_error(cv.err, TRIMKV_E_NONFINITE);
    const u64 key = make_key(S, ((uint32_t)pos << cv.pool_bits) | (uint32_t)(pool_local + cv.pool_offset));
    SelState* st = sel + b;
    if (key < st->cand_lo) {
        atomicOr(reinterpret_cast<unsigned long long*>(evict_mask + (size_t)b * mask_stride + page), 1ull << off);
        atomicAdd(reinterpret_cast<unsigned long long*>(&st->n_below), 1ull);
    } else if (key <= st->cand_hi) {
        const unsigned w = atomicAdd(&st->cand_count, 1u);
        if ((long long)w < cand_cap) {
            Cand cnd;
            cnd.key = key;
            cnd.slot = (u64)((long long)page * PAGE + off);
            cand[(size_t)b * cand_cap + w] = cnd;
        } else {
            latch_error(err, TRIMKV_E_NOMEM);
        }
    }
}

// ------------------------------------------------------------------ sample bracket (cache path)
// One full pass suffices when a candidate range that surely holds the k-th smallest key is known beforehand.
// A Bernoulli sample of the sequence's keys (a hash of the slot decides, about SAMPLE_MEAN keys) is sorted by one
// CTA; the sample keys at ranks k*p -+ a margin of several standard deviations bound the range.  The filter pass
// then counts the keys below the range, and the exact ranking verifies that the k-th key lay inside; if it did
// not (probability below 1e-9 per call), a single-CTA exact selection redoes the sequence.
constexpr int SAMPLE_CAP = 4096;
constexpr int SAMPLE_MEAN = 3072;

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
        const uint32_t tie = ((uint32_t)pos << cv.pool_bits) | (uint32_t)(inf.x + cv.pool_offset);
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
        st->resolved = 0;
        st->passes = ns;
    }
}

constexpr int SHARD_TAG_SHIFT = 56;      // a sharded selection tags a candidate's slot with its rank above this bit

// ------------------------------------------------------------------ exact ranking of the candidates
// One CTA per sequence.  An inconsistent count (the k-th key is not among the candidates, or the list overflowed) means
// the sampled range missed: resolved stays 0 and (redo_inline) this CTA redoes its sequence exactly, or the caller runs
// its own fallback.
__device__ void redo_body(CacheSrc src, SelState* __restrict__ sel, u64* __restrict__ evict_mask, long long mask_stride,
                          long long k_evict, int32_t* err);

__global__ void __launch_bounds__(1024)
resolve_kernel(SelState* __restrict__ sel, Cand* __restrict__ cand, long long cand_cap, u64* __restrict__ evict_mask,
               long long mask_stride, long long k_evict, long long* __restrict__ stats,
               int32_t* __restrict__ cursor, int32_t* err, CacheSrc src, int redo_inline, int my_rank = -1) {
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
    const bool ok = r >= 0 && r <= C && craw <= cand_cap;
    const int sample_n = st->passes;
    if (!ok) {
        if (tid == 0) {
            st->resolved = 0;
            st->sample_count = 0;
            if (stats) { stats[b * 4 + 0] = 1; stats[b * 4 + 1] = C; stats[b * 4 + 2] = k_evict; stats[b * 4 + 3] = sample_n; }
            if (cursor) cursor[b] = 0;
        }
        // the bracket missed (next to never): this CTA redoes its sequence exactly, at once, instead of a further
        // kernel that every call would have to launch just to find nothing to do
        __syncthreads();
        if (redo_inline) redo_body(src, sel, evict_mask, mask_stride, k_evict, err);
        return;
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
            // my_rank >= 0 (a sequence sharded over ranks): the list holds every rank's candidates, tagged with their
            // rank in the slot's top byte; only this rank's own slots exist here
            if (cnd.key <= tau && (my_rank < 0 || (int)(cnd.slot >> SHARD_TAG_SHIFT) == my_rank)) {
                const u64 slot = cnd.slot & ((1ull << SHARD_TAG_SHIFT) - 1ull);
                atomicOr(evict_mask + (size_t)b * mask_stride + (slot >> 6), 1ull << (slot & 63));
            }
        }
    } else {
        tau = st->cand_lo;
    }
    __syncthreads();
    if (tid == 0) {
        if (stats) {
            stats[b * 4 + 0] = 0;
            stats[b * 4 + 1] = C;
            stats[b * 4 + 2] = k_evict;
            stats[b * 4 + 3] = sample_n;
        }
        st->resolved = 1;
        st->cand_count = 0;
        st->sample_count = 0;
        if (cursor) cursor[b] = 0;
    }
}

// Exact redo for a sequence whose sample bracket missed (called by the ranking kernel's CTA of that sequence): the CTA
// radix-selects the k-th smallest key over all of the sequence's entries (DB bits per sweep) and rewrites every eviction
// mask.  Slow and rare.
__device__ void redo_body(CacheSrc src, SelState* __restrict__ sel, u64* __restrict__ evict_mask, long long mask_stride,
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
        return make_key(S, ((uint32_t)pos << cv.pool_bits) | (uint32_t)(pool_local + cv.pool_offset));
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
    s.cand_lo = 0ull; s.cand_hi = 0ull; s.n_below = 0;
    s.resolved = 0; s.passes = 0; s.cand_count = 0; s.sample_count = 0;
    sel[b] = s;
}

int grid_x_for(long long pages, int B) {
    long long g = (pages + 31) / 32;              // at least ~32 pages per CTA
    long long cap = (592 + B - 1) / B;            // ~4 CTAs per SM over the whole grid
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

// ------------------------------------------------------------------ one sequence sharded by layer over ranks
// Every rank holds the pools of a slice of the layers; the budget is global over all of them (Sec. 4.2).  The selection
// is the same as on one GPU (sample -> bracket -> filter -> exact ranking), with three small exchanges between the
// stages: the ranks' sample keys, their counts of keys below the bracket, and their candidates.  After each exchange
// every rank computes the same thing from the same data, so all reach the same threshold and each flags its own slots.
// The kernels below are the rank-local pieces; the exchanges are the caller's (NCCL through torch.distributed).

// Sample keys and their count out of the handle (one CTA per sequence).
__global__ void shard_export_sample_kernel(const SelState* __restrict__ sel, const u64* __restrict__ sample,
                                           u64* __restrict__ keys_out, int32_t* __restrict__ counts_out) {
    const int b = blockIdx.x;
    const unsigned raw = sel[b].sample_count;
    const int ns = (int)min(raw, (unsigned)SAMPLE_CAP);
    for (int i = threadIdx.x; i < ns; i += blockDim.x) keys_out[(size_t)b * SAMPLE_CAP + i] = sample[(size_t)b * SAMPLE_CAP + i];
    if (threadIdx.x == 0) counts_out[b] = ns;
}

// The ranks' samples, concatenated in rank order, become the handle's sample (gkeys [W][B][SAMPLE_CAP], gcounts [W][B]).
__global__ void shard_merge_sample_kernel(const u64* __restrict__ gkeys, const int32_t* __restrict__ gcounts, int W, int B,
                                          SelState* __restrict__ sel, u64* __restrict__ sample) {
    const int b = blockIdx.x;
    long long off = 0;
    for (int w = 0; w < W; ++w) {
        const int cnt = gcounts[(size_t)w * B + b];
        const u64* src = gkeys + ((size_t)w * B + b) * SAMPLE_CAP;
        for (int i = threadIdx.x; i < cnt; i += blockDim.x)
            if (off + i < SAMPLE_CAP) sample[(size_t)b * SAMPLE_CAP + off + i] = src[i];
        off += cnt;
    }
    if (threadIdx.x == 0) sel[b].sample_count = (unsigned)off;
}

__global__ void shard_export_filter_kernel(const SelState* __restrict__ sel, long long cand_cap, long long* __restrict__ n_below_out,
                                           int32_t* __restrict__ cand_count_out, int B) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    n_below_out[b] = sel[b].n_below;
    const long long cc = (long long)sel[b].cand_count;
    cand_count_out[b] = cc > cand_cap ? -1 : (int32_t)cc;                            // -1: the local list overflowed
}

__global__ void shard_export_cands_kernel(const SelState* __restrict__ sel, const Cand* __restrict__ cand, long long cand_cap,
                                          Cand* __restrict__ out, long long cap) {
    const int b = blockIdx.y;
    const long long cnt = min(min((long long)sel[b].cand_count, cand_cap), cap);
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < cnt; i += (long long)gridDim.x * blockDim.x)
        out[(size_t)b * cap + i] = cand[(size_t)b * cand_cap + i];
}

// All ranks' candidates (gcand [W][B][cap], gcounts [W][B]) become the handle's candidate list, each slot tagged with its
// rank; the global count of keys below the bracket replaces the local one.  A list that does not fit, or a rank whose
// own list overflowed, makes the count inconsistent on purpose: the exact ranking then reports a miss.
__global__ void shard_merge_cands_kernel(const Cand* __restrict__ gcand, const int32_t* __restrict__ gcounts,
                                         const long long* __restrict__ n_below_global, int W, int B, long long cap,
                                         SelState* __restrict__ sel, Cand* __restrict__ cand, long long cand_cap) {
    const int b = blockIdx.y;
    long long off = 0;
    bool bad = false;
    for (int w = 0; w < W; ++w) {
        const long long cnt = gcounts[(size_t)w * B + b];
        if (cnt < 0 || cnt > cap) { bad = true; continue; }
        const Cand* src = gcand + ((size_t)w * B + b) * cap;
        for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < cnt; i += (long long)gridDim.x * blockDim.x) {
            if (off + i < cand_cap) {
                Cand c = src[i];
                c.slot |= (u64)w << SHARD_TAG_SHIFT;
                cand[(size_t)b * cand_cap + off + i] = c;
            }
        }
        off += cnt;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        sel[b].cand_count = (bad || off > cand_cap) ? 0xffffffffu : (unsigned)off;
        sel[b].n_below = n_below_global[b];
    }
}

__global__ void shard_export_resolved_kernel(const SelState* __restrict__ sel, int32_t* __restrict__ out, int B) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) out[b] = sel[b].resolved;
}

// Exact fallback, one radix digit per round: local histogram of the digit below `top` over the keys whose bits above
// `top` equal prefix[b] (sequences already resolved contribute nothing).  hist_out [B][2048], zeroed here.
__global__ void __launch_bounds__(1024)
shard_hist_kernel(CacheSrc src, const SelState* __restrict__ sel, const u64* __restrict__ prefix, int top,
                  unsigned* __restrict__ hist_out) {
    constexpr int DB = 11, NBIN = 1 << DB;
    __shared__ unsigned hist[NBIN];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    hist[tid] = 0u;
    hist[tid + 1024] = 0u;
    __syncthreads();
    if (!sel[b].resolved) {
        const int dbits = top < DB ? top : DB, sh = top - dbits;
        const u64 pfx = prefix[b];
        const int sub = lane >> 4, e0 = (lane & 15) * 4;
        const long long P = src.pages();
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
                        if (top >= 64 || (key >> top) == pfx) atomicAdd(&hist[(unsigned)((key >> sh) & ((1u << dbits) - 1u))], 1u);
                    }
                }
            }
        }
    }
    __syncthreads();
    hist_out[(size_t)b * NBIN + tid] = hist[tid];
    hist_out[(size_t)b * NBIN + tid + 1024] = hist[tid + 1024];
}

// From the histogram summed over the ranks: the digit that holds rank r[b]; prefix and rank move one digit down.
__global__ void __launch_bounds__(1024)
shard_digit_kernel(const unsigned* __restrict__ hist, u64* __restrict__ prefix, long long* __restrict__ rank, int top) {
    constexpr int DB = 11, NBIN = 1 << DB;
    __shared__ unsigned wtot[32];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int dbits = top < DB ? top : DB;
    const unsigned h0 = hist[(size_t)b * NBIN + 2 * tid], h1 = hist[(size_t)b * NBIN + 2 * tid + 1];
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
    const long long r = rank[b];
    const u64 p = top >= 64 ? 0ull : (prefix[b] << dbits);
    __syncthreads();
    if (r > excl && r <= excl + h0) { prefix[b] = p | (u64)(2 * tid); rank[b] = r - excl; }
    else if (r > excl + h0 && r <= excl + h0 + h1) { prefix[b] = p | (u64)(2 * tid + 1); rank[b] = r - excl - h0; }
}

// Exact fallback, last step: every local key up to tau[b] is evicted (sequences already resolved keep their masks).
__global__ void __launch_bounds__(1024)
shard_mark_kernel(CacheSrc src, SelState* __restrict__ sel, const u64* __restrict__ tau, u64* __restrict__ evict_mask,
                  long long mask_stride, int32_t* __restrict__ cursor) {
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (sel[b].resolved) return;
    const u64 t = tau[b];
    const int sub = lane >> 4, l16 = lane & 15, e0 = l16 * 4;
    const long long P = src.pages();
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
            if ((vm & (1u << j)) && compose_key(sc[j], tie[j]) <= t) ev |= 1u << j;
        const unsigned nib = ev << (4 * (l16 & 7));
        unsigned wlo = (l16 < 8) ? nib : 0u, whi = (l16 >= 8) ? nib : 0u;
#pragma unroll
        for (int o = 1; o < 16; o <<= 1) {
            wlo |= __shfl_xor_sync(0xffffffffu, wlo, o);
            whi |= __shfl_xor_sync(0xffffffffu, whi, o);
        }
        if (l16 == 0 && page < P && inf.x >= 0) evict_mask[(size_t)b * mask_stride + page] = ((u64)whi << 32) | (u64)wlo;
    }
    __syncthreads();
    if (tid == 0) { sel[b].resolved = 1; sel[b].cand_count = 0; sel[b].sample_count = 0; if (cursor) cursor[b] = 0; }
}

}  // namespace

// ---- launchers of the sharded selection's rank-local stages
int shard_sample_cap() { return SAMPLE_CAP; }

void launch_shard_export_sample(const CacheView& cv, const SelectBuffers& sb, u64* keys_out, int32_t* counts_out, cudaStream_t st) {
    shard_export_sample_kernel<<<cv.B, 256, 0, st>>>(sb.sel, sb.sample, keys_out, counts_out);
    count_launch();
}

void launch_shard_bracket(const CacheView& cv, const SelectBuffers& sb, const u64* gkeys, const int32_t* gcounts, int world,
                          long long n_total, long long k_evict, int distrust, cudaStream_t st) {
    shard_merge_sample_kernel<<<cv.B, 256, 0, st>>>(gkeys, gcounts, world, cv.B, sb.sel, sb.sample);
    bracket_kernel<<<cv.B, 1024, 0, st>>>(sb.sel, sb.sample, k_evict, n_total, distrust, 7.0f);
    count_launch(2);
}

void launch_shard_filter(const CacheView& cv, const SelectBuffers& sb, long long t, long long* n_below_out,
                         int32_t* cand_count_out, cudaStream_t st) {
    CacheSrc src;
    src.cv = cv;
    src.t1 = t + 1;
    dim3 grid(grid_x_for(cv.P_seq, cv.B), cv.B);
    filter_kernel<CacheSrc, true><<<grid, 256, 0, st>>>(src, sb.sel, sb.cand, sb.cand_cap, cv.evict_mask, cv.P_seq, nullptr);
    shard_export_filter_kernel<<<(cv.B + 127) / 128, 128, 0, st>>>(sb.sel, sb.cand_cap, n_below_out, cand_count_out, cv.B);
    count_launch(2);
}

void launch_shard_export_cands(const CacheView& cv, const SelectBuffers& sb, void* out, long long cap, cudaStream_t st) {
    dim3 grid(8, cv.B);
    shard_export_cands_kernel<<<grid, 256, 0, st>>>(sb.sel, sb.cand, sb.cand_cap, (Cand*)out, cap);
    count_launch();
}

void launch_shard_resolve(const CacheView& cv, const SelectBuffers& sb, const void* gcand, const int32_t* gcounts,
                          const long long* n_below_global, int world, int rank, long long cap, long long k_evict,
                          int32_t* compact_cursor, int32_t* resolved_out, cudaStream_t st) {
    dim3 grid(8, cv.B);
    shard_merge_cands_kernel<<<grid, 256, 0, st>>>((const Cand*)gcand, gcounts, n_below_global, world, cv.B, cap, sb.sel, sb.cand,
                                                   sb.cand_cap);
    CacheSrc none;
    none.cv = cv;
    none.t1 = 0;
    resolve_kernel<<<cv.B, 1024, 0, st>>>(sb.sel, sb.cand, sb.cand_cap, cv.evict_mask, cv.P_seq, k_evict, sb.stats,
                                                 compact_cursor, cv.err, none, 0, rank);
    shard_export_resolved_kernel<<<(cv.B + 127) / 128, 128, 0, st>>>(sb.sel, resolved_out, cv.B);
    count_launch(3);
}

void launch_shard_hist(const CacheView& cv, const SelectBuffers& sb, long long t, const u64* prefix, int top, unsigned* hist_out,
                       cudaStream_t st) {
    CacheSrc src;
    src.cv = cv;
    src.t1 = t + 1;
    shard_hist_kernel<<<cv.B, 1024, 0, st>>>(src, sb.sel, prefix, top, hist_out);
    count_launch();
}

void launch_shard_digit(int B, const unsigned* hist, u64* prefix, long long* rank, int top, cudaStream_t st) {
    shard_digit_kernel<<<B, 1024, 0, st>>>(hist, prefix, rank, top);
    count_launch();
}

void launch_shard_mark(const CacheView& cv, const SelectBuffers& sb, long long t, const u64* tau, int32_t* compact_cursor,
                       cudaStream_t st) {
    CacheSrc src;
    src.cv = cv;
    src.t1 = t + 1;
    shard_mark_kernel<<<cv.B, 1024, 0, st>>>(src, sb.sel, tau, cv.evict_mask, cv.P_seq, compact_cursor);
    count_launch();
}

void launch_select_state_init(SelState* sel, int B, cudaStream_t st) {
    state_init_kernel<<<(B + 127) / 128, 128, 0, st>>>(sel, B);
    count_launch();
}

// The sampling pass alone (n_total: the entry count the sampling rate is derived from).
static void launch_sample_only(const CacheView& cv, const SelectBuffers& sb, long long t, long long n_total, int skip_newest,
                               cudaStream_t st) {
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
    const uint32_t seed = (uint32_t)t * 0x9E3779B1u + 0x1234567u + (uint32_t)cv.pool_offset * 0x632BE5ABu;
    const long long threads = cv.P_seq * (sub > 0 ? PAGE / sub : 1);
    dim3 gs((unsigned)((threads + 255) / 256), cv.B);
    sample_kernel<<<gs, 256, 0, st>>>(src, sb.sel, sb.sample, sub, thresh, seed, skip_newest);
    count_launch();
}

void launch_select_cache_sample(const CacheView& cv, const SelectBuffers& sb, long long t, long long n_total,
                                long long k_evict, int skip_newest, int distrust_sample, cudaStream_t st) {
    launch_sample_only(cv, sb, t, n_total, skip_newest, st);
    // 7 sigma: a miss costs the single-CTA exact redo of the whole sequence, so it must be next to impossible
    bracket_kernel<<<cv.B, 1024, 0, st>>>(sb.sel, sb.sample, k_evict, n_total, distrust_sample, 7.0f);
    count_launch();
}

void launch_shard_sample(const CacheView& cv, const SelectBuffers& sb, long long t, long long n_total, u64* keys_out,
                         int32_t* counts_out, cudaStream_t st) {
    launch_sample_only(cv, sb, t, n_total, 0, st);
    launch_shard_export_sample(cv, sb, keys_out, counts_out, st);
}

void launch_select_cache_filter(const CacheView& cv, const SelectBuffers& sb, long long t, int skip_newest, cudaStream_t st) {
    CacheSrc src;
    src.cv = cv;
    src.t1 = t + 1;
    src.skip_newest = skip_newest;
    dim3 grid(grid_x_for(cv.P_seq, cv.B), cv.B);
    filter_kernel<CacheSrc, true><<<grid, 256, 0, st>>>(src, sb.sel, sb.cand, sb.cand_cap, cv.evict_mask, cv.P_seq, cv.err);
    count_launch();
}

void launch_select_cache_finish(const CacheView& cv, const SelectBuffers& sb, long long t, long long k_evict,
                                int32_t* compact_cursor, int newest_left_out, cudaStream_t st) {
    CacheSrc src;
    src.cv = cv;
    src.t1 = t + 1;
    if (newest_left_out) {
        const int pools = cv.B * cv.L * cv.H;
        filter_newest_kernel<<<(pools + 127) / 128, 128, 0, st>>>(src, sb.sel, sb.cand, sb.cand_cap, cv.evict_mask, cv.P_seq, cv.err);
        count_launch();
    }
    resolve_kernel<<<cv.B, 1024, 0, st>>>(sb.sel, sb.cand, sb.cand_cap, cv.evict_mask, cv.P_seq, k_evict,
                                                 sb.stats, compact_cursor, cv.err, src, 1);
    count_launch();
}

void launch_select_cache_rest(const CacheView& cv, const SelectBuffers& sb, long long t, long long k_evict,
                              int32_t* compact_cursor, cudaStream_t st) {
    CacheSrc src;
    src.cv = cv;
    src.t1 = t + 1;
    dim3 grid(grid_x_for(cv.P_seq, cv.B), cv.B);
    filter_kernel<CacheSrc, true><<<grid, 256, 0, st>>>(src, sb.sel, sb.cand, sb.cand_cap, cv.evict_mask, cv.P_seq, cv.err);
    resolve_kernel<<<cv.B, 1024, 0, st>>>(sb.sel, sb.cand, sb.cand_cap, cv.evict_mask, cv.P_seq, k_evict,
                                                 sb.stats, compact_cursor, cv.err, src, 1);
    count_launch(2);
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

}  // namespace tkv
