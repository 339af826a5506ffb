// Global selection (Sec. 4.2): per sequence, evict the k entries with the lowest retention score
// S = (t + 1 - i) * lambda + c  (log of Eq. (global_score)) under the total order
// (score, then newer position first, then higher layer, then higher head are evicted first).
//
// Method: every entry maps to a unique 64-bit key whose integer order is the eviction order.  A
// histogram pass over all keys (shared-memory histogram per CTA, 4094 equal-width bins over a key range
// centred on the previous call's threshold) locates the bin that holds the k-th smallest key; if that
// bin is too full the range is narrowed to it ("zoom") and the pass repeats.  A filter pass then marks
// every key below the bin as evicted (one 64-bit mask per page, built with warp votes) and collects the
// keys inside the bin; a single CTA ranks those candidates exactly (radix select on the differing bits).
// The result is identical to a full sort; no floating-point value is compared after key construction.
#include "trimkv_internal.cuh"

namespace tkv {

namespace {

// ------------------------------------------------------------------ key sources
// A source presents its entries as pages of 64; a half-warp reads one page, 4 consecutive entries per lane.
struct CacheSrc {
    CacheView cv;
    long long t1;   // t + 1
    __device__ long long pages() const { return cv.P_seq; }
    // returns the valid-entry bits (4) of this lane; sets owned = page holds live entries
    __device__ unsigned load4(int b, long long p, int e0, u64 (&key)[4], bool& owned) const {
        const int2 ow = cv.owner[(size_t)b * cv.P_seq + p];
        owned = ow.x >= 0;
        if (!owned) return 0u;
        const int fill = cv.len[(size_t)b * cv.L * cv.H + ow.x] - ow.y * PAGE;
        const size_t s = ((size_t)b * cv.P_seq + p) * PAGE + e0;
        const float4 lm = *reinterpret_cast<const float4*>(cv.lam + s);
        const float4 cc = *reinterpret_cast<const float4*>(cv.c + s);
        const int4 ps = *reinterpret_cast<const int4*>(cv.pos + s);
        const float l4[4] = {lm.x, lm.y, lm.z, lm.w};
        const float c4[4] = {cc.x, cc.y, cc.z, cc.w};
        const int p4[4] = {ps.x, ps.y, ps.z, ps.w};
        unsigned vm = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (e0 + j < fill) {
                const float age = (float)(t1 - (long long)p4[j]);
                const float S = retention_score(l4[j], c4[j], age);
                if (S != S) latch_error(cv.err, TRIMKV_E_NONFINITE);
                const uint32_t tie = ((uint32_t)p4[j] << cv.pool_bits) | (uint32_t)ow.x;
                key[j] = make_key(S, tie);
                vm |= 1u << j;
            }
        }
        return vm;
    }
};

struct ArraySrc {
    const float* s;
    long long n;
    int32_t* err;
    __device__ long long pages() const { return (n + PAGE - 1) / PAGE; }
    __device__ unsigned load4(int, long long p, int e0, u64 (&key)[4], bool& owned) const {
        owned = true;
        const long long i0 = p * PAGE + e0;
        float v[4];
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
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (vm & (1u << j)) {
                if (v[j] != v[j]) latch_error(err, TRIMKV_E_NONFINITE);
                key[j] = make_key(v[j], (uint32_t)(i0 + j));
            }
        }
        return vm;
    }
};

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
            const u64 span = c_hi - c_lo;
            const int bits = 64 - __clzll((long long)span);
            st->lo = c_lo;
            st->shift = bits > ZOOM_BITS ? bits - ZOOM_BITS : 0;
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
    for (long long pp = p0 + warp * 2; pp < p1; pp += (blockDim.x >> 5) * 2) {
        const long long page = pp + sub;
        if (page < p1) {
            u64 key[4];
            bool owned;
            const unsigned vm = src.load4(b, page, e0, key, owned);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (vm & (1u << j)) {
                    kmin = key[j] < kmin ? key[j] : kmin;
                    kmax = key[j] > kmax ? key[j] : kmax;
                    const int bin = bin_of(key[j], lo, shift);
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
        }
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
template <class Src>
__global__ void __launch_bounds__(256)
filter_kernel(Src src, SelState* __restrict__ sel, Cand* __restrict__ cand, long long cand_cap,
              u64* __restrict__ evict_mask, long long mask_stride, int32_t* err) {
    const int b = blockIdx.y;
    SelState* st = sel + b;
    const u64 c_lo = st->cand_lo, c_hi = st->cand_hi;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane >> 4, l16 = lane & 15, e0 = l16 * 4;
    const long long P = src.pages();
    const long long chunk = (P + gridDim.x - 1) / gridDim.x;
    const long long p0 = (long long)blockIdx.x * chunk;
    const long long p1 = min(P, p0 + chunk);
    Cand* cb = cand + (size_t)b * cand_cap;

    for (long long pp = p0 + warp * 2; pp < p1; pp += (blockDim.x >> 5) * 2) {   // warp-uniform trip count
        const long long page = pp + sub;
        u64 key[4];
        bool owned = false;
        unsigned vm = 0;
        if (page < p1) vm = src.load4(b, page, e0, key, owned);
        unsigned ev = 0, cd = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (vm & (1u << j)) {
                if (key[j] < c_lo) ev |= 1u << j;
                else if (key[j] <= c_hi) cd |= 1u << j;
            }
        }
        // candidates: warp-aggregated append
        const int nc = __popc(cd);
        int incl = nc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        const int tot = __shfl_sync(0xffffffffu, incl, 31);
        if (tot > 0) {
            unsigned base = 0;
            if (lane == 0) base = atomicAdd(&st->cand_count, (unsigned)tot);
            base = __shfl_sync(0xffffffffu, base, 0);
            long long w = (long long)base + incl - nc;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (cd & (1u << j)) {
                    if (w < cand_cap) {
                        Cand cnd;
                        cnd.key = key[j];
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
        if (l16 == 0 && page < p1 && owned) evict_mask[(size_t)b * mask_stride + page] = ((u64)whi << 32) | (u64)wlo;
    }
}

// ------------------------------------------------------------------ exact ranking of the candidates
__global__ void __launch_bounds__(1024)
resolve_kernel(SelState* __restrict__ sel, Cand* __restrict__ cand, long long cand_cap, u64* __restrict__ evict_mask,
               long long mask_stride, long long k_evict, unsigned cand_target, long long* __restrict__ stats,
               int32_t* __restrict__ cursor, int32_t* err) {
    __shared__ unsigned hist[256];
    __shared__ u64 s_prefix;
    __shared__ long long s_r;
    const int b = blockIdx.x;
    SelState* st = sel + b;
    const Cand* cb = cand + (size_t)b * cand_cap;
    const long long C = min((long long)st->cand_count, cand_cap);
    long long r = k_evict - st->n_below;
    const u64 lo = st->cand_lo, hi = st->cand_hi;
    if (r < 0 || r > C || (long long)st->cand_expected != (long long)st->cand_count) {
        if (threadIdx.x == 0) latch_error(err, TRIMKV_E_STATE);
        r = r < 0 ? 0 : (r > C ? C : r);
    }
    u64 tau = lo;
    if (r > 0) {
        int top = (lo == hi) ? 0 : 64 - __clzll((long long)(lo ^ hi));   // number of low bits that differ
        u64 prefix = top >= 64 ? 0ull : (lo >> top);
        while (top > 0) {
            const int dbits = top < 8 ? top : 8;
            const int sh = top - dbits;
            for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0u;
            __syncthreads();
            for (long long i = threadIdx.x; i < C; i += blockDim.x) {
                const u64 key = cb[i].key;
                const bool match = top >= 64 ? true : ((key >> top) == prefix);
                if (match) atomicAdd(&hist[(unsigned)((key >> sh) & ((1u << dbits) - 1u))], 1u);
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                long long cum = 0, rr = r;
                unsigned dv = 0;
                for (unsigned q = 0; q < (1u << dbits); ++q) {
                    if (rr <= cum + (long long)hist[q]) { dv = q; rr -= cum; break; }
                    cum += hist[q];
                }
                s_prefix = (top >= 64 ? 0ull : (prefix << dbits)) | (u64)dv;
                s_r = rr;
            }
            __syncthreads();
            prefix = s_prefix;
            r = s_r;
            top = sh;
        }
        tau = prefix;   // the r-th smallest candidate key: everything <= tau is evicted
        for (long long i = threadIdx.x; i < C; i += blockDim.x) {
            const Cand cnd = cb[i];
            if (cnd.key <= tau)
                atomicOr(evict_mask + (size_t)b * mask_stride + (cnd.slot >> 6), 1ull << (cnd.slot & 63));
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (stats) {
            stats[b * 4 + 0] = st->passes;
            stats[b * 4 + 1] = C;
            stats[b * 4 + 2] = k_evict;
            stats[b * 4 + 3] = st->shift;
        }
        // centre the next call's first histogram on this threshold; aim for ~cand_target/8 candidates
        int shift = st->shift;
        const int want = 31 - __clz((int)max(cand_target / 8u, 1u));
        const int have = 31 - __clz((int)max((unsigned)min(C, 0x7fffffffLL), 1u));
        shift += want - have;
        shift = shift < 0 ? 0 : (shift > INIT_SHIFT ? INIT_SHIFT : shift);
        const u64 half = (u64)(REG_BINS / 2) << shift;
        st->lo = tau > half ? tau - half : 0ull;
        st->shift = shift;
        st->resolved = 0;
        st->passes = 0;
        st->cand_count = 0;
        st->kmin = ~0ull;
        st->kmax = 0ull;
        if (cursor) cursor[b] = 0;
    }
}

__global__ void state_init_kernel(SelState* sel, int B) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    SelState s;
    s.lo = 0ull; s.kmin = ~0ull; s.kmax = 0ull; s.cand_lo = 0ull; s.cand_hi = 0ull; s.n_below = 0;
    s.shift = INIT_SHIFT; s.resolved = 0; s.passes = 0; s.cand_count = 0; s.cand_expected = 0; s.pad = 0;
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

template <class Src>
void run_select(const Src& src, long long pages, int B, const SelectBuffers& sb, long long n_total, long long k_evict,
                int max_passes, unsigned cand_target, u64* evict_mask, long long mask_stride, int32_t* cursor,
                int32_t* err, cudaStream_t st) {
    dim3 grid(grid_x_for(pages, B), B);
    for (int p = 0; p < max_passes; ++p)
        hist_kernel<Src><<<grid, 256, 0, st>>>(src, sb.sel, sb.hist, sb.done, k_evict, n_total, p == max_passes - 1,
                                               cand_target);
    filter_kernel<Src><<<grid, 256, 0, st>>>(src, sb.sel, sb.cand, sb.cand_cap, evict_mask, mask_stride, err);
    resolve_kernel<<<B, 1024, 0, st>>>(sb.sel, sb.cand, sb.cand_cap, evict_mask, mask_stride, k_evict, cand_target,
                                       sb.stats, cursor, err);
    count_launch(max_passes + 2);
}

}  // namespace

void launch_select_state_init(SelState* sel, int B, cudaStream_t st) {
    state_init_kernel<<<(B + 127) / 128, 128, 0, st>>>(sel, B);
    count_launch();
}

void launch_select_cache(const CacheView& cv, const SelectBuffers& sb, long long t, long long n_total,
                         long long k_evict, int32_t* compact_cursor, cudaStream_t st) {
    CacheSrc src;
    src.cv = cv;
    src.t1 = t + 1;
    run_select(src, cv.P_seq, cv.B, sb, n_total, k_evict, MAX_HIST_PASSES, 16384u, cv.evict_mask, cv.P_seq,
               compact_cursor, cv.err, st);
}

void launch_select_array(const float* scores, long long n, long long k_evict, u64* evict_mask, const SelectBuffers& sb,
                         int32_t* err, cudaStream_t st) {
    ArraySrc src;
    src.s = scores;
    src.n = n;
    src.err = err;
    const long long pages = (n + PAGE - 1) / PAGE;
    run_select(src, pages, 1, sb, n, k_evict, 7, (unsigned)sb.cand_cap, evict_mask, pages, nullptr, err, st);
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
