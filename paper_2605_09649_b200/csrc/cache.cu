// Paged per-(layer, head) KV pools (Sec. 4.2 "Implementation details": fixed-size pages, one block
// table per head, variable logical length per head): append of new tokens and compaction after an
// eviction round.
#include <algorithm>

#include "trimkv_internal.cuh"

namespace tkv {

namespace {

// One CTA per pool: take pages from the sequence's free stack if the pool grows past its last page,
// then copy the new rows (K, V, retention metadata) to their slots.
// mode bit 0 (APPEND_KV): allocate pages, write K/V rows, positions, page records and the new length.
// mode bit 1 (APPEND_META): write the retention terms (lambda, c).  Alone, it completes an earlier APPEND_KV call
// with the same arguments: the length then already counts the new tokens.
__global__ void __launch_bounds__(256)
append_kernel(CacheView cv, int layer0, int n_new, long long pos0, const float* __restrict__ lam_in,
              const float* __restrict__ c_in, int horizon, const char* __restrict__ k_in,
              const char* __restrict__ v_in, int mode) {
    __shared__ int s_old;
    __shared__ int s_fail;
    const int h = blockIdx.x % cv.H;
    const int b = (blockIdx.x / cv.H) % cv.B;
    const int lb = blockIdx.x / (cv.H * cv.B);
    const int layer = layer0 + lb;
    const int pool_local = layer * cv.H + h;
    const long long pool = (long long)b * cv.L * cv.H + pool_local;
    int32_t* bt = cv.block_table + pool * cv.maxpp;

    if (!(mode & APPEND_KV)) {
        if (cv.append_failed[pool]) return;            // the K/V half of this append failed (its error is latched)
        const int old = cv.len[pool] - n_new;
        if (old < 0) return;
        const size_t in_row0 = (((size_t)lb * cv.B + b) * n_new) * cv.H + h;
        for (int j = threadIdx.x; j < n_new; j += blockDim.x) {
            const int idx = old + j;
            const int page = bt[idx / PAGE];
            const size_t slot = ((size_t)b * cv.P_seq + page) * PAGE + idx % PAGE;
            const size_t mi = (in_row0 + (size_t)j * cv.H);
            const float lm = lam_in[mi];
            const float cc = c_in ? c_in[mi] : horizon_term_f32(lm, horizon);
            if (lm != lm || cc != cc) latch_error(cv.err, TRIMKV_E_NONFINITE);
            cv.lam[slot] = lm;
            cv.c[slot] = cc;
        }
        return;
    }
    if (threadIdx.x == 0) {
        const int old = cv.len[pool];
        const long long nw = (long long)old + n_new;
        const long long p_old = (old + PAGE - 1) / PAGE, p_new = (nw + PAGE - 1) / PAGE;
        int fail = 0;
        if (p_new > cv.maxpp) {
            fail = 1;
        } else if (p_new > p_old) {
            const int need = (int)(p_new - p_old);
            const int prev = atomicSub(&cv.free_count[b], need);
            if (prev < need) {
                atomicAdd(&cv.free_count[b], need);
                fail = 1;
            } else {
                const int32_t* stack = cv.free_stack + (size_t)b * cv.P_seq;
                for (int j = 0; j < need; ++j) {
                    const int page = stack[prev - 1 - j];
                    bt[p_old + j] = page;
                }
            }
        }
        if (fail) latch_error(cv.err, TRIMKV_E_NOMEM);
        cv.append_failed[pool] = fail;                 // read by the halves of this append that run later
        s_old = old;
        s_fail = fail;
    }
    __syncthreads();
    if (s_fail) return;
    const int old = s_old;

    // rows: [lb][b][j][h][d]
    const int rc = cv.row_bytes / 16;                  // 16-byte chunks per row
    const size_t in_row0 = (((size_t)lb * cv.B + b) * n_new) * cv.H + h;
    const int total = (mode & APPEND_ROWS_ELSEWHERE) ? 0 : n_new * rc * 2;   // (a chunk's rows are copied by append_rows_kernel)
    for (int w = threadIdx.x; w < total; w += blockDim.x) {
        const int ci = w % rc;
        const int part = (w / rc) & 1;
        const int j = w / (2 * rc);
        const int idx = old + j;
        const int page = bt[idx / PAGE];
        const int off = idx % PAGE;
        const char* src = (part ? v_in : k_in) + (in_row0 + (size_t)j * cv.H) * cv.row_bytes + (size_t)ci * 16;
        char* dst = cv.kv + kv_row_offset(cv, b, page, part, off) + (size_t)phys_chunk(cv, ci, off) * 16;
        *reinterpret_cast<uint4*>(dst) = __ldg(reinterpret_cast<const uint4*>(src));
    }
    for (int j = threadIdx.x; j < n_new; j += blockDim.x) {
        const int idx = old + j;
        const int page = bt[idx / PAGE];
        const size_t slot = ((size_t)b * cv.P_seq + page) * PAGE + idx % PAGE;
        if (mode & APPEND_META) {
            const size_t mi = (in_row0 + (size_t)j * cv.H);
            const float lm = lam_in[mi];
            const float cc = c_in ? c_in[mi] : horizon_term_f32(lm, horizon);
            if (lm != lm || cc != cc) latch_error(cv.err, TRIMKV_E_NONFINITE);
            cv.lam[slot] = lm;
            cv.c[slot] = cc;
        }
        cv.pos[slot] = (int32_t)(pos0 + j + 1);
    }
    // page records of every page that received entries: owner pool, logical index, live entries
    const int n2 = old + n_new;
    for (int lp = old / PAGE + threadIdx.x; lp * PAGE < n2; lp += blockDim.x)
        cv.owner[(size_t)b * cv.P_seq + bt[lp]] = make_int4(pool_local, lp, min(PAGE, n2 - lp * PAGE), 0);
    __syncthreads();
    if (threadIdx.x == 0) cv.len[pool] = n2;
}

// K/V rows of a chunk: the copy half of an append whose bookkeeping (pages, length) append_kernel has done.
// grid = (pools of the call, blocks of APPEND_TOK tokens): a chunk's copy is spread over the whole GPU instead of one CTA
// per pool.
constexpr int APPEND_TOK = 32;
__global__ void __launch_bounds__(256)
append_rows_kernel(CacheView cv, int layer0, int n_new, const char* __restrict__ k_in, const char* __restrict__ v_in) {
    const int h = blockIdx.x % cv.H;
    const int b = (blockIdx.x / cv.H) % cv.B;
    const int lb = blockIdx.x / (cv.H * cv.B);
    const int pool_local = (layer0 + lb) * cv.H + h;
    const long long pool = (long long)b * cv.L * cv.H + pool_local;
    const int32_t* bt = cv.block_table + pool * cv.maxpp;
    if (cv.append_failed[pool]) return;                // the bookkeeping half failed (its error is latched)
    const int old = cv.len[pool] - n_new;
    if (old < 0) return;
    const int rc = cv.row_bytes / 16;
    const size_t in_row0 = (((size_t)lb * cv.B + b) * n_new) * cv.H + h;
    const int j0 = blockIdx.y * APPEND_TOK;
    const int total = min(APPEND_TOK, n_new - j0) * rc * 2;
    for (int w = threadIdx.x; w < total; w += blockDim.x) {
        const int ci = w % rc;
        const int part = (w / rc) & 1;
        const int j = j0 + w / (2 * rc);
        const int idx = old + j;
        const int page = bt[idx / PAGE];
        const int off = idx % PAGE;
        const char* src = (part ? v_in : k_in) + (in_row0 + (size_t)j * cv.H) * cv.row_bytes + (size_t)ci * 16;
        char* dst = cv.kv + kv_row_offset(cv, b, page, part, off) + (size_t)phys_chunk(cv, ci, off) * 16;
        *reinterpret_cast<uint4*>(dst) = __ldg(reinterpret_cast<const uint4*>(src));
    }
}

__device__ __forceinline__ u64 bits_below(int n) {   // mask with the lowest n bits set, n in [0, 64]
    return n >= 64 ? ~0ull : ((1ull << n) - 1ull);
}

// Block-wide exclusive scan of a 64-bit value over NW warps; returns the exclusive prefix and the total.
template <int NW>
__device__ __forceinline__ u64 block_exscan(u64 v, u64* total, u64* warp_tot /*[NW] shared*/) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    u64 incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        u64 t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    u64 off = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
        const u64 t = warp_tot[w];
        if (w < warp) off += t;
        tot += t;
    }
    *total = tot;
    return off + incl - v;
}

// One CTA per pool.  Entries flagged in evict_mask are removed: with n' = n - E survivors, the E' holes
// at logical index < n' are filled, in ascending order, by the survivors at index >= n' (ascending), so
// only as many rows move as there are holes.  Pages past the new end return to the free stack.
// NT threads: 256 when many rows move (after a prefill chunk), 128 for the one or two evictions per pool of a decode
// step (all CTAs of the launch are then resident at once).
template <int NT>
__global__ void __launch_bounds__(NT)
compact_kernel(CacheView cv, int32_t* __restrict__ hole, int32_t* __restrict__ mover, int32_t* __restrict__ cursor,
               long long e_max) {
    __shared__ u64 warp_tot[NT / 32];
    __shared__ long long s_base;
    __shared__ int s_freebase;
    const long long pool = blockIdx.x;
    const int b = (int)(pool / ((long long)cv.L * cv.H));
    const int n = cv.len[pool];
    if (n == 0) return;
    const int np = (n + PAGE - 1) / PAGE;
    const int32_t* bt = cv.block_table + pool * cv.maxpp;
    const u64* masks = cv.evict_mask + (size_t)b * cv.P_seq;

    // phase 1: number of evicted entries
    u64 e_local = 0;
    for (int lp = threadIdx.x; lp < np; lp += blockDim.x) {
        const u64 valid = bits_below(min(PAGE, n - lp * PAGE));
        e_local += __popcll(masks[bt[lp]] & valid);
    }
    u64 E;
    block_exscan<NT / 32>(e_local, &E, warp_tot);
    if (E == 0) return;
    const int n2 = n - (int)E;

    if (threadIdx.x == 0) {
        const long long base = (long long)atomicAdd(cursor + b, (int)E);
        s_base = base;
        if (base + (long long)E > e_max) latch_error(cv.err, TRIMKV_E_NOMEM);
    }
    __syncthreads();
    if (s_base + (long long)E > e_max) return;
    int32_t* hl = hole + (size_t)b * e_max + s_base;
    int32_t* ml = mover + (size_t)b * e_max + s_base;

    // phase 2: ordered lists of holes (evicted, index < n2) and movers (kept, index >= n2)
    long long run_h = 0, run_m = 0;
    for (int base = 0; base < np; base += blockDim.x) {
        const int lp = base + threadIdx.x;
        u64 hb = 0, mb = 0;
        int page = 0;
        if (lp < np) {
            page = bt[lp];
            const u64 valid = bits_below(min(PAGE, n - lp * PAGE));
            const u64 m = masks[page] & valid;
            const u64 below = bits_below(max(0, min(PAGE, n2 - lp * PAGE)));   // indices < n2 within this page
            hb = m & below;
            mb = ~m & valid & ~below;
        }
        const u64 packed = ((u64)__popcll(hb) << 32) | (u64)__popcll(mb);
        u64 tot;
        const u64 ex = block_exscan<NT / 32>(packed, &tot, warp_tot);
        long long ho = run_h + (long long)(ex >> 32), mo = run_m + (long long)(ex & 0xffffffffu);
        while (hb) {
            const int bit = __ffsll((long long)hb) - 1;
            hb &= hb - 1;
            hl[ho++] = page * PAGE + bit;
        }
        while (mb) {
            const int bit = __ffsll((long long)mb) - 1;
            mb &= mb - 1;
            ml[mo++] = page * PAGE + bit;
        }
        run_h += (long long)(tot >> 32);
        run_m += (long long)(tot & 0xffffffffu);
    }
    __syncthreads();
    if (run_h != run_m) {                       // cannot happen; guards the copy loop against bad masks
        if (threadIdx.x == 0) latch_error(cv.err, TRIMKV_E_STATE);
        return;
    }

    // phase 3: move rows (K, V by 16-byte chunks; metadata by one thread per move)
    const int rc = cv.row_bytes / 16;
    const long long work = run_h * (2 * rc + 1);
    for (long long w = threadIdx.x; w < work; w += blockDim.x) {
        const long long j = w / (2 * rc + 1);
        const int r = (int)(w % (2 * rc + 1));
        const int src = ml[j], dst = hl[j];
        const int sp = src / PAGE, so = src % PAGE, dp = dst / PAGE, dof = dst % PAGE;
        if (r == 2 * rc) {
            const size_t ss = ((size_t)b * cv.P_seq + sp) * PAGE + so, ds = ((size_t)b * cv.P_seq + dp) * PAGE + dof;
            cv.lam[ds] = cv.lam[ss];
            cv.c[ds] = cv.c[ss];
            cv.pos[ds] = cv.pos[ss];
        } else {
            const int part = r / rc, ci = r % rc;
            const char* s = cv.kv + kv_row_offset(cv, b, sp, part, so) + (size_t)phys_chunk(cv, ci, so) * 16;
            char* d = cv.kv + kv_row_offset(cv, b, dp, part, dof) + (size_t)phys_chunk(cv, ci, dof) * 16;
            *reinterpret_cast<uint4*>(d) = *reinterpret_cast<const uint4*>(s);
        }
    }
    __syncthreads();

    // phase 4: new length, release pages past the end
    const int np2 = (n2 + PAGE - 1) / PAGE;
    const int nfree = np - np2;
    if (threadIdx.x == 0) {
        cv.len[pool] = n2;
        s_freebase = nfree > 0 ? atomicAdd(&cv.free_count[b], nfree) : 0;
    }
    __syncthreads();
    for (int j = threadIdx.x; j < nfree; j += blockDim.x) {
        const int page = bt[np2 + j];
        cv.free_stack[(size_t)b * cv.P_seq + s_freebase + j] = page;
        cv.owner[(size_t)b * cv.P_seq + page] = make_int4(-1, 0, 0, 0);
    }
    if (threadIdx.x == 0 && np2 > 0)     // the new last page is the only kept page whose fill changed
        cv.owner[(size_t)b * cv.P_seq + bt[np2 - 1]] = make_int4((int)(pool % ((long long)cv.L * cv.H)), np2 - 1, n2 - (np2 - 1) * PAGE, 0);
}

// Copies one pool's entries, in storage order, to dense device buffers (undoing the chunk permutation).
__global__ void gather_pool_kernel(CacheView cv, int b, long long pool, int n, int32_t* pos, float* lam, float* c,
                                   char* k, char* v) {
    const int rc = cv.row_bytes / 16;
    const int32_t* bt = cv.block_table + pool * cv.maxpp;
    const long long work = (long long)n * (2 * rc + 1);
    for (long long w = blockIdx.x * (long long)blockDim.x + threadIdx.x; w < work;
         w += (long long)gridDim.x * blockDim.x) {
        const int i = (int)(w / (2 * rc + 1));
        const int r = (int)(w % (2 * rc + 1));
        const int page = bt[i / PAGE], off = i % PAGE;
        if (r == 2 * rc) {
            const size_t s = ((size_t)b * cv.P_seq + page) * PAGE + off;
            if (pos) pos[i] = cv.pos[s];
            if (lam) lam[i] = cv.lam[s];
            if (c) c[i] = cv.c[s];
        } else {
            const int part = r / rc, ci = r % rc;
            char* dst = part ? v : k;
            if (dst) {
                const char* s = cv.kv + kv_row_offset(cv, b, page, part, off) + (size_t)phys_chunk(cv, ci, off) * 16;
                *reinterpret_cast<uint4*>(dst + (size_t)i * cv.row_bytes + (size_t)ci * 16) =
                    *reinterpret_cast<const uint4*>(s);
            }
        }
    }
}

// c = ln sum_{k<horizon} beta^k of every live entry, from its stored lambda (Eq. (global_score), the beta-only term).
// One CTA per page; the page table says which pages are live and how far they are filled.
__global__ void __launch_bounds__(PAGE)
rehorizon_kernel(CacheView cv, int horizon) {
    const size_t pg = (size_t)blockIdx.y * cv.P_seq + blockIdx.x;
    const int4 ow = cv.owner[pg];
    if (ow.x < 0 || (int)threadIdx.x >= ow.z) return;
    const size_t slot = pg * PAGE + threadIdx.x;
    cv.c[slot] = horizon_term_f32(cv.lam[slot], horizon);
}

// Fills an EMPTY pool with n entries given as dense arrays (the inverse of gather_pool_kernel): takes pages from the
// sequence's free stack, writes rows (chunk-permuted like every stored row), metadata, page records and the length.
// One CTA.  A pool that is not empty, or a sequence without enough free pages, latches an error and changes nothing.
__global__ void __launch_bounds__(256)
import_pool_kernel(CacheView cv, int b, long long pool, int n, const int32_t* __restrict__ pos, const float* __restrict__ lam,
                   const float* __restrict__ c, const char* __restrict__ k, const char* __restrict__ v) {
    __shared__ int s_fail;
    int32_t* bt = cv.block_table + pool * cv.maxpp;
    const int np = (n + PAGE - 1) / PAGE;
    if (threadIdx.x == 0) {
        int fail = 0;
        if (cv.len[pool] != 0) fail = TRIMKV_E_STATE;
        else if (np > cv.maxpp) fail = TRIMKV_E_NOMEM;
        else {
            const int prev = atomicSub(&cv.free_count[b], np);
            if (prev < np) { atomicAdd(&cv.free_count[b], np); fail = TRIMKV_E_NOMEM; }
            else {
                const int32_t* stack = cv.free_stack + (size_t)b * cv.P_seq;
                for (int j = 0; j < np; ++j) bt[j] = stack[prev - 1 - j];
            }
        }
        if (fail) latch_error(cv.err, fail);
        s_fail = fail;
    }
    __syncthreads();
    if (s_fail) return;
    const int pool_local = (int)(pool % ((long long)cv.L * cv.H));
    const int rc = cv.row_bytes / 16;
    const long long work = (long long)n * (2 * rc + 1);
    for (long long w = threadIdx.x; w < work; w += blockDim.x) {
        const int i = (int)(w / (2 * rc + 1));
        const int r = (int)(w % (2 * rc + 1));
        const int page = bt[i / PAGE], off = i % PAGE;
        if (r == 2 * rc) {
            const size_t slot = ((size_t)b * cv.P_seq + page) * PAGE + off;
            if (lam[i] != lam[i] || c[i] != c[i]) latch_error(cv.err, TRIMKV_E_NONFINITE);
            cv.pos[slot] = pos[i];
            cv.lam[slot] = lam[i];
            cv.c[slot] = c[i];
        } else {
            const int part = r / rc, ci = r % rc;
            const char* src = (part ? v : k) + (size_t)i * cv.row_bytes + (size_t)ci * 16;
            char* dst = cv.kv + kv_row_offset(cv, b, page, part, off) + (size_t)phys_chunk(cv, ci, off) * 16;
            *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
        }
    }
    for (int lp = threadIdx.x; lp < np; lp += blockDim.x)
        cv.owner[(size_t)b * cv.P_seq + bt[lp]] = make_int4(pool_local, lp, min(PAGE, n - lp * PAGE), 0);
    __syncthreads();
    if (threadIdx.x == 0) cv.len[pool] = n;
}

// Self-check of the cache's bookkeeping (tests run it where a memory checker would otherwise be used): every pool's
// block table against the page records, every owned page against its pool, the free stack against the page records,
// positions and retention terms of live entries.  viol: OR of the violated rules; owned [B]: pages with an owner.
//   1 page id out of range   2 page record disagrees with the pool   4 owned page not referenced by its pool
//   8 free-stack entry owned or out of range   16 position outside 1..tokens   64 NaN retention term
__global__ void check_kernel(CacheView cv, long long tokens, unsigned* __restrict__ viol, unsigned* __restrict__ owned) {
    const long long gid = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    const int LH = cv.L * cv.H;
    unsigned v = 0;
    if (blockIdx.y == 0) {                                    // pools
        if (gid < (long long)cv.B * LH) {
            const int b = (int)(gid / LH), pool_local = (int)(gid % LH);
            const int n = cv.len[gid];
            if (n < 0) v |= 2;
            for (int lp = 0; lp * PAGE < n; ++lp) {
                const int page = cv.block_table[(size_t)gid * cv.maxpp + lp];
                if (page < 0 || page >= cv.P_seq) { v |= 1; continue; }
                const int4 ow = cv.owner[(size_t)b * cv.P_seq + page];
                if (ow.x != pool_local || ow.y != lp || ow.z != min(PAGE, n - lp * PAGE)) v |= 2;
            }
        }
    } else if (blockIdx.y == 1) {                             // pages
        if (gid < (long long)cv.B * cv.P_seq) {
            const int b = (int)(gid / cv.P_seq);
            const int4 ow = cv.owner[gid];
            if (ow.x >= 0) {
                atomicAdd(owned + b, 1u);
                if (ow.x >= LH) v |= 4;
                else {
                    const long long pool = (long long)b * LH + ow.x;
                    const int n = cv.len[pool];
                    if (ow.y < 0 || (long long)ow.y * PAGE >= n || cv.block_table[pool * cv.maxpp + ow.y] != (int)(gid % cv.P_seq)) v |= 4;
                    for (int off = 0; off < ow.z && off < PAGE; ++off) {
                        const size_t slot = (size_t)gid * PAGE + off;
                        const int pos = cv.pos[slot];
                        if (pos < 1 || pos > tokens) v |= 16;
                        if (cv.lam[slot] != cv.lam[slot] || cv.c[slot] != cv.c[slot]) v |= 64;
                    }
                }
            }
        }
    } else {                                                  // free stacks
        if (gid < (long long)cv.B * cv.P_seq) {
            const int b = (int)(gid / cv.P_seq);
            const long long i = gid % cv.P_seq;
            if (i < cv.free_count[b]) {
                const int page = cv.free_stack[gid];
                if (page < 0 || page >= cv.P_seq || cv.owner[(size_t)b * cv.P_seq + page].x >= 0) v |= 8;
            }
        }
    }
    if (v) atomicOr(viol, v);
}

}  // namespace

void launch_import_pool(const CacheView& cv, int seq, int layer, int head, int n, const int32_t* pos, const float* lam,
                        const float* c, const void* k, const void* v, cudaStream_t st) {
    if (n <= 0) return;
    const long long pool = ((long long)seq * cv.L + layer) * cv.H + head;
    import_pool_kernel<<<1, 256, 0, st>>>(cv, seq, pool, n, pos, lam, c, (const char*)k, (const char*)v);
    count_launch();
}

void launch_check(const CacheView& cv, long long tokens, unsigned* viol, unsigned* owned, cudaStream_t st) {
    const long long work = std::max<long long>((long long)cv.B * cv.P_seq, (long long)cv.B * cv.L * cv.H);
    dim3 grid((unsigned)((work + 255) / 256), 3);
    check_kernel<<<grid, 256, 0, st>>>(cv, tokens, viol, owned);
    count_launch();
}

void launch_append(const CacheView& cv, int layer0, int nlayers, int n_new, long long pos0, const float* lam,
                   const float* c, int horizon, const void* k, const void* v, int mode, cudaStream_t st) {
    const int grid = nlayers * cv.B * cv.H;
    const bool split = (mode & APPEND_KV) && n_new >= 4 * APPEND_TOK;     // a chunk: copy its rows with a grid of their own
    const int threads = n_new <= 2 ? 64 : 256;        // a decode step's row pair is 64 chunks: small CTAs, all resident at once
    append_kernel<<<grid, threads, 0, st>>>(cv, layer0, n_new, pos0, lam, c, horizon, (const char*)k, (const char*)v,
                                            split ? (mode | APPEND_ROWS_ELSEWHERE) : mode);
    count_launch();
    if (split) {
        dim3 g2(grid, (n_new + APPEND_TOK - 1) / APPEND_TOK);
        append_rows_kernel<<<g2, 256, 0, st>>>(cv, layer0, n_new, (const char*)k, (const char*)v);
        count_launch();
    }
}

void launch_compact(const CacheView& cv, int32_t* hole, int32_t* mover, int32_t* cursor, long long e_max,
                    long long evictions_per_seq, cudaStream_t st) {
    const long long pools = (long long)cv.B * cv.L * cv.H;
    if (evictions_per_seq <= 4LL * cv.L * cv.H)
        compact_kernel<128><<<(unsigned)pools, 128, 0, st>>>(cv, hole, mover, cursor, e_max);
    else
        compact_kernel<256><<<(unsigned)pools, 256, 0, st>>>(cv, hole, mover, cursor, e_max);
    count_launch();
}

void launch_rehorizon(const CacheView& cv, int horizon, cudaStream_t st) {
    dim3 grid((unsigned)cv.P_seq, (unsigned)cv.B);
    rehorizon_kernel<<<grid, PAGE, 0, st>>>(cv, horizon);
    count_launch();
}

void launch_gather_pool(const CacheView& cv, int seq, int layer, int head, int32_t* pos, float* lam, float* c, void* k,
                        void* v, int n, cudaStream_t st) {
    if (n <= 0) return;
    const long long pool = ((long long)seq * cv.L + layer) * cv.H + head;
    gather_pool_kernel<<<64, 256, 0, st>>>(cv, seq, pool, n, pos, lam, c, (char*)k, (char*)v);
    count_launch();
}

}  // namespace tkv
