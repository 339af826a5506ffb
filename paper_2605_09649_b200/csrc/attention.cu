// Decode attention over the ragged per-(layer, head) pools (Sec. 2.1 softmax attention restricted to
// the retained set, Eq. (1) with r in {0,1}; GQA: query head j reads the pool of KV head j / g).
//
// bf16, d = 128 path ("split-KV"): the pools of the call are cut into work items of a fixed number of
// 32-entry tiles.  Each warp is an independent worker: lane 0 streams its tiles' K and V rows from HBM
// to shared memory with bulk asynchronous copies (cp.async.bulk + mbarrier, 3 stages of 16 KB per warp),
// the warp computes S^T = K Q^T and O^T += V^T P^T with mma.sync m16n8k16 (the GQA group is the N
// dimension, so no tensor-core work is spent on padding rows), keeps an online softmax in registers with
// warp-shuffle reductions over the entries, and writes (m, l, O) partials.  The warp that finishes the last item
// of a pool (a per-pool ticket) merges that pool's partials and writes the output, so no second kernel is needed.
// The kernel is bound by HBM bandwidth: every K/V byte is read once.
//
// Any other shape / fp32 uses a plain one-warp-per-query-head kernel.
#include <algorithm>

#include "async_copy.cuh"
#include "mma_sync.cuh"
#include "trimkv_internal.cuh"

namespace tkv {

namespace {

constexpr int TILE = 32;                       // entries per pipeline stage
constexpr int ATT_WARPS = 4;
constexpr int ATT_STAGES = 3;
constexpr int ROWB = 256;                      // bytes per K or V row (d = 128, bf16)
constexpr int STAGE_BYTES = 2 * TILE * ROWB;   // K tile + V tile
constexpr int ATT_MAX_TPI = 512;               // tiles per work item, at most (page ids are fetched 32 at a time)
constexpr int ATT_GROUPS = 1024;               // pool groups of the in-kernel item table
constexpr int ATT_BAR_OFF = ATT_WARPS * ATT_STAGES * STAGE_BYTES;
constexpr int ATT_GRP_OFF = ATT_BAR_OFF + 256;
constexpr int ATT_RING = 8;                    // per-warp queue of item ids fetched by the producer, read by the consumer
constexpr int ATT_RING_OFF = ATT_GRP_OFF + (ATT_GROUPS + 1) * 4 + 12;
constexpr int ATT_META_OFF = (ATT_RING_OFF + ATT_WARPS * ATT_RING * 4 + 127) & ~127;   // per warp and stage: lambda[32], pos[32]
constexpr int ATT_META_BYTES = 2 * TILE * 4;
constexpr int ATT_SMEM = ATT_META_OFF + ATT_WARPS * ATT_STAGES * ATT_META_BYTES;
constexpr unsigned WAIT_LIMIT_TEST = 1u << 8;  // the limit of the testing aid under which no copy is ever issued

// ------------------------------------------------------------------ work plan
// Scope = pools of layers [layer0, layer0 + nlayers): scope index si = (lb * B + b) * H + h.
__device__ __forceinline__ long long scope_pool(const CacheView& cv, int layer0, int si) {
    const int h = si % cv.H;
    const int b = (si / cv.H) % cv.B;
    const int lb = si / (cv.H * cv.B);
    return ((long long)b * cv.L + layer0 + lb) * cv.H + h;
}

// ------------------------------------------------------------------ bf16 / d = 128 worker kernel
struct ItemCtx {
    int item;        // global item index, -1 = none
    int si;          // scope index
    int b;           // sequence
    int first_tile;  // first tile of the item inside its pool
    int ntile;       // tiles in the item
    int len;         // pool length
    int pool_items;  // items of this pool
    int pool_base;   // global index of the pool's first item
    int page_id;     // lane i holds the physical page of the item's i-th page
};

// A pool of `len` entries is cut into items_of_len() items of tiles_per_item() tiles each (the last one shorter):
// as few items as the cap of tpi tiles per item allows, of equal size, each starting on a page boundary.
// Items are handed out in pool order, so the pools at the end of the scope are the tail of the launch: the last eighth of
// the pools is cut into items a quarter of the size, which shortens the stretch in which a few warps finish alone.
// Measured at the Llama shape, step time: pool lengths 0..33.7K 0.751 -> 0.728 ms, 18..33.7K 0.74 -> 0.715, equal pools
// unchanged (0.70; restricting the rule to pools that are cut anyway lost the gain for the second case).
__device__ __forceinline__ int tail_tpi(int si, int n_scope, int tpi) {
    return ((long long)si * 8 >= (long long)n_scope * 7) ? max(2, ((tpi >> 2) + 1) & ~1) : tpi;
}
__device__ __forceinline__ int items_of_len(int len, int tpi) {
    const int tiles = (len + TILE - 1) / TILE;
    return (tiles + tpi - 1) / tpi;
}
__device__ __forceinline__ int tiles_per_item(int len, int items) {
    const int tiles = (len + TILE - 1) / TILE;
    return (((tiles + items - 1) / items) + 1) & ~1;
}

// NT = ceil(g / 8): column tiles of 8 query heads.  BIAS: retention-gated weights beta_i^(t-i) e^{z_i} (Sec. 2.2): the
// entries' lambda and position travel with each tile and (t_now - pos) * lambda is added to the logit.
// NO_COPY (testing aid): the producer issues no asynchronous copy at all and the waits use a short limit, so every
// wait runs out with nothing in flight: the kernel latches TRIMKV_E_TIMEOUT and returns; its output is not written.
template <int NT, bool BIAS, bool NO_COPY = false>
__global__ void __launch_bounds__(ATT_WARPS * 32, 1)
attn_mma_kernel(CacheView cv, int layer0, int n_scope, int tpi, int gsz, int g, int Hq, int t_now, int32_t* __restrict__ pool_done,
                int32_t* __restrict__ sched,
                const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ out, float* __restrict__ part_o,
                float* __restrict__ part_ml, float scale_log2, long long max_items) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned char* wbuf = smem_raw + (size_t)warp * ATT_STAGES * STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw + ATT_BAR_OFF) + warp * ATT_STAGES;
    int* grp = reinterpret_cast<int*>(smem_raw + ATT_GRP_OFF);     // grp[i] = items before pool group i
    volatile int* ring = reinterpret_cast<volatile int*>(smem_raw + ATT_RING_OFF) + warp * ATT_RING;
    unsigned char* meta = smem_raw + ATT_META_OFF + (size_t)warp * ATT_STAGES * ATT_META_BYTES;

    // ---- item table: items per group of gsz pools, then an exclusive scan (every CTA computes the same table)
    const int ngrp = (n_scope + gsz - 1) / gsz;
    for (int gi = threadIdx.x; gi <= ngrp; gi += blockDim.x) grp[gi] = 0;
    __syncthreads();
#pragma unroll 4
    for (int si = threadIdx.x; si < n_scope; si += blockDim.x) {        // independent, coalesced length loads
        const int len = cv.len[scope_pool(cv, layer0, si)];
        const int it = items_of_len(len, tail_tpi(si, n_scope, tpi));
        if (it) atomicAdd(&grp[si / gsz + 1], it);
        if (len == 0 && blockIdx.x == 0) {              // an empty pool has no item: its outputs are zero
            __nv_bfloat16* op = out + ((size_t)(si / cv.H) * Hq + (size_t)(si % cv.H) * g) * 128;
            for (int e = 0; e < g * 128; ++e) op[e] = __float2bfloat16_rn(0.f);
        }
    }
    // stale shared memory must hold finite values: masked entries still multiply V rows by zero
    for (int i = lane * 16; i < ATT_STAGES * STAGE_BYTES; i += 32 * 16)
        *reinterpret_cast<uint4*>(wbuf + i) = make_uint4(0u, 0u, 0u, 0u);
    if (lane == 0) {
        for (int s = 0; s < ATT_STAGES; ++s) mbar_init(bars + s, 1);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (warp == 0) {                                      // exclusive scan of the group sums by one warp
        const int per = (ngrp + 31) / 32;
        const int g0 = lane * per, g1 = min(ngrp, g0 + per);
        int local = 0;
        for (int gi = g0; gi < g1; ++gi) local += grp[gi + 1];
        int incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        int run = incl - local;
        for (int gi = g0; gi < g1; ++gi) {
            const int v = grp[gi + 1];
            grp[gi + 1] = run + v;                        // inclusive: grp[gi + 1] = items before group gi + 1
            run += v;
        }
        if (lane == 0) grp[0] = 0;
    }
    __syncthreads();
    const int all_items = grp[ngrp];
    if (all_items > max_items && threadIdx.x == 0 && blockIdx.x == 0) latch_error(cv.err, TRIMKV_E_NOMEM);
    const int total_items = (int)min((long long)all_items, max_items);
    const int gw = blockIdx.x * ATT_WARPS + warp;
    const int GW = gridDim.x * ATT_WARPS;

    auto load_item = [&](int item) -> ItemCtx {
        ItemCtx c;
        c.item = -1; c.si = 0; c.b = 0; c.first_tile = 0; c.ntile = 0; c.len = 0; c.pool_items = 0; c.pool_base = 0; c.page_id = 0;
        if (item >= total_items) return c;
        int lo = 0, hi = ngrp - 1;                       // last group whose first item is <= item
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (grp[mid] <= item) lo = mid; else hi = mid - 1;
        }
        int base = grp[lo], si = lo * gsz, len = 0, cnt = 0;
        const int si_end = min(n_scope, (lo + 1) * gsz);
        bool found = false;
        for (; si < si_end; ++si) {                       // ends inside the group: item < grp[lo + 1]
            len = cv.len[scope_pool(cv, layer0, si)];
            cnt = items_of_len(len, tail_tpi(si, n_scope, tpi));
            if (item < base + cnt) { found = true; break; }
            base += cnt;
        }
        if (!found) return c;
        c.item = item;
        c.si = si;
        c.len = len;
        c.pool_items = cnt;
        c.pool_base = base;
        const int per = tiles_per_item(len, cnt);
        c.first_tile = (item - base) * per;
        const long long pool = scope_pool(cv, layer0, si);
        c.b = (si / cv.H) % cv.B;
        const int tiles = (len + TILE - 1) / TILE;
        c.ntile = max(0, min(per, tiles - c.first_tile));
        const int npage_item = (c.ntile + 1) / 2;
        c.page_id = (lane < npage_item) ? cv.block_table[pool * cv.maxpp + c.first_tile / 2 + lane] : 0;
        return c;
    };

    // Items are handed out dynamically (ragged pools make a static split uneven): a warp starts with item gw and then
    // takes GW + (a global counter), one item at a time.  The producer runs ahead of the consumer by at most the
    // pipeline depth, so a short per-warp ring of item ids links the two.
    ItemCtx prod = load_item(gw), cons = prod;
    int prod_tile = 0;
    unsigned issued = 0, consumed = 0;
    unsigned prod_seq = prod.item >= 0 ? 1u : 0u, cons_seq = 0;
    if (lane == 0) ring[0] = gw;
    __syncwarp();
    bool failed = false;

    auto issue_one = [&]() {   // issue the producer cursor's tile into stage (issued % STAGES), advance
        if (prod.item < 0) return;
        const int tt = prod_tile;
        if (tt > 0 && (tt & 63) == 0) {                  // next 32 pages of a long item
            const long long pool = scope_pool(cv, layer0, prod.si);
            const int left = (prod.ntile - tt + 1) / 2;
            prod.page_id = (lane < left) ? cv.block_table[pool * cv.maxpp + (prod.first_tile + tt) / 2 + lane] : 0;
        }
        const int page = __shfl_sync(0xffffffffu, prod.page_id, (tt >> 1) & 31);
        const int half = (prod.first_tile + tt) & 1;
        if (lane == 0 && !NO_COPY) {
            const unsigned s = issued % ATT_STAGES;
            unsigned char* dst = wbuf + (size_t)s * STAGE_BYTES;
            const char* ksrc = cv.kv + kv_row_offset(cv, prod.b, page, 0, half * TILE);
            const char* vsrc = cv.kv + kv_row_offset(cv, prod.b, page, 1, half * TILE);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_expect_tx(bars + s, STAGE_BYTES + (BIAS ? ATT_META_BYTES : 0));
            bulk_g2s(dst, ksrc, TILE * ROWB, bars + s);
            bulk_g2s(dst + TILE * ROWB, vsrc, TILE * ROWB, bars + s);
            if (BIAS) {
                const size_t slot0 = ((size_t)prod.b * cv.P_seq + page) * PAGE + half * TILE;
                bulk_g2s(meta + s * ATT_META_BYTES, cv.lam + slot0, TILE * 4, bars + s);
                bulk_g2s(meta + s * ATT_META_BYTES + TILE * 4, cv.pos + slot0, TILE * 4, bars + s);
            }
        }
        ++issued;
        if (++prod_tile == prod.ntile) {
            int nxt = 0;
            if (lane == 0) nxt = GW + atomicAdd(sched, 1);
            nxt = __shfl_sync(0xffffffffu, nxt, 0);
            prod = load_item(nxt);                        // item = -1 past the end: the producer then stays idle
            prod_tile = 0;
            if (prod.item >= 0) {
                if (lane == 0) ring[prod_seq % ATT_RING] = nxt;
                ++prod_seq;
                __syncwarp();
            }
        }
    };

    for (int s = 0; s < ATT_STAGES - 1; ++s) issue_one();

    // per-item state
    uint32_t bq[NT][8][2];
    float o[NT][8][4];
    float m_run[NT][2], l_run[NT][2];

    while (cons.item >= 0 && !failed) {
        // ---- item prologue: Q fragments (B operand of S^T = K Q^T: k = d, n = query head)
        const int h = cons.si % cv.H;
        const int lbb = cons.si / cv.H;   // lb * B + b
        const __nv_bfloat16* qb = q + ((size_t)lbb * Hq + (size_t)h * g) * 128;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int head = nt * 8 + (lane >> 2);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                uint32_t v0 = 0u, v1 = 0u;
                if (head < g) {
                    const __nv_bfloat16* p = qb + (size_t)head * 128 + ks * 16 + 2 * (lane & 3);
                    v0 = *reinterpret_cast<const uint32_t*>(p);
                    v1 = *reinterpret_cast<const uint32_t*>(p + 8);
                }
                bq[nt][ks][0] = v0;
                bq[nt][ks][1] = v1;
            }
#pragma unroll
            for (int dt = 0; dt < 8; ++dt) { o[nt][dt][0] = o[nt][dt][1] = o[nt][dt][2] = o[nt][dt][3] = 0.f; }
            m_run[nt][0] = m_run[nt][1] = -INFINITY;
            l_run[nt][0] = l_run[nt][1] = 0.f;
        }

        for (int tt = 0; tt < cons.ntile; ++tt) {
            issue_one();    // refill the stage freed by the previous tile
            const unsigned s = consumed % ATT_STAGES;
            if (!mbar_wait_bounded(bars + s, (consumed / ATT_STAGES) & 1u, NO_COPY ? WAIT_LIMIT_TEST : WAIT_LIMIT)) { failed = true; break; }
            ++consumed;
            const uint32_t kbase = smem_u32(wbuf + (size_t)s * STAGE_BYTES);
            const uint32_t vbase = kbase + TILE * ROWB;
            const int valid = min(TILE, cons.len - (cons.first_tile + tt) * TILE);
            float rb[2][2] = {{0.f, 0.f}, {0.f, 0.f}};           // log2-domain retention bias of this thread's four rows
            if (BIAS) {
                const float* mlam = reinterpret_cast<const float*>(meta + s * ATT_META_BYTES);
                const int* mpos = reinterpret_cast<const int*>(meta + s * ATT_META_BYTES + TILE * 4);
#pragma unroll
                for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int r = mt * 16 + hh * 8 + (lane >> 2);
                        // age 0 (the token of this step): beta^0 = 1 whatever lambda is; its stored lambda may not be
                        // written yet, and 0 * -inf would be NaN
                        const int age = t_now - mpos[r];
                        rb[mt][hh] = age == 0 ? 0.f : (float)age * mlam[r] * 1.4426950408889634f;
                    }
            }

            // ---- S^T[entry][head] = K Q^T
            float sacc[2][NT][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) sacc[mt][nt][0] = sacc[mt][nt][1] = sacc[mt][nt][2] = sacc[mt][nt][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    const int row = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                    const int chunk = (2 * ks + (lane >> 4)) ^ (row & 7);
                    uint32_t a[4];
                    ldsm_x4(a, kbase + row * ROWB + chunk * 16);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) mma_bf16(sacc[mt][nt], a, bq[nt][ks][0], bq[nt][ks][1]);
                }
            }
            // ---- online softmax over the entries (rows); this thread owns heads 2*(lane&3), +1 of each nt
            uint32_t pb[2][NT][2];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    const int r0 = mt * 16 + (lane >> 2);
                    float* sc = sacc[mt][nt];
                    sc[0] = (r0 < valid) ? sc[0] * scale_log2 + rb[mt][0] : -INFINITY;
                    sc[1] = (r0 < valid) ? sc[1] * scale_log2 + rb[mt][0] : -INFINITY;
                    sc[2] = (r0 + 8 < valid) ? sc[2] * scale_log2 + rb[mt][1] : -INFINITY;
                    sc[3] = (r0 + 8 < valid) ? sc[3] * scale_log2 + rb[mt][1] : -INFINITY;
                    mx0 = fmaxf(mx0, fmaxf(sc[0], sc[2]));
                    mx1 = fmaxf(mx1, fmaxf(sc[1], sc[3]));
                }
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) {
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
                }
                const float mn0 = fmaxf(m_run[nt][0], mx0), mn1 = fmaxf(m_run[nt][1], mx1);
                const float f0 = exp2f(m_run[nt][0] - mn0), f1 = exp2f(m_run[nt][1] - mn1);   // 0 on the first tile
                m_run[nt][0] = mn0;
                m_run[nt][1] = mn1;
                float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    float* sc = sacc[mt][nt];
                    const __nv_bfloat162 plo = __floats2bfloat162_rn(exp2f(sc[0] - mn0), exp2f(sc[1] - mn1));
                    const __nv_bfloat162 phi = __floats2bfloat162_rn(exp2f(sc[2] - mn0), exp2f(sc[3] - mn1));
                    ls0 += __low2float(plo) + __low2float(phi);     // sum what the tensor cores will see
                    ls1 += __high2float(plo) + __high2float(phi);
                    pb[mt][nt][0] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&plo));
                    pb[mt][nt][1] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&phi));
                }
                l_run[nt][0] = l_run[nt][0] * f0 + ls0;
                l_run[nt][1] = l_run[nt][1] * f1 + ls1;
#pragma unroll
                for (int dt = 0; dt < 8; ++dt) {
                    o[nt][dt][0] *= f0; o[nt][dt][1] *= f1; o[nt][dt][2] *= f0; o[nt][dt][3] *= f1;
                }
            }
            // ---- O^T[d][head] += V^T P^T
#pragma unroll
            for (int dt = 0; dt < 8; ++dt) {
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    const int row = mt * 16 + (lane & 7) + (lane >> 4) * 8;
                    const int chunk = (2 * dt + ((lane >> 3) & 1)) ^ (row & 7);
                    uint32_t a[4];
                    ldsm_x4_trans(a, vbase + row * ROWB + chunk * 16);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) mma_bf16(o[nt][dt], a, pb[mt][nt][0], pb[mt][nt][1]);
                }
            }
            __syncwarp();   // all lanes are done reading this stage before it is refilled
        }
        if (failed) break;

        // ---- item epilogue.  A pool with a single item is finished here; otherwise the partial (m, l, O) is stored
        // and the warp that completes the pool's last item merges all of them.
        const bool single = cons.pool_items == 1;
        __nv_bfloat16* outp = out + ((size_t)lbb * Hq + (size_t)h * g) * 128;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            float l0 = l_run[nt][0], l1 = l_run[nt][1];
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                l0 += __shfl_xor_sync(0xffffffffu, l0, off);
                l1 += __shfl_xor_sync(0xffffffffu, l1, off);
            }
            const int head0 = nt * 8 + 2 * (lane & 3);
            if (single) {
                const float r0 = l0 > 0.f ? 1.0f / l0 : 0.f, r1 = l1 > 0.f ? 1.0f / l1 : 0.f;
#pragma unroll
                for (int dt = 0; dt < 8; ++dt) {
                    const int dr = dt * 16 + (lane >> 2);
                    if (head0 < g) {
                        outp[(size_t)head0 * 128 + dr] = __float2bfloat16_rn(o[nt][dt][0] * r0);
                        outp[(size_t)head0 * 128 + dr + 8] = __float2bfloat16_rn(o[nt][dt][2] * r0);
                    }
                    if (head0 + 1 < g) {
                        outp[(size_t)(head0 + 1) * 128 + dr] = __float2bfloat16_rn(o[nt][dt][1] * r1);
                        outp[(size_t)(head0 + 1) * 128 + dr + 8] = __float2bfloat16_rn(o[nt][dt][3] * r1);
                    }
                }
                continue;
            }
            if ((lane >> 2) == 0) {
                if (head0 < g) {
                    part_ml[((size_t)cons.item * g + head0) * 2 + 0] = m_run[nt][0];
                    part_ml[((size_t)cons.item * g + head0) * 2 + 1] = l0;
                }
                if (head0 + 1 < g) {
                    part_ml[((size_t)cons.item * g + head0 + 1) * 2 + 0] = m_run[nt][1];
                    part_ml[((size_t)cons.item * g + head0 + 1) * 2 + 1] = l1;
                }
            }
#pragma unroll
            for (int dt = 0; dt < 8; ++dt) {
                const int dr = dt * 16 + (lane >> 2);
                if (head0 < g) {
                    float* po = part_o + ((size_t)cons.item * g + head0) * 128;
                    po[dr] = o[nt][dt][0];
                    po[dr + 8] = o[nt][dt][2];
                }
                if (head0 + 1 < g) {
                    float* po = part_o + ((size_t)cons.item * g + head0 + 1) * 128;
                    po[dr] = o[nt][dt][1];
                    po[dr + 8] = o[nt][dt][3];
                }
            }
        }
        if (!single) {
            __threadfence();                              // partials visible before the ticket
            __syncwarp();
            int ticket = 0;
            if (lane == 0) ticket = atomicAdd(pool_done + cons.si, 1);
            ticket = __shfl_sync(0xffffffffu, ticket, 0);
            if (ticket == cons.pool_items - 1) {          // this warp completed the pool: merge
                __threadfence();
                if (lane == 0) pool_done[cons.si] = 0;    // ready for the next call
                const int i0 = cons.pool_base, i1 = min(cons.pool_base + cons.pool_items, total_items);
                const int n = i1 - i0;
                constexpr int GM = NT * 8;
                // (m, l) of every item and head: lane t holds item t0 + t; running max and denominator per head
                float Mj[GM], Dj[GM];
#pragma unroll
                for (int j = 0; j < GM; ++j) { Mj[j] = -INFINITY; Dj[j] = 0.f; }
                for (int t0 = 0; t0 < n; t0 += 32) {
                    const int t = t0 + lane;
                    float mj[GM], lj[GM];
#pragma unroll
                    for (int j = 0; j < GM; ++j) {
                        mj[j] = -INFINITY; lj[j] = 0.f;
                        if (j < g && t < n) {
                            const float2 v = __ldcg(reinterpret_cast<const float2*>(part_ml + ((size_t)(i0 + t) * g + j) * 2));
                            mj[j] = v.x; lj[j] = v.y;
                        }
                    }
#pragma unroll
                    for (int j = 0; j < GM; ++j) {
                        if (j < g) {
                            float mx = mj[j];
#pragma unroll
                            for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
                            const float Mn = fmaxf(Mj[j], mx);
                            float d = exp2f(mj[j] - Mn) * lj[j];
#pragma unroll
                            for (int off = 16; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
                            Dj[j] = Dj[j] * exp2f(Mj[j] - Mn) + d;
                            Mj[j] = Mn;
                        }
                    }
                }
                // O: four heads at a time, two items per batch (8 independent 16-byte loads per lane in flight)
#pragma unroll
                for (int jq = 0; jq < GM; jq += 4) {
                    if (jq < g) {
                        float4 num[4];
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj) num[jj] = make_float4(0.f, 0.f, 0.f, 0.f);
                        for (int t = 0; t < n; t += 2) {
                            float4 po[2][4];
                            float mm[2][4];
#pragma unroll
                            for (int u = 0; u < 2; ++u)
#pragma unroll
                                for (int jj = 0; jj < 4; ++jj) {
                                    po[u][jj] = make_float4(0.f, 0.f, 0.f, 0.f);
                                    mm[u][jj] = -INFINITY;
                                    if (t + u < n && jq + jj < g) {
                                        const size_t row = (size_t)(i0 + t + u) * g + jq + jj;
                                        po[u][jj] = __ldcg(reinterpret_cast<const float4*>(part_o + row * 128) + lane);
                                        mm[u][jj] = __ldcg(part_ml + row * 2);
                                    }
                                }
#pragma unroll
                            for (int u = 0; u < 2; ++u)
#pragma unroll
                                for (int jj = 0; jj < 4; ++jj) {
                                    const float w = exp2f(mm[u][jj] - Mj[jq + jj]);     // 0 for the padded slots
                                    num[jj].x += w * po[u][jj].x; num[jj].y += w * po[u][jj].y;
                                    num[jj].z += w * po[u][jj].z; num[jj].w += w * po[u][jj].w;
                                }
                        }
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj) {
                            if (jq + jj < g) {
                                const float r = Dj[jq + jj] > 0.f ? 1.0f / Dj[jq + jj] : 0.f;
                                __nv_bfloat162 a = __floats2bfloat162_rn(num[jj].x * r, num[jj].y * r);
                                __nv_bfloat162 c2 = __floats2bfloat162_rn(num[jj].z * r, num[jj].w * r);
                                uint2 pk;
                                pk.x = *reinterpret_cast<uint32_t*>(&a);
                                pk.y = *reinterpret_cast<uint32_t*>(&c2);
                                *reinterpret_cast<uint2*>(outp + (size_t)(jq + jj) * 128 + lane * 4) = pk;
                            }
                        }
                    }
                }
            }
        }
        // next item of this warp: the producer has already moved past the one just finished
        ++cons_seq;
        if (cons_seq < prod_seq) {
            const int id = ring[cons_seq % ATT_RING];
            cons = (prod.item == id) ? prod : load_item(id);
        } else {
            cons.item = -1;
        }
    }

    if (failed) {
        latch_error(cv.err, TRIMKV_E_TIMEOUT);
        // drain: wait (bounded) for the copies still in flight before leaving shared memory
        while (!NO_COPY && consumed < issued) {
            const unsigned s = consumed % ATT_STAGES;
            mbar_wait_bounded(bars + s, (consumed / ATT_STAGES) & 1u);
            ++consumed;
        }
    }
    // the last warp of the grid to finish rearms the item counter for the next launch
    if (lane == 0) {
        const int d = atomicAdd(sched + 1, 1);
        if (d == GW - 1) { sched[0] = 0; sched[1] = 0; }
    }
}

// ------------------------------------------------------------------ plain kernel: any d, fp32 or bf16
// One warp per (pool in scope, query head of its group).  Lanes split d; per entry one warp reduction.
template <typename T, int MAXD>
__global__ void __launch_bounds__(128)
attn_plain_kernel(CacheView cv, int layer0, int n_scope, int g, int Hq, const T* __restrict__ q, T* __restrict__ out,
                  float scale, int bias, int t_now) {
    const int wid = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (wid >= n_scope * g) return;
    const int si = wid / g, j = wid % g;
    const int h = si % cv.H, lbb = si / cv.H, b = lbb % cv.B;
    const long long pool = scope_pool(cv, layer0, si);
    const int n = cv.len[pool];
    const int d = cv.d;
    constexpr int PER = MAXD / 32;
    const int epc = 16 / (int)sizeof(T);          // elements per 16-byte chunk
    float qr[PER], acc[PER];
    const T* qp = q + ((size_t)lbb * Hq + (size_t)h * g + j) * d;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int dd = lane + 32 * i;
        qr[i] = dd < d ? to_f32<T>(qp[dd]) * scale : 0.f;
        acc[i] = 0.f;
    }
    float m = -INFINITY, l = 0.f;
    const int32_t* bt = cv.block_table + pool * cv.maxpp;
    for (int e = 0; e < n; ++e) {
        const int page = bt[e / PAGE], off = e % PAGE;
        const T* kr = reinterpret_cast<const T*>(cv.kv + kv_row_offset(cv, b, page, 0, off));
        const T* vr = reinterpret_cast<const T*>(cv.kv + kv_row_offset(cv, b, page, 1, off));
        float s = 0.f;
        int pidx[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int dd = lane + 32 * i;
            pidx[i] = phys_chunk(cv, dd / epc, off) * epc + dd % epc;
            if (dd < d) s = fmaf(qr[i], to_f32<T>(kr[pidx[i]]), s);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (bias) {                                       // retention-gated weights: + (t - i) * lambda_i
            const size_t slot = ((size_t)b * cv.P_seq + page) * PAGE + off;
            const int age = t_now - cv.pos[slot];
            if (age != 0) s += (float)age * cv.lam[slot];     // age 0: beta^0 = 1 (and 0 * -inf would be NaN)
        }
        const float mn = fmaxf(m, s);
        const float f = __expf(m - mn), p = __expf(s - mn);
        l = l * f + p;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int dd = lane + 32 * i;
            if (dd < d) acc[i] = acc[i] * f + p * to_f32<T>(vr[pidx[i]]);
        }
        m = mn;
    }
    T* op = out + ((size_t)lbb * Hq + (size_t)h * g + j) * d;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int dd = lane + 32 * i;
        if (dd < d) op[dd] = from_f32<T>(n > 0 ? acc[i] / l : 0.f);
    }
}

}  // namespace

void launch_attention(const CacheView& cv, const AttnBuffers& ab, int layer0, int nlayers, int Hq, int is_bf16,
                      long long tiles_estimate, long long tiles_upper, int retention_bias, long long t_now, int reserve_sms,
                      bool test_no_copy, const void* q, void* out, cudaStream_t st, PhaseMarker* pm) {
    const int n_scope = nlayers * cv.B * cv.H;
    const int g = Hq / cv.H;
    const float scale = 1.0f / sqrtf((float)cv.d);
    if (is_bf16 && cv.d == 128 && g <= 16) {
        if (first_use_on_device(0)) {
            cudaFuncSetAttribute(attn_mma_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM);
            cudaFuncSetAttribute(attn_mma_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM);
            cudaFuncSetAttribute(attn_mma_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM);
            cudaFuncSetAttribute(attn_mma_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM);
            cudaFuncSetAttribute(attn_mma_kernel<1, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM);
        }
        int dev = 0, sms = 148;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        // The kernel is bound by HBM long before it needs every SM.  SMs left free take the one-CTA-per-sequence kernels of
        // the selection (1024 threads each: they cannot share an SM with a resident attention CTA, whose registers leave
        // room for 512 more threads at most) while the attention kernel is still running.
        sms = std::max(sms - std::max(reserve_sms, 0), (sms * 3 + 3) / 4);
        const long long workers = (long long)sms * ATT_WARPS;
        // Items of about half a worker's share: most pools are then one item and need no merge, while a pool that
        // dominates the cache is still cut up.  (Few warps suffice to saturate HBM, so coarse items cost no bandwidth.)
        // (A cross-warp merge costs a device-scope fence per item, which drains the warp's copy pipeline.)
        long long tpi = tiles_estimate / (workers * 2);
        // ... but no coarser than a little above the average pool, down to a quarter of a worker's share: equal pools
        // stay whole either way, while the few long pools of a ragged cache are cut finer and balance better
        // (measured with pool lengths 17..32813: 0.786 -> 0.74 ms per step; equal pools: unchanged).
        if (n_scope > 0) {
            const long long avg = tiles_estimate / n_scope;
            tpi = std::min(tpi, std::max(avg + avg / 4 + 1, tiles_estimate / (workers * 4)));
        }
        // With at least half as many pools as workers and short pools (up to 4096 entries on average), whole pools are the
        // better items even when they are shorter than that: nothing is merged (the per-item fence weighs most on short
        // items), and the warps that get no item are not missed (HBM is saturated by a third of them).  Measured: workload
        // qwen_vl_16k 99 -> 94 us; longer pools (stress_128k: 8192 entries) do better cut in three.
        if ((long long)n_scope * 2 >= workers) {
            const long long avg = tiles_estimate / n_scope;
            if (avg <= 128) tpi = std::max(tpi, avg + avg / 4 + 1);
        }
        const long long room = ab.max_items - n_scope;          // items <= 1.5 tiles / tpi + n_scope must fit (the last eighth
                                                                // of the pools is cut four times finer)
        if (room > 0) tpi = std::max(tpi, (tiles_upper * 3 / 2 + room - 1) / room);
        tpi = (tpi + 1) & ~1LL;
        if (tpi < 2) tpi = 2;
        if (tpi > ATT_MAX_TPI) tpi = ATT_MAX_TPI;
        int gsz = 1;
        while ((n_scope + gsz - 1) / gsz > ATT_GROUPS) gsz <<= 1;
        if (pm) pm->mark(PH_ATTN_MAIN, 0, st);
        const float scale_log2 = scale * 1.4426950408889634f;
        auto launch = [&](auto kernel) {
            kernel<<<sms, ATT_WARPS * 32, ATT_SMEM, st>>>(cv, layer0, n_scope, (int)tpi, gsz, g, Hq, (int)t_now, ab.pool_done, ab.sched,
                                                          (const __nv_bfloat16*)q, (__nv_bfloat16*)out, ab.part_o, ab.part_ml,
                                                          scale_log2, ab.max_items);
        };
        if (test_no_copy) launch(attn_mma_kernel<1, false, true>);      // testing aid: every wait runs out (see the kernel)
        else if (g <= 8) { if (retention_bias) launch(attn_mma_kernel<1, true>); else launch(attn_mma_kernel<1, false>); }
        else        { if (retention_bias) launch(attn_mma_kernel<2, true>); else launch(attn_mma_kernel<2, false>); }
        if (pm) pm->mark(PH_ATTN_MAIN, 1, st);
        count_launch(1);
    } else {
        const int warps = n_scope * g;
        const int grid = (warps + 3) / 4;
        if (pm) pm->mark(PH_ATTN_MAIN, 0, st);
        if (is_bf16)
            attn_plain_kernel<__nv_bfloat16, 256><<<grid, 128, 0, st>>>(cv, layer0, n_scope, g, Hq, (const __nv_bfloat16*)q,
                                                                         (__nv_bfloat16*)out, scale, retention_bias, (int)t_now);
        else
            attn_plain_kernel<float, 256><<<grid, 128, 0, st>>>(cv, layer0, n_scope, g, Hq, (const float*)q, (float*)out,
                                                                scale, retention_bias, (int)t_now);
        if (pm) pm->mark(PH_ATTN_MAIN, 1, st);
        count_launch();
    }
}

}  // namespace tkv
