// Causal attention of a chunk that has just been appended, over the ragged per-(layer, head) pools (Sec. 2.1 attention
// restricted to the retained set, Eq. (1) with r in {0,1}): token j of the chunk attends to every entry kept from before
// the chunk and to the chunk's own tokens up to itself.  The chunk's entries sit at the tail of each pool in token order,
// so the causal mask is an index test: entry e is visible to chunk token j iff e < n_old + j + 1.
//
// bf16, d = 128: one CTA per (pool, block of chunk tokens).  Thread 0 streams the pool's 32-entry K/V tiles into a 3-stage
// shared-memory ring with bulk asynchronous copies (one full and one empty mbarrier per stage); the four warps share every
// tile.  A warp owns 16 (token, query head) columns: S^T = K Q^T and O^T += V^T P^T with mma.sync m16n8k16, online softmax
// in registers, as in the decode kernel, with the columns now spread over tokens.  Every wait is bounded.
// Any other shape / fp32: one warp per (pool, token, query head).
#include "async_copy.cuh"
#include "mma_sync.cuh"
#include "trimkv_internal.cuh"

namespace tkv {

namespace {

constexpr int PT = 32;                          // entries per tile
constexpr int P_STAGES = 3;
constexpr int P_ROWB = 256;                     // bytes per K or V row (d = 128, bf16)
constexpr int P_STAGE_BYTES = 2 * PT * P_ROWB;  // K tile + V tile
constexpr int P_SMEM = P_STAGES * P_STAGE_BYTES + 128;
constexpr int P_WARPS = 4;
constexpr int P_COLS = 16;                      // (token, head) columns per warp
// grid = (token blocks, B * H pools of `layer`); q, out: [B, n_new, Hq, 128] bf16.
__global__ void __launch_bounds__(P_WARPS * 32, 2)
prefill_attn_mma_kernel(CacheView cv, int layer, int n_new, int g, int Hq, const __nv_bfloat16* __restrict__ q,
                        __nv_bfloat16* __restrict__ out, float scale_log2) {
    extern __shared__ __align__(128) unsigned char psm[];
    uint64_t* full = reinterpret_cast<uint64_t*>(psm + P_STAGES * P_STAGE_BYTES);
    uint64_t* empty = full + P_STAGES;
    volatile int* s_fail = reinterpret_cast<volatile int*>(empty + P_STAGES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tw = P_COLS / g;                               // chunk tokens per warp
    const int tc = P_WARPS * tw;                             // chunk tokens per CTA
    const int i0 = blockIdx.x * tc;
    if (i0 >= n_new) return;
    const int h = blockIdx.y % cv.H, b = blockIdx.y / cv.H;
    const long long pool = ((long long)b * cv.L + layer) * cv.H + h;
    const int len = cv.len[pool];
    const int n_old = len - n_new;                           // entries kept from before the chunk
    if (n_old < 0) return;                                   // the append of this chunk failed (its error is latched)
    const int limit = n_old + min(n_new, i0 + tc);           // entries any token of this block may see
    const int ntile = (limit + PT - 1) / PT;
    const int32_t* bt = cv.block_table + pool * cv.maxpp;

    for (int i = threadIdx.x * 16; i < P_STAGES * P_STAGE_BYTES; i += blockDim.x * 16)
        *reinterpret_cast<uint4*>(psm + i) = make_uint4(0u, 0u, 0u, 0u);      // masked rows must hold finite values
    if (threadIdx.x == 0) {
        for (int s = 0; s < P_STAGES; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, P_WARPS); }
        *s_fail = 0;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();

    // ---- producer state (warp 0): lane i holds the page of tiles 2i, 2i + 1 of the current run of 64 tiles
    int page_id = 0;
    auto issue = [&](int tt) {                               // warp 0, all lanes
        if ((tt & 63) == 0) {
            const int left = (ntile - tt + 1) / 2;
            page_id = (lane < left) ? bt[tt / 2 + lane] : 0;
        }
        const int page = __shfl_sync(0xffffffffu, page_id, (tt >> 1) & 31);
        if (lane == 0) {
            const int s = tt % P_STAGES;
            unsigned char* dst = psm + (size_t)s * P_STAGE_BYTES;
            const char* ksrc = cv.kv + kv_row_offset(cv, b, page, 0, (tt & 1) * PT);
            const char* vsrc = cv.kv + kv_row_offset(cv, b, page, 1, (tt & 1) * PT);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_expect_tx(full + s, P_STAGE_BYTES);
            bulk_g2s(dst, ksrc, PT * P_ROWB, full + s);
            bulk_g2s(dst + PT * P_ROWB, vsrc, PT * P_ROWB, full + s);
        }
    };
    if (warp == 0) {
        for (int tt = 0; tt < min(P_STAGES - 1, ntile); ++tt) issue(tt);
    }

    // ---- this warp's columns: col = token_local * g + head
    const int wtok0 = i0 + warp * tw;
    uint32_t bq[2][8][2];
    int lim[2][2];                                            // entries visible to the two columns this thread owns per n-tile
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        const int col = nt * 8 + (lane >> 2);
        const int tl = col / g, head = col % g;
        const bool okc = tl < tw && wtok0 + tl < n_new;
        const __nv_bfloat16* qp = q + (((size_t)b * n_new + (okc ? wtok0 + tl : 0)) * Hq + (size_t)h * g + head) * 128;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t v0 = 0u, v1 = 0u;
            if (okc) {
                const __nv_bfloat16* p = qp + ks * 16 + 2 * (lane & 3);
                v0 = *reinterpret_cast<const uint32_t*>(p);
                v1 = *reinterpret_cast<const uint32_t*>(p + 8);
            }
            bq[nt][ks][0] = v0;
            bq[nt][ks][1] = v1;
        }
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
            const int c2 = nt * 8 + 2 * (lane & 3) + cc;
            const int t2 = c2 / g;
            lim[nt][cc] = (t2 < tw && wtok0 + t2 < n_new) ? n_old + wtok0 + t2 + 1 : 1;   // idle columns see entry 0 only
        }
    }
    float o[2][8][4];
    float m_run[2][2], l_run[2][2];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) { o[nt][dt][0] = o[nt][dt][1] = o[nt][dt][2] = o[nt][dt][3] = 0.f; }
        m_run[nt][0] = m_run[nt][1] = -INFINITY;
        l_run[nt][0] = l_run[nt][1] = 0.f;
    }

    bool failed = false;
    for (int tt = 0; tt < ntile; ++tt) {
        if (warp == 0 && tt + P_STAGES - 1 < ntile) {        // refill the stage that tile tt - 1 used
            const int nx = tt + P_STAGES - 1;
            bool ok = true;
            if (nx >= P_STAGES) {
                int got = 1;
                if (lane == 0) got = mbar_wait_bounded(empty + nx % P_STAGES, ((nx / P_STAGES) - 1) & 1) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, got, 0) != 0;
            }
            if (!ok) { failed = true; break; }
            issue(nx);
        }
        const int s = tt % P_STAGES;
        {
            int got = 1;
            if (lane == 0) got = mbar_wait_bounded(full + s, (tt / P_STAGES) & 1) ? 1 : 0;
            if (__shfl_sync(0xffffffffu, got, 0) == 0) { failed = true; break; }
        }
        const uint32_t kbase = smem_u32(psm + (size_t)s * P_STAGE_BYTES);
        const uint32_t vbase = kbase + PT * P_ROWB;
        // ---- S^T[entry][column] = K Q^T
        float sacc[2][2][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) sacc[mt][nt][0] = sacc[mt][nt][1] = sacc[mt][nt][2] = sacc[mt][nt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                const int row = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                const int chunk = (2 * ks + (lane >> 4)) ^ (row & 7);
                uint32_t a[4];
                ldsm_x4(a, kbase + row * P_ROWB + chunk * 16);
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) mma_bf16(sacc[mt][nt], a, bq[nt][ks][0], bq[nt][ks][1]);
            }
        }
        // ---- causal mask by entry index, online softmax per column
        uint32_t pb[2][2][2];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                const int e0 = tt * PT + mt * 16 + (lane >> 2);
                float* sc = sacc[mt][nt];
                sc[0] = (e0 < lim[nt][0]) ? sc[0] * scale_log2 : -INFINITY;
                sc[1] = (e0 < lim[nt][1]) ? sc[1] * scale_log2 : -INFINITY;
                sc[2] = (e0 + 8 < lim[nt][0]) ? sc[2] * scale_log2 : -INFINITY;
                sc[3] = (e0 + 8 < lim[nt][1]) ? sc[3] * scale_log2 : -INFINITY;
                mx0 = fmaxf(mx0, fmaxf(sc[0], sc[2]));
                mx1 = fmaxf(mx1, fmaxf(sc[1], sc[3]));
            }
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
            }
            const float mn0 = fmaxf(m_run[nt][0], mx0), mn1 = fmaxf(m_run[nt][1], mx1);   // finite from tile 0 on
            const float f0 = exp2f(m_run[nt][0] - mn0), f1 = exp2f(m_run[nt][1] - mn1);
            m_run[nt][0] = mn0;
            m_run[nt][1] = mn1;
            float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                float* sc = sacc[mt][nt];
                const __nv_bfloat162 plo = __floats2bfloat162_rn(exp2f(sc[0] - mn0), exp2f(sc[1] - mn1));
                const __nv_bfloat162 phi = __floats2bfloat162_rn(exp2f(sc[2] - mn0), exp2f(sc[3] - mn1));
                ls0 += __low2float(plo) + __low2float(phi);
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
        // ---- O^T[d][column] += V^T P^T
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                const int row = mt * 16 + (lane & 7) + (lane >> 4) * 8;
                const int chunk = (2 * dt + ((lane >> 3) & 1)) ^ (row & 7);
                uint32_t a[4];
                ldsm_x4_trans(a, vbase + row * P_ROWB + chunk * 16);
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) mma_bf16(o[nt][dt], a, pb[mt][nt][0], pb[mt][nt][1]);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty + s);               // this warp is done with the stage
    }
    if (failed) {
        if (lane == 0) { *s_fail = 1; latch_error(cv.err, TRIMKV_E_TIMEOUT); }
        return;
    }
    // ---- normalise and store: column -> (token, head)
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        float l0 = l_run[nt][0], l1 = l_run[nt][1];
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            l0 += __shfl_xor_sync(0xffffffffu, l0, off);
            l1 += __shfl_xor_sync(0xffffffffu, l1, off);
        }
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
            const int col = nt * 8 + 2 * (lane & 3) + cc;
            const int tl = col / g, head = col % g;
            if (tl < tw && wtok0 + tl < n_new) {
                const float r = (cc ? l1 : l0) > 0.f ? 1.0f / (cc ? l1 : l0) : 0.f;
                __nv_bfloat16* op = out + (((size_t)b * n_new + wtok0 + tl) * Hq + (size_t)h * g + head) * 128;
#pragma unroll
                for (int dt = 0; dt < 8; ++dt) {
                    const int dr = dt * 16 + (lane >> 2);
                    op[dr] = __float2bfloat16_rn(o[nt][dt][cc] * r);
                    op[dr + 8] = __float2bfloat16_rn(o[nt][dt][2 + cc] * r);
                }
            }
        }
    }
}

// Plain form for any head size and fp32: one warp per (sequence, chunk token, query head); lanes split d.
template <typename T, int MAXD>
__global__ void __launch_bounds__(128)
prefill_attn_plain_kernel(CacheView cv, int layer, int n_new, int g, int Hq, const T* __restrict__ q, T* __restrict__ out,
                          float scale) {
    const long long wid = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (wid >= (long long)cv.B * n_new * Hq) return;
    const int hq = (int)(wid % Hq);
    const int j = (int)((wid / Hq) % n_new);
    const int b = (int)(wid / ((long long)Hq * n_new));
    const int h = hq / g;
    const long long pool = ((long long)b * cv.L + layer) * cv.H + h;
    const int n_old = cv.len[pool] - n_new;
    const int d = cv.d;
    constexpr int PER = MAXD / 32;
    const int epc = 16 / (int)sizeof(T);
    T* op = out + (((size_t)b * n_new + j) * Hq + hq) * d;
    if (n_old < 0) return;
    const int n = n_old + j + 1;                             // entries visible to this token
    float qr[PER], acc[PER];
    const T* qp = q + (((size_t)b * n_new + j) * Hq + hq) * d;
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
        for (int o2 = 16; o2 > 0; o2 >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o2);
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
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int dd = lane + 32 * i;
        if (dd < d) op[dd] = from_f32<T>(acc[i] / l);
    }
}

}  // namespace

void launch_prefill_attention(const CacheView& cv, int layer, int n_new, int Hq, int is_bf16, const PrefillTcState* tc,
                              const void* q, void* out, cudaStream_t st) {
    if (tc && prefill_tc_wanted(cv, n_new, Hq)) {
        launch_prefill_attention_tc(tc, cv, layer, n_new, Hq, q, out, st);
        return;
    }
    const int g = Hq / cv.H;
    const float scale = 1.0f / sqrtf((float)cv.d);
    if (is_bf16 && cv.d == 128 && g <= P_COLS) {
        if (first_use_on_device(1))
            cudaFuncSetAttribute(prefill_attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM);
        const int tc = P_WARPS * (P_COLS / g);
        dim3 grid((n_new + tc - 1) / tc, cv.B * cv.H);
        prefill_attn_mma_kernel<<<grid, P_WARPS * 32, P_SMEM, st>>>(cv, layer, n_new, g, Hq, (const __nv_bfloat16*)q,
                                                                     (__nv_bfloat16*)out, scale * 1.4426950408889634f);
    } else {
        const long long warps = (long long)cv.B * n_new * Hq;
        const unsigned grid = (unsigned)((warps + 3) / 4);
        if (is_bf16)
            prefill_attn_plain_kernel<__nv_bfloat16, 256><<<grid, 128, 0, st>>>(cv, layer, n_new, g, Hq, (const __nv_bfloat16*)q,
                                                                                 (__nv_bfloat16*)out, scale);
        else
            prefill_attn_plain_kernel<float, 256><<<grid, 128, 0, st>>>(cv, layer, n_new, g, Hq, (const float*)q, (float*)out,
                                                                        scale);
    }
    count_launch();
}

}  // namespace tkv
