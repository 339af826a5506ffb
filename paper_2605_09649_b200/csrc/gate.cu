// Retention gate (Sec. 4.1, Sec. 5.1): beta = sigmoid(w_g . Proj_{l,h}(x) + b_g) with
// Proj_{l,h}(x) = W2[l,h] SiLU(W1[l] x + b1[l]) + b2[l,h]; (w_g, b_g) shared by all layers and heads.
// Outputs per (row, head): beta, lambda = ln beta, c = ln sum_{k<horizon} beta^k.
//
// Proj's second layer and the shared readout are both linear, so they compose exactly:
//   s = w_g . (W2 u + b2) + b_g = v . u + s0,  v[l,h,:] = W2[l,h]^T w_g,  s0[l,h] = w_g . b2[l,h] + b_g.
// v and s0 are folded once when the weights are set (fp64 accumulation); per token the gate then
// streams W1 once (the bulk of the bytes; stored transposed, input dimension major) and 2 KB of v per (layer, head).
//
// fp32 CUDA-core arithmetic: at decode the op streams the weights once (HBM bound); the 1e-5
// relative output tolerance excludes single-pass bf16/tf32 tensor-core math.
#include "trimkv_internal.cuh"

namespace tkv {

namespace {

constexpr int GH_THREADS = 128;  // threads per CTA of the hidden-layer kernel; a thread owns 4 consecutive hidden units
constexpr int GH_DC = 128;       // input dimensions per CTA (its x tile lives in shared memory)
constexpr int GH_U = 8;          // input dimensions (16-byte weight loads per lane) in flight

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float4 ld_stream(const float* p) {   // read-once data: do not keep it in L1
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p));
    return v;
}

// v[l][h][j] = sum_k w_g[k] W2[l][h][k][j];  s0[l][h] = sum_k w_g[k] b2[l][h][k] + b_g.   One CTA per (layer, head).
__global__ void __launch_bounds__(256)
gate_fold_kernel(const float* __restrict__ W2, const float* __restrict__ b2, const float* __restrict__ w_g, float b_g,
                 int layer0, int H, int dg, int de, float* __restrict__ v, float* __restrict__ s0) {
    const int h = blockIdx.x, layer = layer0 + blockIdx.y;
    const float* W2h = W2 + ((size_t)layer * H + h) * de * dg;
    for (int j = threadIdx.x; j < dg; j += blockDim.x) {
        double acc = 0.0;
        for (int k = 0; k < de; ++k) acc += (double)w_g[k] * (double)W2h[(size_t)k * dg + j];
        v[((size_t)layer * H + h) * dg + j] = (float)acc;
    }
    if (threadIdx.x == 0) {
        double acc = (double)b_g;
        for (int k = 0; k < de; ++k) acc += (double)w_g[k] * (double)b2[((size_t)layer * H + h) * de + k];
        s0[(size_t)layer * H + h] = (float)acc;
    }
}

// Two fp32 multiply-adds per instruction (each lane rounded as a scalar fmaf would).
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}

// JT consecutive floats of read-once data.
template <int JT>
__device__ __forceinline__ void ld_stream_n(const float* p, float (&dst)[JT]) {
    if constexpr (JT == 4) {
        const float4 v = ld_stream(p);
        dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
    } else if constexpr (JT == 2) {
        asm volatile("ld.global.nc.L1::no_allocate.v2.f32 {%0,%1}, [%2];" : "=f"(dst[0]), "=f"(dst[1]) : "l"(p));
    } else {
        asm volatile("ld.global.nc.L1::no_allocate.f32 %0, [%1];" : "=f"(dst[0]) : "l"(p));
    }
}

// Partial pre-activations: zpart[lb][chunk][r][j] = sum over the chunk's input dimensions d of x[lb][r][d] W1[layer][j][d],
// for RW rows and one GH_DC-wide chunk of the input dimension per CTA.  W1 is kept transposed (W1T[layer][d][j]): a
// thread owns JT consecutive hidden units, so a warp's weight load is contiguous, the x values of a dimension are
// broadcast reads of shared memory for the whole warp, and every thread finishes its own JT * RW = 32 sums (no
// shuffles; the multiply-adds are packed fp32x2 over pairs of rows).  RW = 8 with JT = 4 serves up to 8 rows; larger
// batches use RW = 16, JT = 2, which halves the number of times the weights are streamed (RW = 32, JT = 1 was slower: its
// 4-byte weight loads quadruple the load instructions; measured at 32 rows: 0.254 against 0.164 ms).  U dimensions are in
// flight per thread, and the next U are requested before the current ones are used.
// grid = (row tiles * chunks, ceil(dg / (JT * GH_THREADS)), layers).
template <int RW, int JT>
__global__ void __launch_bounds__(GH_THREADS, 4)
gate_hidden_kernel(const float* __restrict__ x, const float* __restrict__ W1T, float* __restrict__ zpart, int layer0,
                   int R, int D, int dg, int nchunk) {
    constexpr int U = JT == 4 ? GH_U : 2 * GH_U;
    __shared__ __align__(16) float xs[GH_DC][RW];
    const int lb = blockIdx.z;
    const int layer = layer0 + lb;
    const int chunk = blockIdx.x % nchunk;
    const int r0 = (blockIdx.x / nchunk) * RW;
    const int nr = min(RW, R - r0);
    const int dbase = chunk * GH_DC;
    const int dn = min(GH_DC, D - dbase);
    for (int i = threadIdx.x; i < GH_DC * RW; i += blockDim.x) {
        const int rr = i / GH_DC, dd = i % GH_DC;
        xs[dd][rr] = (rr < nr && dd < dn) ? __ldg(x + ((size_t)lb * R + r0 + rr) * D + dbase + dd) : 0.f;
    }
    __syncthreads();
    const int j = (blockIdx.y * GH_THREADS + threadIdx.x) * JT;
    if (j >= dg) return;
    const float* Wp = W1T + ((size_t)layer * D + dbase) * dg + j;
    unsigned long long acc[JT][RW / 2];                                  // pairs of rows: packed fp32x2 multiply-adds
#pragma unroll
    for (int q = 0; q < JT; ++q)
#pragma unroll
        for (int rr = 0; rr < RW / 2; ++rr) acc[q][rr] = 0ull;
    float w[U][JT], wn[U][JT];
    auto fetch = [&](float (&dst)[U][JT], int d0) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (d0 + u < dn) {
                ld_stream_n<JT>(Wp + (size_t)(d0 + u) * dg, dst[u]);
            } else {
#pragma unroll
                for (int q = 0; q < JT; ++q) dst[u][q] = 0.f;
            }
        }
    };
    fetch(w, 0);
    for (int d0 = 0; d0 < dn; d0 += U) {
        fetch(wn, d0 + U);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (d0 + u < GH_DC) {                                        // (rows of xs beyond dn hold zeros)
                unsigned long long w2[JT];
#pragma unroll
                for (int q = 0; q < JT; ++q) w2[q] = pack_f32x2(w[u][q], w[u][q]);
#pragma unroll
                for (int r4 = 0; r4 < RW / 4; ++r4) {
                    const ulonglong2 xv = *reinterpret_cast<const ulonglong2*>(&xs[d0 + u][4 * r4]);   // rows 4 r4 .. 4 r4 + 3
#pragma unroll
                    for (int q = 0; q < JT; ++q) {
                        acc[q][2 * r4] = fma_f32x2(xv.x, w2[q], acc[q][2 * r4]);
                        acc[q][2 * r4 + 1] = fma_f32x2(xv.y, w2[q], acc[q][2 * r4 + 1]);
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int q = 0; q < JT; ++q) w[u][q] = wn[u][q];
    }
    float* zp = zpart + (((size_t)lb * nchunk + chunk) * R + r0) * dg + j;
#pragma unroll
    for (int rp = 0; rp < RW / 2; ++rp) {
#pragma unroll
        for (int q = 0; q < JT; ++q) {
            float lo, hi;
            asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(acc[q][rp]));
            if (2 * rp < nr) zp[(size_t)(2 * rp) * dg + q] = lo;
            if (2 * rp + 1 < nr) zp[(size_t)(2 * rp + 1) * dg + q] = hi;
        }
    }
}

// W1T[d][j] = W1[j][d] for one layer (32 x 32 tiles through shared memory).  grid = (ceil(D / 32), ceil(dg / 32)).
__global__ void __launch_bounds__(256)
gate_transpose_kernel(const float* __restrict__ W1, float* __restrict__ W1T, int dg, int D) {
    __shared__ float tile[32][33];
    const int d0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int k = ty; k < 32; k += 8)
        if (j0 + k < dg && d0 + tx < D) tile[k][tx] = W1[(size_t)(j0 + k) * D + d0 + tx];
    __syncthreads();
    for (int k = ty; k < 32; k += 8)
        if (d0 + k < D && j0 + tx < dg) W1T[(size_t)(d0 + k) * dg + j0 + tx] = tile[tx][k];
}

constexpr int GO_RT = 2;  // rows per CTA of the output kernel (few: at decode the kernel is a chain of dependent loads per thread)

// s[lb][r][h] = v[layer][h] . u[lb][r] + s0[layer][h]; then beta / lambda / c.   grid = (row tiles, layers).
// to_cache (a decode step: row r is sequence r's new token, whose K/V half of the append has run): the retention terms
// also go straight to the token's slot, the newest entry of pool (r, layer, h).
__global__ void __launch_bounds__(256)
gate_out_kernel(const float* __restrict__ zpart, const float* __restrict__ b1, const float* __restrict__ v,
                const float* __restrict__ s0, int layer0, int R, int dg, int nchunk, int H, int horizon,
                float* __restrict__ beta, float* __restrict__ lam, float* __restrict__ cterm, int to_cache, CacheView cv) {
    extern __shared__ float su[];           // [GO_RT][dg] rows of u = SiLU(sum of the chunk partials + b1)
    const int lb = blockIdx.y;
    const int layer = layer0 + lb;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = blockIdx.x * GO_RT;
    const int nr = min(GO_RT, R - r0);
    for (int i = threadIdx.x * 4; i < nr * dg; i += blockDim.x * 4) {
        float4 z = __ldg(reinterpret_cast<const float4*>(b1 + (size_t)layer * dg + i % dg));
        // the chunk partials are added in a fixed order (deterministic), their loads issued eight at a time
        for (int ch0 = 0; ch0 < nchunk; ch0 += 8) {
            float4 p[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
                p[q] = (ch0 + q < nchunk)
                           ? __ldcg(reinterpret_cast<const float4*>(zpart + (((size_t)lb * nchunk + ch0 + q) * R + r0) * dg + i))
                           : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int q = 0; q < 8; ++q) { z.x += p[q].x; z.y += p[q].y; z.z += p[q].z; z.w += p[q].w; }
        }
        z.x = z.x / (1.0f + expf(-z.x)); z.y = z.y / (1.0f + expf(-z.y));
        z.z = z.z / (1.0f + expf(-z.z)); z.w = z.w / (1.0f + expf(-z.w));
        *reinterpret_cast<float4*>(su + i) = z;
    }
    __syncthreads();
    for (int h = warp; h < H; h += 8) {
        const float* vh = v + ((size_t)layer * H + h) * dg;
        float acc[GO_RT];
#pragma unroll
        for (int rr = 0; rr < GO_RT; ++rr) acc[rr] = 0.f;
        for (int j = lane * 4; j < dg; j += 128) {
            const float4 w = __ldg(reinterpret_cast<const float4*>(vh + j));
#pragma unroll
            for (int rr = 0; rr < GO_RT; ++rr) {
                if (rr < nr) {
                    const float4 uv = *reinterpret_cast<const float4*>(su + rr * dg + j);
                    acc[rr] = fmaf(uv.x, w.x, acc[rr]);
                    acc[rr] = fmaf(uv.y, w.y, acc[rr]);
                    acc[rr] = fmaf(uv.z, w.z, acc[rr]);
                    acc[rr] = fmaf(uv.w, w.w, acc[rr]);
                }
            }
        }
        const float base = __ldg(s0 + (size_t)layer * H + h);
#pragma unroll
        for (int rr = 0; rr < GO_RT; ++rr) {
            const float dot = warp_sum(acc[rr]);
            if (lane == 0 && rr < nr) {
                const float s = dot + base;
                // beta = sigmoid(s); lambda = ln sigmoid(s) = -softplus(-s), evaluated without cancellation
                const float e = expf(-fabsf(s));
                const float l1p = log1pf(e);
                const float bt = (s >= 0.f) ? 1.0f / (1.0f + e) : e / (1.0f + e);
                const float lm = (s >= 0.f) ? -l1p : (s - l1p);
                const size_t o = ((size_t)lb * R + r0 + rr) * H + h;
                if (beta) beta[o] = bt;
                if (lam) lam[o] = lm;
                const float ct = horizon_term_f32(lm, horizon);
                if (cterm) cterm[o] = ct;
                if (to_cache) {
                    const int b = r0 + rr;
                    const long long pool = ((long long)b * cv.L + layer) * cv.H + h;
                    const int idx = cv.len[pool] - 1;
                    if (!cv.append_failed[pool] && idx >= 0) {
                        const int page = cv.block_table[pool * cv.maxpp + idx / PAGE];
                        const size_t slot = ((size_t)b * cv.P_seq + page) * PAGE + idx % PAGE;
                        if (lm != lm || ct != ct) latch_error(cv.err, TRIMKV_E_NONFINITE);
                        cv.lam[slot] = lm;
                        cv.c[slot] = ct;
                    }
                }
            }
        }
    }
}

}  // namespace

void launch_gate_fold(const GateParams& gp, int layer0, int nlayers, float* v, float* s0, cudaStream_t st) {
    dim3 grid(gp.H, nlayers);
    gate_fold_kernel<<<grid, 256, 0, st>>>(gp.W2, gp.b2, gp.w_g, gp.b_g, layer0, gp.H, gp.dg, gp.de, v, s0);
    count_launch();
}

int gate_chunks(int D) { return (D + GH_DC - 1) / GH_DC; }

void launch_gate_transpose(const float* W1, float* W1T, int dg, int D, cudaStream_t st) {
    dim3 grid((D + 31) / 32, (dg + 31) / 32);
    gate_transpose_kernel<<<grid, 256, 0, st>>>(W1, W1T, dg, D);
    count_launch();
}

void launch_gate_out(const GateParams& gp, const float* z_scratch, int nchunk, int layer0, int nlayers, int rows_per_layer,
                     float* beta, float* lam, float* c, cudaStream_t st, const CacheView* to_cache) {
    dim3 g2((rows_per_layer + GO_RT - 1) / GO_RT, nlayers);
    const size_t smem = (size_t)GO_RT * gp.dg * sizeof(float);
    CacheView none{};
    gate_out_kernel<<<g2, 256, smem, st>>>(z_scratch, gp.b1, gp.v, gp.s0, layer0, rows_per_layer, gp.dg, nchunk, gp.H,
                                           gp.horizon, beta, lam, c, to_cache ? 1 : 0, to_cache ? *to_cache : none);
    count_launch();
}

void launch_gate_hidden(const GateParams& gp, const float* x, float* z_scratch, int layer0, int nlayers, int rows_per_layer,
                        cudaStream_t st) {
    const int nchunk = gate_chunks(gp.D);
    auto run = [&](auto kernel, int rw, int jt) {
        dim3 g1(((rows_per_layer + rw - 1) / rw) * nchunk, (gp.dg + jt * GH_THREADS - 1) / (jt * GH_THREADS), nlayers);
        kernel<<<g1, GH_THREADS, 0, st>>>(x, gp.W1T, z_scratch, layer0, rows_per_layer, gp.D, gp.dg, nchunk);
    };
    if (rows_per_layer <= 8) run(gate_hidden_kernel<8, 4>, 8, 4);
    else run(gate_hidden_kernel<16, 2>, 16, 2);                 // row tiles of 16
    count_launch();
}

void launch_gate(const GateParams& gp, const float* x, float* z_scratch, int layer0, int nlayers, int rows_per_layer,
                 float* beta, float* lam, float* c, cudaStream_t st) {
    launch_gate_hidden(gp, x, z_scratch, layer0, nlayers, rows_per_layer, st);
    launch_gate_out(gp, z_scratch, gate_chunks(gp.D), layer0, nlayers, rows_per_layer, beta, lam, c, st, nullptr);
}

}  // namespace tkv
