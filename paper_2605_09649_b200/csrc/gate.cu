// Retention gate (Sec. 4.1, Sec. 5.1): beta = sigmoid(w_g . Proj_{l,h}(x) + b_g) with
// Proj_{l,h}(x) = W2[l,h] SiLU(W1[l] x + b1[l]) + b2[l,h]; (w_g, b_g) shared by all layers and heads.
// Outputs per (row, head): beta, lambda = ln beta, c = ln sum_{k<horizon} beta^k.
//
// Proj's second layer and the shared readout are both linear, so they compose exactly:
//   s = w_g . (W2 u + b2) + b_g = v . u + s0,  v[l,h,:] = W2[l,h]^T w_g,  s0[l,h] = w_g . b2[l,h] + b_g.
// v and s0 are folded once when the weights are set (fp64 accumulation); per token the gate then
// streams W1 once (the bulk of the bytes) and 2 KB of v per (layer, head).
//
// fp32 CUDA-core arithmetic: at decode the op streams the weights once (HBM bound); the 1e-5
// relative output tolerance excludes single-pass bf16/tf32 tensor-core math.
#include "trimkv_internal.cuh"

namespace tkv {

namespace {

constexpr int GH_WARPS = 8;    // warps per CTA of the hidden-layer kernel
constexpr int GH_DC = 512;     // floats of the input dimension per CTA (its x tile lives in shared memory)
constexpr int GH_RW = 8;       // rows per CTA
constexpr int GH_JP = 2;       // hidden units per warp pass
constexpr int GH_JSPLIT = 4;   // CTAs that share the hidden units of one (layer, input chunk)

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sums 16 per-lane values over the warp with 20 shuffles: afterwards lanes 0..15 hold the warp totals of v[0..15].
__device__ __forceinline__ float warp_transpose_sum16(float (&v)[16], int lane) {
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] += __shfl_xor_sync(0xffffffffu, v[i], 16);   // fold the two half-warps
#pragma unroll
    for (int s = 8, n = 16; s >= 1; s >>= 1, n >>= 1) {
        const bool upper = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (i < n / 2) {
                const float send = upper ? v[i] : v[i + n / 2];
                const float keep = upper ? v[i + n / 2] : v[i];
                v[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
            }
        }
    }
    return v[0];
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

// Partial pre-activations: zpart[lb][chunk][r][j] = x[lb][r][chunk] . W1[layer][j][chunk] for GH_RW rows, one
// GH_DC-float chunk of the input dimension and a quarter of the hidden units per CTA.  The x tile is staged in
// shared memory once and W1 is streamed past it, two hidden units per warp pass with eight 16-byte loads in flight
// per lane.  grid = (row tiles * chunks, GH_JSPLIT, layers): CTAs that share a slice of W1 are neighbours in launch
// order (chunked-prefill calls re-read W1 from L2).
__global__ void __launch_bounds__(GH_WARPS * 32, 2)
gate_hidden_kernel(const float* __restrict__ x, const float* __restrict__ W1, float* __restrict__ zpart, int layer0,
                   int R, int D, int dg, int nchunk) {
    __shared__ __align__(16) float xs[GH_RW][GH_DC];
    const int lb = blockIdx.z;
    const int layer = layer0 + lb;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int chunk = blockIdx.x % nchunk;
    const int r0 = (blockIdx.x / nchunk) * GH_RW;
    const int nr = min(GH_RW, R - r0);
    const int dbase = chunk * GH_DC;
    const int jper = (dg + GH_JSPLIT - 1) / GH_JSPLIT;
    const int jbeg = blockIdx.y * jper, jend = min(dg, jbeg + jper);

    for (int i = threadIdx.x; i < GH_RW * (GH_DC / 4); i += blockDim.x) {
        const int rr = i / (GH_DC / 4), dd = (i % (GH_DC / 4)) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (rr < nr && dbase + dd < D) v = __ldg(reinterpret_cast<const float4*>(x + ((size_t)lb * R + r0 + rr) * D + dbase + dd));
        *reinterpret_cast<float4*>(&xs[rr][dd]) = v;
    }
    __syncthreads();

    const float* Wl = W1 + (size_t)layer * dg * D + dbase;
    float* zp = zpart + (((size_t)lb * nchunk + chunk) * R + r0) * dg;
    for (int j0 = jbeg + warp * GH_JP; j0 < jend; j0 += GH_WARPS * GH_JP) {
        float4 w[GH_JP][GH_DC / 128];
#pragma unroll
        for (int jj = 0; jj < GH_JP; ++jj)
#pragma unroll
            for (int sl = 0; sl < GH_DC / 128; ++sl) {
                const int dd = sl * 128 + lane * 4;
                w[jj][sl] = (j0 + jj < jend && dbase + dd < D) ? ld_stream(Wl + (size_t)(j0 + jj) * D + dd)
                                                               : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        float acc[GH_JP * GH_RW];
#pragma unroll
        for (int a = 0; a < GH_JP * GH_RW; ++a) acc[a] = 0.f;
#pragma unroll
        for (int sl = 0; sl < GH_DC / 128; ++sl) {
#pragma unroll
            for (int rr = 0; rr < GH_RW; ++rr) {
                const float4 xv = *reinterpret_cast<const float4*>(&xs[rr][sl * 128 + lane * 4]);
#pragma unroll
                for (int jj = 0; jj < GH_JP; ++jj) {
                    float a = acc[jj * GH_RW + rr];
                    a = fmaf(xv.x, w[jj][sl].x, a);
                    a = fmaf(xv.y, w[jj][sl].y, a);
                    a = fmaf(xv.z, w[jj][sl].z, a);
                    a = fmaf(xv.w, w[jj][sl].w, a);
                    acc[jj * GH_RW + rr] = a;
                }
            }
        }
        static_assert(GH_JP * GH_RW == 16, "the warp reduction below sums exactly 16 values");
        const float tot = warp_transpose_sum16(acc, lane);      // lane = jj * GH_RW + rr
        if (lane < 16) {
            const int jj = lane / GH_RW, rr = lane % GH_RW;
            if (rr < nr && j0 + jj < jend) zp[(size_t)rr * dg + j0 + jj] = tot;
        }
    }
}

constexpr int GO_RT = 8;  // rows per CTA of the output kernel

// s[lb][r][h] = v[layer][h] . u[lb][r] + s0[layer][h]; then beta / lambda / c.   grid = (row tiles, layers).
__global__ void __launch_bounds__(256)
gate_out_kernel(const float* __restrict__ zpart, const float* __restrict__ b1, const float* __restrict__ v,
                const float* __restrict__ s0, int layer0, int R, int dg, int nchunk, int H, int horizon,
                float* __restrict__ beta, float* __restrict__ lam, float* __restrict__ cterm) {
    extern __shared__ float su[];           // [GO_RT][dg] rows of u = SiLU(sum of the chunk partials + b1)
    const int lb = blockIdx.y;
    const int layer = layer0 + lb;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = blockIdx.x * GO_RT;
    const int nr = min(GO_RT, R - r0);
    for (int i = threadIdx.x * 4; i < nr * dg; i += blockDim.x * 4) {
        float4 z = __ldg(reinterpret_cast<const float4*>(b1 + (size_t)layer * dg + i % dg));
        for (int ch = 0; ch < nchunk; ++ch) {           // fixed order: deterministic
            const float4 p = *reinterpret_cast<const float4*>(zpart + (((size_t)lb * nchunk + ch) * R + r0) * dg + i);
            z.x += p.x; z.y += p.y; z.z += p.z; z.w += p.w;
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
                if (cterm) cterm[o] = horizon_term_f32(lm, horizon);
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

void launch_gate_out(const GateParams& gp, const float* z_scratch, int nchunk, int layer0, int nlayers, int rows_per_layer,
                     float* beta, float* lam, float* c, cudaStream_t st) {
    dim3 g2((rows_per_layer + GO_RT - 1) / GO_RT, nlayers);
    const size_t smem = (size_t)GO_RT * gp.dg * sizeof(float);
    gate_out_kernel<<<g2, 256, smem, st>>>(z_scratch, gp.b1, gp.v, gp.s0, layer0, rows_per_layer, gp.dg, nchunk, gp.H,
                                           gp.horizon, beta, lam, c);
    count_launch();
}

void launch_gate(const GateParams& gp, const float* x, float* z_scratch, int layer0, int nlayers, int rows_per_layer,
                 float* beta, float* lam, float* c, cudaStream_t st) {
    const int nchunk = gate_chunks(gp.D);
    dim3 g1(((rows_per_layer + GH_RW - 1) / GH_RW) * nchunk, GH_JSPLIT, nlayers);
    gate_hidden_kernel<<<g1, GH_WARPS * 32, 0, st>>>(x, gp.W1, z_scratch, layer0, rows_per_layer, gp.D, gp.dg, nchunk);
    count_launch();
    launch_gate_out(gp, z_scratch, nchunk, layer0, nlayers, rows_per_layer, beta, lam, c, st);
}

}  // namespace tkv
