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

constexpr int GH_WARPS = 4;    // warps per CTA of the hidden-layer kernel; they split the input dimension
constexpr int GH_JW = 4;       // hidden units per CTA
constexpr int GH_RW = 8;       // rows per CTA
constexpr int GH_UNROLL = 4;   // 128-float slices of the input dimension in flight per warp

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sums 32 per-lane values over the warp with 31 shuffles: afterwards lane i holds the warp total of v[i].
__device__ __forceinline__ float warp_transpose_sum32(float (&v)[32], int lane) {
#pragma unroll
    for (int s = 16, n = 32; s >= 1; s >>= 1, n >>= 1) {
        const bool upper = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
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

// u[lb][r][j] = SiLU(x[lb][r][:] . W1[layer][j][:] + b1[layer][j]) for GH_RW rows and GH_JW hidden units per CTA.
// grid = (row tiles, hidden-unit groups, layers): CTAs that share a slice of W1 are neighbours in launch order.
__global__ void __launch_bounds__(GH_WARPS * 32, 4)
gate_hidden_kernel(const float* __restrict__ x, const float* __restrict__ W1, const float* __restrict__ b1,
                   float* __restrict__ u, int layer0, int R, int D, int dg) {
    __shared__ float red[GH_WARPS][GH_RW * GH_JW];
    const int lb = blockIdx.z;
    const int layer = layer0 + lb;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j0 = blockIdx.y * GH_JW;
    const int r0 = blockIdx.x * GH_RW;
    const int nj = min(GH_JW, dg - j0);
    const int nr = min(GH_RW, R - r0);
    const float* Wb = W1 + ((size_t)layer * dg + j0) * D;
    const float* xb = x + ((size_t)lb * R + r0) * D;

    float acc[GH_RW * GH_JW];                     // [row][hidden unit]
#pragma unroll
    for (int a = 0; a < GH_RW * GH_JW; ++a) acc[a] = 0.f;

    const int nslice = (D + 127) / 128;
    for (int c0 = warp; c0 < nslice; c0 += GH_WARPS * GH_UNROLL) {
        float4 w[GH_UNROLL][GH_JW];
#pragma unroll
        for (int un = 0; un < GH_UNROLL; ++un) {
            const int d0 = (c0 + un * GH_WARPS) * 128 + lane * 4;
#pragma unroll
            for (int jj = 0; jj < GH_JW; ++jj)
                w[un][jj] = (d0 < D && jj < nj) ? ld_stream(Wb + (size_t)jj * D + d0) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int un = 0; un < GH_UNROLL; ++un) {
            const int d0 = (c0 + un * GH_WARPS) * 128 + lane * 4;
            if (d0 < D) {
#pragma unroll
                for (int rh = 0; rh < GH_RW; rh += 4) {          // rows in batches of four: loads first, then the FMAs
                    float4 xv[4];
#pragma unroll
                    for (int r4 = 0; r4 < 4; ++r4)
                        xv[r4] = (rh + r4 < nr) ? __ldg(reinterpret_cast<const float4*>(xb + (size_t)(rh + r4) * D + d0))
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int r4 = 0; r4 < 4; ++r4)
#pragma unroll
                        for (int jj = 0; jj < GH_JW; ++jj) {
                            float a = acc[(rh + r4) * GH_JW + jj];
                            a = fmaf(xv[r4].x, w[un][jj].x, a);
                            a = fmaf(xv[r4].y, w[un][jj].y, a);
                            a = fmaf(xv[r4].z, w[un][jj].z, a);
                            a = fmaf(xv[r4].w, w[un][jj].w, a);
                            acc[(rh + r4) * GH_JW + jj] = a;
                        }
                }
            }
        }
    }
    static_assert(GH_RW * GH_JW == 32, "the warp reduction below sums exactly 32 values");
    red[warp][lane] = warp_transpose_sum32(acc, lane);   // lane = row * GH_JW + hidden unit
    __syncthreads();
    if (threadIdx.x < GH_RW * GH_JW) {
        const int rr = threadIdx.x / GH_JW, jj = threadIdx.x % GH_JW;
        if (rr < nr && jj < nj) {
            float z = 0.f;
#pragma unroll
            for (int w8 = 0; w8 < GH_WARPS; ++w8) z += red[w8][threadIdx.x];   // fixed order: deterministic
            z += __ldg(b1 + (size_t)layer * dg + j0 + jj);
            u[((size_t)lb * R + r0 + rr) * dg + j0 + jj] = z / (1.0f + expf(-z));
        }
    }
}

constexpr int GO_RT = 8;  // rows per CTA of the output kernel

// s[lb][r][h] = v[layer][h] . u[lb][r] + s0[layer][h]; then beta / lambda / c.   grid = (row tiles, layers).
__global__ void __launch_bounds__(256)
gate_out_kernel(const float* __restrict__ u, const float* __restrict__ v, const float* __restrict__ s0, int layer0, int R,
                int dg, int H, int horizon, float* __restrict__ beta, float* __restrict__ lam, float* __restrict__ cterm) {
    extern __shared__ float su[];           // [GO_RT][dg] rows of u
    const int lb = blockIdx.y;
    const int layer = layer0 + lb;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = blockIdx.x * GO_RT;
    const int nr = min(GO_RT, R - r0);
    for (int i = threadIdx.x * 4; i < nr * dg; i += blockDim.x * 4)
        *reinterpret_cast<float4*>(su + i) = *reinterpret_cast<const float4*>(u + ((size_t)lb * R + r0) * dg + i);
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

void launch_gate(const GateParams& gp, const float* x, float* u_scratch, int layer0, int nlayers, int rows_per_layer,
                 float* beta, float* lam, float* c, cudaStream_t st) {
    dim3 g1((rows_per_layer + GH_RW - 1) / GH_RW, (gp.dg + GH_JW - 1) / GH_JW, nlayers);
    gate_hidden_kernel<<<g1, GH_WARPS * 32, 0, st>>>(x, gp.W1, gp.b1, u_scratch, layer0, rows_per_layer, gp.D, gp.dg);
    dim3 g2((rows_per_layer + GO_RT - 1) / GO_RT, nlayers);
    const size_t smem = (size_t)GO_RT * gp.dg * sizeof(float);
    gate_out_kernel<<<g2, 256, smem, st>>>(u_scratch, gp.v, gp.s0, layer0, rows_per_layer, gp.dg, gp.H, gp.horizon, beta,
                                           lam, c);
    count_launch(2);
}

}  // namespace tkv
