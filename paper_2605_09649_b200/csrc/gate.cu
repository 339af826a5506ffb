// Retention gate (Sec. 4.1, Sec. 5.1): beta = sigmoid(w_g . Proj_{l,h}(x) + b_g) with
// Proj_{l,h}(x) = W2[l,h] SiLU(W1[l] x + b1[l]) + b2[l,h]; (w_g, b_g) shared by all layers and heads.
// Outputs per (row, head): beta, lambda = ln beta, c = ln sum_{k<horizon} beta^k.
// fp32 CUDA-core arithmetic: at decode the op streams the weights once (HBM bound); the 1e-5
// relative output tolerance excludes single-pass bf16/tf32 tensor-core math.
#include "trimkv_internal.cuh"

namespace tkv {

namespace {

constexpr int GH_WARPS = 8;   // warps per CTA of the hidden-layer kernel
constexpr int GH_JW = 4;      // hidden units per warp
constexpr int GH_RW = 8;      // rows per register tile

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// u[lb][r][j] = SiLU(x[lb][r][:] . W1[layer][j][:] + b1[layer][j])
__global__ void __launch_bounds__(GH_WARPS * 32)
gate_hidden_kernel(const float* __restrict__ x, const float* __restrict__ W1, const float* __restrict__ b1,
                   float* __restrict__ u, int layer0, int R, int D, int dg) {
    const int lb = blockIdx.y;
    const int layer = layer0 + lb;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j0 = (blockIdx.x * GH_WARPS + warp) * GH_JW;
    if (j0 >= dg) return;
    const float* Wb = W1 + ((size_t)layer * dg + j0) * D;
    const float* xb = x + (size_t)lb * R * D;
    const int nj = min(GH_JW, dg - j0);

    for (int r0 = 0; r0 < R; r0 += GH_RW) {
        const int nr = min(GH_RW, R - r0);
        float acc[GH_RW][GH_JW];
#pragma unroll
        for (int a = 0; a < GH_RW; ++a)
#pragma unroll
            for (int b = 0; b < GH_JW; ++b) acc[a][b] = 0.f;

        for (int d0 = lane * 4; d0 < D; d0 += 128) {
            float4 w[GH_JW];
#pragma unroll
            for (int jj = 0; jj < GH_JW; ++jj)
                w[jj] = (jj < nj) ? __ldg(reinterpret_cast<const float4*>(Wb + (size_t)jj * D + d0))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int rr = 0; rr < GH_RW; ++rr) {
                if (rr < nr) {
                    const float4 xv = __ldg(reinterpret_cast<const float4*>(xb + (size_t)(r0 + rr) * D + d0));
#pragma unroll
                    for (int jj = 0; jj < GH_JW; ++jj) {
                        acc[rr][jj] = fmaf(xv.x, w[jj].x, acc[rr][jj]);
                        acc[rr][jj] = fmaf(xv.y, w[jj].y, acc[rr][jj]);
                        acc[rr][jj] = fmaf(xv.z, w[jj].z, acc[rr][jj]);
                        acc[rr][jj] = fmaf(xv.w, w[jj].w, acc[rr][jj]);
                    }
                }
            }
        }
#pragma unroll
        for (int rr = 0; rr < GH_RW; ++rr) {
#pragma unroll
            for (int jj = 0; jj < GH_JW; ++jj) {
                float s = warp_sum(acc[rr][jj]);
                if (lane == 0 && rr < nr && jj < nj) {
                    float z = s + __ldg(b1 + (size_t)layer * dg + j0 + jj);
                    float sil = z / (1.0f + expf(-z));
                    u[((size_t)lb * R + r0 + rr) * dg + j0 + jj] = sil;
                }
            }
        }
    }
}

constexpr int GO_RT = 8;  // rows per tile of the output kernel

// s[lb][r][h] = w_g . (W2[layer][h] u[lb][r] + b2[layer][h]) + b_g ; then beta / lambda / c.
__global__ void __launch_bounds__(256)
gate_out_kernel(const float* __restrict__ u, const float* __restrict__ W2, const float* __restrict__ b2,
                const float* __restrict__ w_g, float b_g, int layer0, int R, int dg, int de, int H, int horizon,
                float* __restrict__ beta, float* __restrict__ lam, float* __restrict__ cterm) {
    extern __shared__ float sm[];           // [GO_RT][dg] rows of u, then [8 warps][GO_RT] partial sums
    float* su = sm;
    float* spart = sm + GO_RT * dg;
    const int h = blockIdx.x, lb = blockIdx.y;
    const int layer = layer0 + lb;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float* W2h = W2 + ((size_t)layer * H + h) * de * dg;
    const float* b2h = b2 + ((size_t)layer * H + h) * de;

    for (int r0 = blockIdx.z * GO_RT; r0 < R; r0 += gridDim.z * GO_RT) {
        const int nr = min(GO_RT, R - r0);
        __syncthreads();
        for (int i = threadIdx.x; i < nr * dg; i += blockDim.x)
            su[i] = u[((size_t)lb * R + r0) * dg + i];
        __syncthreads();
        float part[GO_RT];
#pragma unroll
        for (int rr = 0; rr < GO_RT; ++rr) part[rr] = 0.f;
        for (int k = warp; k < de; k += 8) {
            float acc[GO_RT];
#pragma unroll
            for (int rr = 0; rr < GO_RT; ++rr) acc[rr] = 0.f;
            for (int j = lane * 4; j < dg; j += 128) {
                const float4 w = __ldg(reinterpret_cast<const float4*>(W2h + (size_t)k * dg + j));
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
            const float wg = __ldg(w_g + k), bb = __ldg(b2h + k);
#pragma unroll
            for (int rr = 0; rr < GO_RT; ++rr) {
                float e = warp_sum(acc[rr]) + bb;
                part[rr] = fmaf(wg, e, part[rr]);
            }
        }
        if (lane == 0) {
#pragma unroll
            for (int rr = 0; rr < GO_RT; ++rr) spart[warp * GO_RT + rr] = part[rr];
        }
        __syncthreads();
        if (threadIdx.x < nr) {
            const int rr = threadIdx.x;
            float s = 0.f;
            for (int w = 0; w < 8; ++w) s += spart[w * GO_RT + rr];
            s += b_g;
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

}  // namespace

void launch_gate(const GateParams& gp, const float* x, float* u_scratch, int layer0, int nlayers, int rows_per_layer,
                 float* beta, float* lam, float* c, cudaStream_t st) {
    const int per_cta = GH_WARPS * GH_JW;
    dim3 g1((gp.dg + per_cta - 1) / per_cta, nlayers);
    gate_hidden_kernel<<<g1, GH_WARPS * 32, 0, st>>>(x, gp.W1, gp.b1, u_scratch, layer0, rows_per_layer, gp.D, gp.dg);
    int zt = (rows_per_layer + GO_RT - 1) / GO_RT;
    if (zt > 64) zt = 64;
    dim3 g2(gp.H, nlayers, zt);
    size_t smem = (size_t)(GO_RT * gp.dg + 8 * GO_RT) * sizeof(float);
    gate_out_kernel<<<g2, 256, smem, st>>>(u_scratch, gp.W2, gp.b2, gp.w_g, gp.b_g, layer0, rows_per_layer, gp.dg,
                                           gp.de, gp.H, gp.horizon, beta, lam, c);
    count_launch(2);
}

}  // namespace tkv
