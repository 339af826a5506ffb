// Tensor-core form of the gate's hidden layer for chunk-sized calls (Sec. 4.1 / 5.1: Proj's first layer,
// z = W1 x, here for hundreds to thousands of token rows of one layer at once, i.e. a dense contraction
// Z[R, d_g] = X[R, D] W1[d_g, D]^T).
//
// The 1e-5 relative tolerance on the gate outputs rules out one-pass TF32, so the product is evaluated as
// three TF32 products with fp32 accumulation ("3xTF32"): every fp32 operand a is split into hi = a rounded to
// TF32 and lo = a - hi (exact in fp32), and Z = Xhi Whi^T + Xhi Wlo^T + Xlo Whi^T (the dropped lo*lo term is
// below 2^-22 relative).  W1 is split once when the gate is set, X by a small kernel per call.
//
// Kernel: one 128 x 128 output tile per CTA, K in blocks of 32 floats.  A producer thread streams the four
// operand tiles of a k-block (Xhi, Xlo, Whi, Wlo; 16 KB each, 128-byte swizzle) with TMA into a 3-stage ring;
// one thread issues tcgen05.mma (kind::tf32, M 128, N 128, K 8) with the accumulator in tensor memory; four
// warps read the accumulator back with tcgen05.ld and store the tile.  Every wait is bounded.
#include <cuda.h>

#include <algorithm>

#include "trimkv_internal.cuh"

namespace tkv {

namespace {

constexpr int TM = 128, TN = 128, TK = 32;          // tile (rows, hidden units, floats of K per block)
constexpr int TC_STAGES = 3;
constexpr int TILE_BYTES = TM * TK * 4;             // 16 KB: one operand tile of a k-block
constexpr int STAGE_BYTES_TC = 4 * TILE_BYTES;      // Xhi, Xlo, Whi, Wlo
constexpr int TC_SMEM = TC_STAGES * STAGE_BYTES_TC + 1024 /*alignment slack*/ + 256 /*barriers, tmem address*/;
constexpr int TC_THREADS = 192;                     // warps 0-3 epilogue, warp 4 TMA producer, warp 5 MMA issuer
constexpr unsigned TC_WAIT_LIMIT = 1u << 22;
constexpr int TC_SEG = 8;                           // k-blocks per accumulation segment of the main term (32 MMA steps)
constexpr int TMEM_COLS = 512;                      // columns 0-127, 128-255: main accumulators (ping-pong); 256-383: small terms

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void bar_init(uint32_t bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool bar_wait_bounded(uint32_t bar, uint32_t parity) {
    for (unsigned it = 0; it < TC_WAIT_LIMIT; ++it)
        if (bar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
// Shared-memory matrix descriptor of a K-major operand tile stored with the 128-byte swizzle: rows of 128 bytes,
// groups of 8 rows 1024 bytes apart (stride byte offset), tile base aligned to 1024 bytes.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= (uint64_t)1 << 16;                           // leading byte offset (unused with swizzle): 1
    d |= (uint64_t)(1024 >> 4) << 32;                 // stride byte offset: 1024 bytes
    d |= (uint64_t)1 << 46;                           // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                           // layout: 128-byte swizzle
    return d;
}
// Instruction descriptor: D fp32, A and B TF32, both K-major, N = 128, M = 128.
constexpr uint32_t UMMA_IDESC_TF32 = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(TN >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);

__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(UMMA_IDESC_TF32), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// hi = a rounded to TF32 (10 explicit mantissa bits, round to nearest), lo = a - hi.
__global__ void __launch_bounds__(256)
split_tf32_kernel(const float4* __restrict__ in, float4* __restrict__ hi, float4* __restrict__ lo, long long n4) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
        const float4 a = in[i];
        float4 h, l;
        auto sp = [](float x, float& xh, float& xl) {
            const uint32_t u = __float_as_uint(x);
            const uint32_t r = ((u & 0x7f800000u) == 0x7f800000u) ? u : ((u + 0x1000u) & 0xffffe000u);   // inf/NaN kept
            xh = __uint_as_float(r);
            xl = x - xh;
        };
        sp(a.x, h.x, l.x); sp(a.y, h.y, l.y); sp(a.z, h.z, l.z); sp(a.w, h.w, l.w);
        hi[i] = h;
        lo[i] = l;
    }
}

// Z[r][n] = sum_k X[r][k] W[n][k] for the tile (blockIdx.x: 128 rows of X, blockIdx.y: 128 rows of W), written to
// z[r * ldz + n].  Tensor maps: X hi / lo over [rows_alloc][D], W hi / lo over [L * d_g][D]; w_row0 = layer * d_g.
__global__ void __launch_bounds__(TC_THREADS, 1)
gate_gemm_tf32x3_kernel(const __grid_constant__ CUtensorMap map_xhi, const __grid_constant__ CUtensorMap map_xlo,
                        const __grid_constant__ CUtensorMap map_whi, const __grid_constant__ CUtensorMap map_wlo,
                        float* __restrict__ z, int R, int D, int ldz, int w_row0, int32_t* err) {
    extern __shared__ unsigned char tc_smem_raw[];
    const uint32_t raw = smem_addr(tc_smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;                        // operand tiles need 1024-byte alignment
    const uint32_t bars = base + TC_STAGES * STAGE_BYTES_TC;             // full[3], empty[3], accum: 8 bytes each
    unsigned char* gen = tc_smem_raw + (base - raw) + TC_STAGES * STAGE_BYTES_TC;
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(gen + 128);
    volatile int* s_fail = reinterpret_cast<volatile int*>(gen + 136);
    const uint32_t full0 = bars, empty0 = bars + 8 * TC_STAGES, accum = bars + 16 * TC_STAGES;
    const uint32_t segfull0 = accum + 8, segfree0 = accum + 24;          // two each
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
    const int KB = D / TK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_STAGES; ++s) { bar_init(full0 + 8 * s, 1); bar_init(empty0 + 8 * s, 1); }
        bar_init(accum, 1);
        for (int a = 0; a < 2; ++a) { bar_init(segfull0 + 8 * a, 1); bar_init(segfree0 + 8 * a, 4); }
        *s_fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 5) {                                                     // tensor memory: 128 columns for the accumulator
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr((const void*)s_tmem)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *s_tmem;

    if (warp == 4) {
        if (lane == 0) {                                                 // ---- TMA producer
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % TC_STAGES;
                if (kb >= TC_STAGES && !bar_wait_bounded(empty0 + 8 * s, ((kb / TC_STAGES) - 1) & 1)) { *s_fail = 1; break; }
                const uint32_t dst = base + s * STAGE_BYTES_TC;
                bar_expect_tx(full0 + 8 * s, STAGE_BYTES_TC);
                tma_load_2d(dst, &map_xhi, kb * TK, m0, full0 + 8 * s);
                tma_load_2d(dst + TILE_BYTES, &map_xlo, kb * TK, m0, full0 + 8 * s);
                tma_load_2d(dst + 2 * TILE_BYTES, &map_whi, kb * TK, w_row0 + n0, full0 + 8 * s);
                tma_load_2d(dst + 3 * TILE_BYTES, &map_wlo, kb * TK, w_row0 + n0, full0 + 8 * s);
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {                                                 // ---- MMA issuer
            bool ok = true;
            for (int kb = 0; kb < KB && ok; ++kb) {
                const int s = kb % TC_STAGES;
                if (!bar_wait_bounded(full0 + 8 * s, (kb / TC_STAGES) & 1)) { *s_fail = 1; ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t st = base + s * STAGE_BYTES_TC;
                const uint64_t xhi = umma_desc_sw128(st), xlo = umma_desc_sw128(st + TILE_BYTES);
                const uint64_t whi = umma_desc_sw128(st + 2 * TILE_BYTES), wlo = umma_desc_sw128(st + 3 * TILE_BYTES);
                // Tensor-core accumulation truncates, so the error of an accumulation chain grows with its length and
                // with the accumulator's magnitude.  The main term is therefore accumulated in segments of TC_SEG
                // k-blocks, alternating between two accumulators that the epilogue warps drain into fp32 registers
                // (rounded adds) while the next segment runs; the two small cross terms have an accumulator of their own.
                const int seg = kb / TC_SEG, a = seg & 1;
                const bool seg_first = kb % TC_SEG == 0, seg_last = kb % TC_SEG == TC_SEG - 1 || kb == KB - 1;
                if (seg_first && seg >= 2) {
                    if (!bar_wait_bounded(segfree0 + 8 * a, ((seg >> 1) - 1) & 1)) { *s_fail = 1; ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                }
                const uint32_t acc_main = tmem + (uint32_t)(a * TN), acc_small = tmem + (uint32_t)(2 * TN);
#pragma unroll
                for (int k8 = 0; k8 < TK / 8; ++k8) {                    // K = 8 per instruction: 32 bytes along the row
                    const uint64_t adv = (uint64_t)(k8 * 32 >> 4);
                    umma_tf32(acc_small, xlo + adv, whi + adv, (kb | k8) != 0);
                    umma_tf32(acc_small, xhi + adv, wlo + adv, 1u);
                    umma_tf32(acc_main, xhi + adv, whi + adv, (seg_first && k8 == 0) ? 0u : 1u);
                }
                umma_commit(empty0 + 8 * s);                             // frees the stage when these MMAs have read it
                if (seg_last) umma_commit(segfull0 + 8 * a);             // this segment's accumulator is complete
            }
            if (ok) umma_commit(accum);                                  // everything, the small terms included
        }
    } else {
        // ---- epilogue: warp w owns accumulator lanes (rows) 32 w .. 32 w + 31; a thread sums its row's 128 columns
        float sum[TN];
#pragma unroll
        for (int q = 0; q < TN; ++q) sum[q] = 0.f;
        auto drain = [&](uint32_t col0) {                                // sum += accumulator columns col0 .. col0 + 127
#pragma unroll
            for (int c = 0; c < TN / 32; ++c) {
                uint32_t t[32];
                const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + col0 + (uint32_t)(c * 32);
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                    "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                    "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                    : "=r"(t[0]), "=r"(t[1]), "=r"(t[2]), "=r"(t[3]), "=r"(t[4]), "=r"(t[5]), "=r"(t[6]), "=r"(t[7]), "=r"(t[8]),
                      "=r"(t[9]), "=r"(t[10]), "=r"(t[11]), "=r"(t[12]), "=r"(t[13]), "=r"(t[14]), "=r"(t[15]), "=r"(t[16]),
                      "=r"(t[17]), "=r"(t[18]), "=r"(t[19]), "=r"(t[20]), "=r"(t[21]), "=r"(t[22]), "=r"(t[23]), "=r"(t[24]),
                      "=r"(t[25]), "=r"(t[26]), "=r"(t[27]), "=r"(t[28]), "=r"(t[29]), "=r"(t[30]), "=r"(t[31])
                    : "r"(taddr));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int q = 0; q < 32; ++q) sum[c * 32 + q] += __uint_as_float(t[q]);
            }
        };
        const int nseg = (KB + TC_SEG - 1) / TC_SEG;
        bool ok = true;
        for (int seg = 0; seg < nseg && ok; ++seg) {
            const int a = seg & 1;
            int got = 1;
            if (lane == 0) got = bar_wait_bounded(segfull0 + 8 * a, (seg >> 1) & 1) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, got, 0) != 0;
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            drain((uint32_t)(a * TN));
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(segfree0 + 8 * a) : "memory");
        }
        if (ok) {
            int got = 1;
            if (lane == 0) got = bar_wait_bounded(accum, 0) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, got, 0) != 0;
        }
        if (!ok) {
            if (lane == 0) *s_fail = 1;
        } else {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            drain((uint32_t)(2 * TN));                                   // the small cross terms
            const int row = m0 + warp * 32 + lane;
            if (row < R) {
                float4* dstp = reinterpret_cast<float4*>(z + (size_t)row * ldz + n0);
#pragma unroll
                for (int q = 0; q < TN / 4; ++q) dstp[q] = make_float4(sum[4 * q], sum[4 * q + 1], sum[4 * q + 2], sum[4 * q + 3]);
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 5) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *s_fail) latch_error(err, TRIMKV_E_TIMEOUT);
}

}  // namespace

// ------------------------------------------------------------------ host side
struct GateTcState {
    CUtensorMap xhi, xlo, whi, wlo;
    float *d_xhi, *d_xlo;
    long long rows_alloc;
    int D, dg;
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// fp32 matrix [rows][D], row-major; box = 32 floats (128 bytes) x 128 rows, 128-byte swizzle, zero fill outside.
bool encode_map(CUtensorMap* m, float* base, long long rows, int D) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)D * 4};
    const cuuint32_t box[2] = {(cuuint32_t)TK, (cuuint32_t)TM};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool gate_tc_supported(int D, int dg) { return D % TK == 0 && dg % TN == 0 && D >= 4 * TK; }   // every K-third needs a block

GateTcState* gate_tc_create(float* xhi, float* xlo, long long rows_alloc, float* whi, float* wlo, int L, int dg, int D) {
    if (!gate_tc_supported(D, dg)) return nullptr;
    GateTcState* s = new GateTcState();
    s->d_xhi = xhi; s->d_xlo = xlo; s->rows_alloc = rows_alloc; s->D = D; s->dg = dg;
    const bool ok = encode_map(&s->xhi, xhi, rows_alloc, D) && encode_map(&s->xlo, xlo, rows_alloc, D) &&
                    encode_map(&s->whi, whi, (long long)L * dg, D) && encode_map(&s->wlo, wlo, (long long)L * dg, D) &&
                    cudaFuncSetAttribute(gate_gemm_tf32x3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        delete s;
        return nullptr;
    }
    return s;
}

void gate_tc_destroy(GateTcState* s) { delete s; }

void launch_split_tf32(const float* in, float* hi, float* lo, long long n, cudaStream_t st) {
    const long long n4 = n / 4;                      // callers pass multiples of 4
    int grid = (int)std::min<long long>((n4 + 255) / 256, 148 * 8);
    if (grid < 1) grid = 1;
    split_tf32_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const float4*>(in), reinterpret_cast<float4*>(hi),
                                            reinterpret_cast<float4*>(lo), n4);
    count_launch();
}

// z[r][j] = x[r][:] . W1[layer][j][:] for R rows (R <= rows_alloc of the state); ldz = dg.
void launch_gate_gemm_tc(GateTcState* s, const float* x, int R, int layer, float* z, int32_t* err, cudaStream_t st) {
    launch_split_tf32(x, s->d_xhi, s->d_xlo, (long long)R * s->D, st);
    dim3 grid((R + TM - 1) / TM, s->dg / TN);
    gate_gemm_tf32x3_kernel<<<grid, TC_THREADS, TC_SMEM, st>>>(s->xhi, s->xlo, s->whi, s->wlo, z, R, s->D, s->dg,
                                                               layer * s->dg, err);
    count_launch();
}

}  // namespace tkv
