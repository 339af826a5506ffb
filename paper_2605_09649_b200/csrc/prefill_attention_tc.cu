// Tensor-core (tcgen05) form of the chunk's causal attention over the ragged per-(layer, head) pools (Sec. 2.1 attention
// restricted to the retained set, Eq. (1) with r in {0,1}; same contract as the mma.sync kernel next door): chunk token j
// sees entry e of its pool iff e < n_old + j + 1.  bf16, d = 128.
//
// One CTA per (pool, block of 256 / g chunk tokens): 256 (token, query head) rows in two groups of 128 that share every
// K/V tile.  A tile is one 64-entry page.  The page's rows are stored with their 16-byte chunks permuted inside each
// 128-byte half by (slot & 7); copied half by half with TMA (box 64 columns x 64 rows of the arena seen as a matrix of
// 256-byte rows) they land in shared memory exactly in the tensor core's 128-byte-swizzle layout: K halves as K-major
// operands of S = Q K^T, V halves as MN-major operands of O += P V.  Roles: warps 0-3 / 4-7 are the softmax warps of
// group 0 / 1 (a thread owns one row: S read from tensor memory, masked, exponentiated, P written back to tensor memory as
// bf16 pairs, where the P V product reads it as its A operand), warp 8 issues the TMA copies into a 4-stage ring, warps 9
// and 10 each issue the MMAs of one group (S is double-buffered in tensor memory and issued two tiles ahead of the P V that
// needs the softmax result, so the tensor pipe works while the softmax warps compute, and neither group's issuer ever
// waits for the other group; P overwrites the first half of its tile's S).  O accumulates in tensor memory; the
// running maximum is only raised (and O rescaled) when it grows by more than 2^8, which keeps every exponential finite and
// leaves the final O / l unchanged.  A third of the exponentials are evaluated with FMAs instead of the special-function
// unit.  Every wait is bounded; a wait that runs out latches TRIMKV_E_TIMEOUT.
#include <cuda.h>

#include "trimkv_internal.cuh"

namespace tkv {

namespace {

constexpr int A_TILE = 64;                            // entries per tile: one page
constexpr int A_ROWS = 128;                           // query rows per softmax group
constexpr int A_STAGES = 4;
constexpr int A_PLANE = A_TILE * 128;                 // 8 KB: 64 entries x one 128-byte half of the row
constexpr int A_STAGE_BYTES = 4 * A_PLANE;            // K half 0, K half 1, V half 0, V half 1
constexpr int A_QPLANE = A_ROWS * 128;                // 16 KB: 128 query rows x one half
constexpr int A_Q_BYTES = 2 * 2 * A_QPLANE;           // two groups, two halves
constexpr int A_OFF_Q = A_STAGES * A_STAGE_BYTES;
constexpr int A_OFF_BAR = A_OFF_Q + A_Q_BYTES;
constexpr int A_SMEM = A_OFF_BAR + 256 + 1024;        // barriers and flags, alignment slack
constexpr int A_THREADS = 352;                       // 8 softmax warps, the TMA warp, one MMA-issuing warp per group
constexpr unsigned A_WAIT_LIMIT = 1u << 22;
constexpr int A_TMEM_COLS = 512;                      // group g: S of even / odd tiles at columns 128 g, 128 g + 64; O at 256 + 128 g.
                                                      // P of a tile (bf16 pairs, the A operand of P V) overwrites the first 32
                                                      // columns of that tile's S once the softmax threads hold S in registers
constexpr int A_POLY_EVERY = 3;                       // share of the exponentials computed with FMAs: 1 / A_POLY_EVERY
constexpr float A_RESCALE_STEP = 8.0f;                // log2 units the running maximum may lag behind

__device__ __forceinline__ uint32_t a_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void a_bar_init(uint32_t bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void a_bar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void a_bar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool a_bar_wait(uint32_t bar, uint32_t parity) {      // false: gave up
    for (unsigned it = 0; it < A_WAIT_LIMIT; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void a_tma_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
// Shared-memory matrix descriptor, 128-byte swizzle: rows of 128 bytes, groups of 8 rows 1024 bytes apart (stride byte
// offset).  lead_bytes: distance between 64-element blocks along M/N of an MN-major operand (unused for K-major: 16).
__device__ __forceinline__ uint64_t a_desc(uint32_t saddr, uint32_t lead_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lead_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptors: D fp32, A and B bf16, M = 128.  S: both K-major, N = 64.  P V: B (V) MN-major, N = 128.
constexpr uint32_t A_IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(64 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
constexpr uint32_t A_IDESC_PV =
    (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

__device__ __forceinline__ void a_umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// A operand in tensor memory: row = lane, two bf16 per 32-bit column (lower k in the low half), 8 columns per K = 16.
__device__ __forceinline__ void a_umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(tmem_d),
        "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void a_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void a_tmem_ld32(uint32_t taddr, uint32_t* t) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(t[0]), "=r"(t[1]), "=r"(t[2]), "=r"(t[3]), "=r"(t[4]), "=r"(t[5]), "=r"(t[6]), "=r"(t[7]), "=r"(t[8]),
          "=r"(t[9]), "=r"(t[10]), "=r"(t[11]), "=r"(t[12]), "=r"(t[13]), "=r"(t[14]), "=r"(t[15]), "=r"(t[16]),
          "=r"(t[17]), "=r"(t[18]), "=r"(t[19]), "=r"(t[20]), "=r"(t[21]), "=r"(t[22]), "=r"(t[23]), "=r"(t[24]),
          "=r"(t[25]), "=r"(t[26]), "=r"(t[27]), "=r"(t[28]), "=r"(t[29]), "=r"(t[30]), "=r"(t[31])
        : "r"(taddr));
}
__device__ __forceinline__ void a_tmem_st32(uint32_t taddr, const uint32_t* t) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(t[0]), "r"(t[1]), "r"(t[2]), "r"(t[3]), "r"(t[4]), "r"(t[5]), "r"(t[6]), "r"(t[7]), "r"(t[8]), "r"(t[9]), "r"(t[10]),
        "r"(t[11]), "r"(t[12]), "r"(t[13]), "r"(t[14]), "r"(t[15]), "r"(t[16]), "r"(t[17]), "r"(t[18]), "r"(t[19]), "r"(t[20]),
        "r"(t[21]), "r"(t[22]), "r"(t[23]), "r"(t[24]), "r"(t[25]), "r"(t[26]), "r"(t[27]), "r"(t[28]), "r"(t[29]), "r"(t[30]),
        "r"(t[31])
        : "memory");
}
// Two fp32 values per 64-bit register: the packed fma / add forms halve the instruction count of the softmax loop.
__device__ __forceinline__ uint64_t a_pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void a_unpack2(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t a_fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t a_add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float a_ex2(float x) {                      // 2^x, one instruction; 2^-inf = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 2^x for two values on the FMA pipe (the special-function unit is the softmax loop's narrowest pipe, so a share of the
// exponentials goes this way): x = n + f with n = round(x) taken from the mantissa of x + 1.5 * 2^23 and f in [-1/2, 1/2];
// 2^f by a cubic (relative error 7.5e-5, far below the bf16 rounding of P); n is added into the exponent field.
// x is clamped at -125 from below, so a masked entry weighs 2^-125 instead of 0.
__device__ __forceinline__ void a_exp2_fma2(uint64_t x2, float& p0, float& p1) {
    float x0, x1;
    a_unpack2(x2, x0, x1);
    const uint64_t xc = a_pack2(fmaxf(x0, -125.0f), fmaxf(x1, -125.0f));
    const uint64_t magic = a_pack2(12582912.0f, 12582912.0f), nmagic = a_pack2(-12582912.0f, -12582912.0f);
    const uint64_t t2 = a_add2(xc, magic);
    const uint64_t f2 = a_fma2(a_add2(t2, nmagic), a_pack2(-1.0f, -1.0f), xc);
    uint64_t q2 = a_fma2(a_pack2(0.055171650f, 0.055171650f), f2, a_pack2(0.24261113f, 0.24261113f));
    q2 = a_fma2(q2, f2, a_pack2(0.69326097f, 0.69326097f));
    q2 = a_fma2(q2, f2, a_pack2(0.99992806f, 0.99992806f));
    float q0, q1, t0, t1;
    a_unpack2(q2, q0, q1);
    a_unpack2(t2, t0, t1);
    p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(t0) << 23));
    p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(t1) << 23));
}
__device__ __forceinline__ float a_max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint32_t a_bf16x2(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ void a_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void a_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// grid = (token blocks, B * H pools of `layer`); q, out: [B, n_new, Hq, 128] bf16.  map_kv: the K/V arena as a matrix of
// 256-byte rows (128 bf16), box 64 columns x 64 rows.
__global__ void __launch_bounds__(A_THREADS, 1)
prefill_attn_tc_kernel(const __grid_constant__ CUtensorMap map_kv, CacheView cv, int layer, int n_new, int g, int Hq,
                       const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ out, float scale_log2) {
    extern __shared__ unsigned char a_smem_raw[];
    const uint32_t raw = a_smem(a_smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;                        // operand tiles need 1024-byte alignment
    unsigned char* gen = a_smem_raw + (base - raw);
    const uint32_t bars = base + A_OFF_BAR;
    const uint32_t full0 = bars, empty0 = bars + 32, s_ready0 = bars + 64 /* [group][tile parity] */, p_ready0 = bars + 96,
                   pv_done0 = bars + 112;
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(gen + A_OFF_BAR + 128);
    volatile int* s_fail = reinterpret_cast<volatile int*>(gen + A_OFF_BAR + 136);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const int tt = 256 / g;                                              // chunk tokens per CTA
    const int i0 = ((int)gridDim.x - 1 - (int)blockIdx.x) * tt;          // longest blocks first
    const int h = blockIdx.y % cv.H, b = blockIdx.y / cv.H;
    const long long pool = ((long long)b * cv.L + layer) * cv.H + h;
    const int n_old = cv.len[pool] - n_new;                              // entries kept from before the chunk
    if (i0 >= n_new || n_old < 0) return;                                // (n_old < 0: the append failed; its error is latched)
    const int limit_max = n_old + min(n_new, i0 + tt);                   // entries any token of this block may see
    const int ntile = (limit_max + A_TILE - 1) / A_TILE;
    const int32_t* bt = cv.block_table + pool * cv.maxpp;

    if (threadIdx.x == 0) {
        for (int s = 0; s < A_STAGES; ++s) { a_bar_init(full0 + 8 * s, 1); a_bar_init(empty0 + 8 * s, 2); }   // both issuers free a stage
        for (int gq = 0; gq < 2; ++gq) {
            a_bar_init(s_ready0 + 16 * gq, 1);
            a_bar_init(s_ready0 + 16 * gq + 8, 1);
            a_bar_init(p_ready0 + 8 * gq, 4);
            a_bar_init(pv_done0 + 8 * gq, 1);
        }
        *s_fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(a_smem((const void*)s_tmem)),
                     "r"(A_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // ---- per-row facts of the softmax threads, and the Q tile: row R of the block = (token i0 + R / g, head R % g)
    const int grp = (warp >> 2) & 1, wl = warp & 3;
    const int r = wl * 32 + lane;                                        // row inside the group = tensor-memory lane
    const int R = grp * A_ROWS + r;
    const int tok = i0 + R / g, head = R % g;
    const bool valid = warp < 8 && R < tt * g && tok < n_new;
    const int limit = valid ? n_old + tok + 1 : 0;                       // entries this row sees
    if (warp < 8) {
        const uint4* src = reinterpret_cast<const uint4*>(q + (((size_t)b * n_new + (valid ? tok : 0)) * Hq + (size_t)h * g + head) * 128);
        unsigned char* qdst = gen + A_OFF_Q + grp * 2 * A_QPLANE + r * 128;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
            const uint4 v = valid ? src[c] : make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(qdst + (c >> 3) * A_QPLANE + (((c & 7) ^ (r & 7)) << 4)) = v;
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");         // Q and the barriers, before the async proxy uses them
    a_fence_before();
    __syncthreads();
    a_fence_after();
    const uint32_t tmem = *s_tmem;

    if (warp == 8) {
        // ---- TMA producer: lane l holds the page of tile i0 + l of the current run of 32 tiles
        int page_id = 0;
        for (int i = 0; i < ntile; ++i) {
            if ((i & 31) == 0) page_id = (i + lane < ntile) ? bt[i + lane] : 0;
            const int page = __shfl_sync(0xffffffffu, page_id, i & 31);
            const int s = i % A_STAGES;
            int ok = 1;
            if (lane == 0) {
                if (i >= A_STAGES) ok = a_bar_wait(empty0 + 8 * s, ((i / A_STAGES) - 1) & 1) ? 1 : 0;
                if (ok) {
                    const uint32_t dst = base + s * A_STAGE_BYTES;
                    const int krow = (int)((((long long)b * cv.P_seq + page) * 2) * PAGE);
                    a_bar_expect_tx(full0 + 8 * s, A_STAGE_BYTES);
                    a_tma_2d(dst, &map_kv, 0, krow, full0 + 8 * s);
                    a_tma_2d(dst + A_PLANE, &map_kv, 64, krow, full0 + 8 * s);
                    a_tma_2d(dst + 2 * A_PLANE, &map_kv, 0, krow + PAGE, full0 + 8 * s);
                    a_tma_2d(dst + 3 * A_PLANE, &map_kv, 64, krow + PAGE, full0 + 8 * s);
                }
            }
            if (__shfl_sync(0xffffffffu, ok, 0) == 0) {
                if (lane == 0) *s_fail = 1;
                break;
            }
        }
    } else if (warp >= 9) {
        if (lane == 0) {
            // ---- MMA issuer of group gq.  S has two buffers, so S of tiles i + 1 and i + 2 are issued before P V of tile
            // i needs its P: the softmax threads never wait for S, and the tensor pipe has the other group's and the
            // next tiles' products to run while a group computes its exponentials.  S of tile i + 2 overwrites the buffer
            // that held S and P of tile i; it is issued after P V of tile i, and the pipe runs in issue order.
            const int gq = warp - 9;
            bool ok = true;
            const uint32_t d_s0 = tmem + 128 * gq, d_o = tmem + 256 + 128 * gq;
            const uint64_t qdesc0 = a_desc(base + A_OFF_Q + (gq * 2) * A_QPLANE, 16), qdesc1 = a_desc(base + A_OFF_Q + (gq * 2 + 1) * A_QPLANE, 16);
            auto issue_s = [&](int t) {                                  // S = Q K^T of tile t into buffer t & 1
                const int s = t % A_STAGES;
                if (!a_bar_wait(full0 + 8 * s, (t / A_STAGES) & 1)) { ok = false; return; }
                a_fence_after();
                const uint32_t st = base + s * A_STAGE_BYTES, d_s = d_s0 + 64 * (t & 1);
                const uint64_t kdesc0 = a_desc(st, 16), kdesc1 = a_desc(st + A_PLANE, 16);
#pragma unroll
                for (int j = 0; j < 4; ++j)                              // 16 of d per instruction, 32 bytes along the row
                    a_umma(d_s, qdesc0 + (uint64_t)(j * 32 >> 4), kdesc0 + (uint64_t)(j * 32 >> 4), A_IDESC_S, j != 0);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    a_umma(d_s, qdesc1 + (uint64_t)(j * 32 >> 4), kdesc1 + (uint64_t)(j * 32 >> 4), A_IDESC_S, 1u);
                a_commit(s_ready0 + 16 * gq + 8 * (t & 1));
            };
            auto issue_pv = [&](int t) {                                 // O += P V of tile t
                const uint32_t st = base + (t % A_STAGES) * A_STAGE_BYTES, a_p = d_s0 + 64 * (t & 1);
                if (!a_bar_wait(p_ready0 + 8 * gq, t & 1)) { ok = false; return; }
                a_fence_after();
                const uint64_t vdesc = a_desc(st + 2 * A_PLANE, A_PLANE);         // the second 64 dims: one plane further
#pragma unroll
                for (int j = 0; j < A_TILE / 16; ++j)                    // 16 entries per instruction: P +8 columns, V +2 row groups
                    a_umma_ts(d_o, a_p + j * 8, vdesc + (uint64_t)(j * 2048 >> 4), A_IDESC_PV, (t | j) != 0);
                a_commit(pv_done0 + 8 * gq);
                a_commit(empty0 + 8 * (t % A_STAGES));                   // this group is done with the stage
            };
            issue_s(0);
            if (ok && ntile > 1) issue_s(1);
            for (int i = 0; i < ntile && ok; ++i) {
                issue_pv(i);
                if (ok && i + 2 < ntile) issue_s(i + 2);
            }
            if (!ok) *s_fail = 1;
        }
    } else {
        // ---- softmax warps
        const uint32_t lane_addr = tmem + ((uint32_t)(wl * 32) << 16);
        const uint32_t s_col0 = (uint32_t)(128 * grp), o_col = (uint32_t)(256 + 128 * grp);
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;
        for (int i = 0; i < ntile; ++i) {
            ok = __all_sync(0xffffffffu, a_bar_wait(s_ready0 + 16 * grp + 8 * (i & 1), (i >> 1) & 1));
            const uint32_t s_col = s_col0 + 64u * (uint32_t)(i & 1);
            if (!ok) break;
            a_fence_after();
            uint32_t sv[64];
            a_tmem_ld32(lane_addr + s_col, sv);
            a_tmem_ld32(lane_addr + s_col + 32, sv + 32);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            const int e0 = i * A_TILE;
            if (e0 + A_TILE > limit) {                                   // the tile crosses this row's causal limit
#pragma unroll
                for (int e = 0; e < 64; ++e)
                    if (e0 + e >= limit) sv[e] = 0xff800000u;            // -inf
            }
            float mq[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // four independent chains
#pragma unroll
            for (int e = 0; e < 64; e += 8) {
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    mq[c] = a_max3(mq[c], __uint_as_float(sv[e + 2 * c]), __uint_as_float(sv[e + 2 * c + 1]));
            }
            const float mx = fmaxf(fmaxf(mq[0], mq[1]), fmaxf(mq[2], mq[3]));
            const float m_new = mx * scale_log2;                         // scale_log2 > 0
            const bool resc = __any_sync(0xffffffffu, m_new > m_used + A_RESCALE_STEP);
            float alpha = 1.0f;
            if (resc) {
                const float mn = fmaxf(m_used, m_new);
                alpha = (m_used == -INFINITY) ? 0.0f : exp2f(m_used - mn);
                m_used = mn;
            }
            const float mref = (m_used == -INFINITY) ? 0.0f : m_used;    // a row that has seen nothing yet: every p = 0
            const uint64_t sc2 = a_pack2(scale_log2, scale_log2), nm2 = a_pack2(-mref, -mref);
            uint64_t sq[4] = {0ull, 0ull, 0ull, 0ull};                   // packed partial sums, four chains
            uint32_t pk[32];
#pragma unroll
            for (int e = 0; e < 64; e += 2) {
                const uint64_t x2 = a_fma2(a_pack2(__uint_as_float(sv[e]), __uint_as_float(sv[e + 1])), sc2, nm2);
                float p0, p1;
                if ((e >> 1) % A_POLY_EVERY == A_POLY_EVERY - 1) {       // every A_POLY_EVERY-th pair on the FMA pipe
                    a_exp2_fma2(x2, p0, p1);
                } else {
                    float x0, x1;
                    a_unpack2(x2, x0, x1);
                    p0 = a_ex2(x0);
                    p1 = a_ex2(x1);
                }
                sq[(e >> 1) & 3] = a_add2(sq[(e >> 1) & 3], a_pack2(p0, p1));
                pk[e >> 1] = a_bf16x2(p0, p1);
            }
            float sum;
            {
                float a0, a1;
                a_unpack2(a_add2(a_add2(sq[0], sq[1]), a_add2(sq[2], sq[3])), a0, a1);
                sum = a0 + a1;
            }
            l = l * alpha + sum;
            if (i > 0) {                                                 // P V of the previous tile: O complete (each phase is awaited once, in order)
                ok = __all_sync(0xffffffffu, a_bar_wait(pv_done0 + 8 * grp, (i - 1) & 1));
                if (!ok) break;
                a_fence_after();
                if (resc) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t ov[32];
                        a_tmem_ld32(lane_addr + o_col + c * 32, ov);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                        for (int e = 0; e < 32; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * alpha);
                        a_tmem_st32(lane_addr + o_col + c * 32, ov);
                    }
                    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                }
            }
            a_tmem_st32(lane_addr + s_col, pk);                          // P over the first half of this tile's S: the A operand of P V
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            a_fence_before();
            __syncwarp();
            if (lane == 0) a_bar_arrive(p_ready0 + 8 * grp);
        }
        if (ok) ok = __all_sync(0xffffffffu, a_bar_wait(pv_done0 + 8 * grp, (ntile - 1) & 1));
        if (!ok) {
            if (lane == 0) *s_fail = 1;
        } else {
            a_fence_after();
            const float inv = l > 0.f ? 1.0f / l : 0.f;
            uint4* op = reinterpret_cast<uint4*>(out + (((size_t)b * n_new + (valid ? tok : 0)) * Hq + (size_t)h * g + head) * 128);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t ov[32];
                a_tmem_ld32(lane_addr + o_col + c * 32, ov);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (valid) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint32_t w[4];
#pragma unroll
                        for (int k2 = 0; k2 < 4; ++k2) {
                            const __nv_bfloat162 pp = __floats2bfloat162_rn(__uint_as_float(ov[e + 2 * k2]) * inv,
                                                                             __uint_as_float(ov[e + 2 * k2 + 1]) * inv);
                            w[k2] = *reinterpret_cast<const uint32_t*>(&pp);
                        }
                        op[c * 4 + (e >> 3)] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        }
    }
    a_fence_before();
    __syncthreads();
    if (warp == 9) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(A_TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *s_fail) latch_error(cv.err, TRIMKV_E_TIMEOUT);
}

}  // namespace

// ------------------------------------------------------------------ host side
struct PrefillTcState {
    CUtensorMap map_kv;
};

namespace {

typedef CUresult (*EncodeTiledFnA)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFnA a_encode_fn() {
    static EncodeTiledFnA fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFnA>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

}  // namespace

bool prefill_tc_supported(const CacheView& cv, int is_bf16, int Hq) {
    const int g = cv.H > 0 ? Hq / cv.H : 0;
    const long long rows = (long long)cv.B * cv.P_seq * 2 * PAGE;
    return is_bf16 && cv.d == 128 && cv.swizzle && g >= 1 && g <= 128 && rows < (1LL << 31);
}

// The arena kv[b][page][2][64][256 bytes] as a bf16 matrix [rows][128]; box 64 columns x 64 rows, no swizzle (the rows
// are stored permuted already), nothing is ever read outside it.
PrefillTcState* prefill_tc_create(const CacheView& cv, int is_bf16, int Hq) {
    if (!prefill_tc_supported(cv, is_bf16, Hq)) return nullptr;
    EncodeTiledFnA fn = a_encode_fn();
    if (!fn) return nullptr;
    PrefillTcState* s = new PrefillTcState();
    const cuuint64_t dims[2] = {128, (cuuint64_t)cv.B * (cuuint64_t)cv.P_seq * 2 * PAGE};
    const cuuint64_t strides[1] = {256};
    const cuuint32_t box[2] = {64, (cuuint32_t)A_TILE};
    const cuuint32_t estr[2] = {1, 1};
    const bool ok = fn(&s->map_kv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, cv.kv, dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS &&
                    cudaFuncSetAttribute(prefill_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, A_SMEM) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        delete s;
        return nullptr;
    }
    return s;
}

void prefill_tc_destroy(PrefillTcState* s) { delete s; }

// Rows of a block that carry a query: worth it once at least half of the 256 do.
bool prefill_tc_wanted(const CacheView& cv, int n_new, int Hq) { return (long long)n_new * (Hq / cv.H) >= 128; }

void launch_prefill_attention_tc(const PrefillTcState* s, const CacheView& cv, int layer, int n_new, int Hq, const void* q,
                                 void* out, cudaStream_t st) {
    const int g = Hq / cv.H;
    const int tt = 256 / g;
    dim3 grid((n_new + tt - 1) / tt, cv.B * cv.H);
    prefill_attn_tc_kernel<<<grid, A_THREADS, A_SMEM, st>>>(s->map_kv, cv, layer, n_new, g, Hq, (const __nv_bfloat16*)q,
                                                            (__nv_bfloat16*)out, 1.4426950408889634f / sqrtf((float)cv.d));
    count_launch();
}

}  // namespace tkv
