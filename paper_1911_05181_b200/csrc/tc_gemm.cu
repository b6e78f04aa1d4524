// tcgen05 engine: TF32 tensor-core GEMM for sm_100a with TMEM accumulators, TMA-fed shared-memory ring,
// an on-chip hi/lo operand split for the error-compensated 3xTF32 mode, and the fused epilogues.
//
// One persistent CTA per SM, 14 warps with fixed roles:
//   warp 0      TMA producer      global -> 128B-swizzled shared-memory stages (cp.async.bulk.tensor, no multicast)
//   warp 1      MMA issuer        one thread issues tcgen05.mma.kind::tf32 (128 x BN x 8 per instruction)
//   warps 2-5   epilogue          tcgen05.ld of the 128 x BN fp32 accumulator (one row per thread), fused math, stores
//   warps 6-13  operand pass      only in 3xTF32 mode or when A is formed from logits: reads a landed stage,
//                                 writes hi = tf32(x) in place and lo = tf32(x - hi) beside it
// TMEM holds two 256-column accumulator regions.  A tile's total lives in one of them, so its epilogue overlaps
// the products of the next tile, which uses the other.  The tensor core adds into an fp32 accumulator with
// truncation, a bias that grows with the number of instructions chained on one accumulator; in 3xTF32 mode the
// K loop is therefore cut into chunks of 256: each chunk starts a fresh accumulator in the second region and
// the epilogue warps add it (round-to-nearest) into the tile's total, kept in TMEM.
// 3xTF32: D += lo_a*hi_b; D += hi_a*lo_b; D += hi_a*hi_b (small terms first).
// MN-major fp32 operands use the 128B swizzle with 32-byte atoms (the only one the tensor core transposes
// for 32-bit types); K-major operands the plain 128B swizzle.
// Both operands may be K-major or MN-major in memory (transpose bits of the instruction descriptor), so the
// four forms of Section 3.1 and the three product shapes of Section 4.2 are one kernel.
// Every wait is bounded: on expiry the CTA raises an abort flag, records DEV_TIMEOUT in the device status
// word, drains and frees its TMEM.
#include "common.cuh"
#include <cuda.h>
#include <math.h>
#include <mutex>

namespace ulsnn {

static __device__ int g_dev_status;

namespace {

constexpr int BM = 128;                 // rows of an output tile (TMEM lanes)
constexpr int BN_MAX = 256;             // widest column tile (TMEM columns per accumulator stage)
constexpr int BK = 32;                  // fp32 elements per 128-byte swizzle row
constexpr int UMMA_K = 8;               // K of one tcgen05.mma.kind::tf32
constexpr int NUM_EPI_WARPS = 4;
constexpr int NUM_SPLIT_WARPS = 8;
constexpr int NUM_WARPS = 2 + NUM_EPI_WARPS + NUM_SPLIT_WARPS;
constexpr int NUM_THREADS = NUM_WARPS * 32;
constexpr int MAX_STAGES = 8;
constexpr int A_TILE_BYTES = BM * BK * 4;                       // 16 KB
constexpr int SMEM_BUDGET = 227 * 1024;
constexpr int EPI_SCRATCH_BYTES = NUM_EPI_WARPS * 32 * 33 * 4;   // column-sum staging, one padded 32x32 tile per warp
constexpr int CTRL_BYTES = 1024;                                // barriers, TMEM base, abort flag
constexpr unsigned long long WAIT_LIMIT_CYCLES = 3000000000ull; // ~1.5 s at 2 GHz

struct TcParams {
    GemmDesc d;
    int bn;                 // column-tile width (multiple of 16; multiple of 32 when B is MN-major)
    int tiles_m, tiles_n;
    int units;              // tiles_m * tiles_n * splits
    int stages;
    int b_tile_bytes;       // bn * 128
    int stage_bytes;
    int three_x, a_mn, b_mn, split_pass;
    int chunk_blocks;       // k-blocks accumulated on one TMEM accumulator before it is added into the tile total
    int fast_math;          // TF32 mode: approximate exp
    int64_t n_patterns, n_classes;      // bounds of the logits operand when a_transform
    int* status;
};

// ------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float to_tf32(float x) {
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
    return __uint_as_float(u);
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// exp(x) for x <= ~0 with ~3e-7 relative error: two-constant reduction so that the rounding of x*log2(e) does not
// grow with |x|, one ex2.approx, one correction.
__device__ __forceinline__ float exp_fast_accurate(float x) {
    const float L2E_HI = 1.44269502162933349609375f, L2E_LO = 1.925963033500011e-8f;
    const float th = x * L2E_HI;
    const float tl = fmaf(x, L2E_HI, -th) + x * L2E_LO;
    const float p = ex2_approx(th);
    return fmaf(p, tl * 0.693147180559945f, p);
}
__device__ __forceinline__ float exp_mode(float x, int fast) { return fast ? __expf(x) : exp_fast_accurate(x); }

// Shared-memory matrix descriptor of a swizzled tile (sm_100 format: version 1 at bit 46; layout type at bits
// 61-63: 2 = 128B swizzle of 16-byte units, 1 = 128B swizzle of 32-byte units).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)layout << 61);
}

struct Ctrl {
    uint64_t full[MAX_STAGES];      // TMA bytes landed
    uint64_t ready[MAX_STAGES];     // operand pass done
    uint64_t empty[MAX_STAGES];     // products that read the stage have completed
    uint64_t reg_full[2];           // the products chained on TMEM region r have completed
    uint64_t reg_free[2];           // the epilogue warps have read region r: it may be overwritten
    uint32_t tmem_base;
    volatile int abort;
};

// Bounded wait.  Returns false (after raising the abort flag and the device status) if the phase did not complete.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, Ctrl* ctrl, int* status) {
    const uint32_t b = smem_u32(bar);
    if (mbar_try_wait(b, parity)) return true;
    const unsigned long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try_wait(b, parity)) {
        if ((++spins & 255u) == 0) {
            if (ctrl->abort) return false;
            if ((unsigned long long)clock64() - t0 > WAIT_LIMIT_CYCLES) {
                ctrl->abort = 1;
                atomicExch(status, DEV_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ void unit_coords(const TcParams& p, int u, int& mt, int& nt, int& sp) {
    nt = u % p.tiles_n;
    const int r = u / p.tiles_n;
    mt = r % p.tiles_m;
    sp = r / p.tiles_m;
}

__device__ __forceinline__ void unit_k_range(const TcParams& p, int sp, int64_t& kbeg, int& nkb, int& tail_steps) {
    kbeg = (p.d.epi == EPI_PARTIAL) ? (int64_t)sp * p.d.k_per_split : 0;
    int64_t kend = (p.d.epi == EPI_PARTIAL) ? kbeg + p.d.k_per_split : p.d.K;
    if (kend > p.d.K) kend = p.d.K;
    const int64_t len = kend - kbeg;
    nkb = (int)((len + BK - 1) / BK);
    const int rem = (int)(len - (int64_t)(nkb - 1) * BK);      // 1..32 elements in the last block
    tail_steps = (rem + UMMA_K - 1) / UMMA_K;
}

template <int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: the 128B swizzle pattern repeats every 8 rows of 128 bytes
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_base = smem;
    float* epi_scratch = (float*)(smem + (size_t)p.stages * p.stage_bytes);
    Ctrl* ctrl = (Ctrl*)((uint8_t*)epi_scratch + EPI_SCRATCH_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const GemmDesc& d = p.d;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->ready[s]), NUM_SPLIT_WARPS);
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&ctrl->reg_full[a]), 1);
            mbar_init(smem_u32(&ctrl->reg_free[a]), NUM_EPI_WARPS);
        }
        ctrl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctrl->tmem_base), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;

    // offsets inside a stage
    const int off_a_hi = 0, off_b_hi = A_TILE_BYTES;
    const int off_a_lo = A_TILE_BYTES + p.b_tile_bytes, off_b_lo = 2 * A_TILE_BYTES + p.b_tile_bytes;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            const uint32_t tx_bytes = (uint32_t)(A_TILE_BYTES + p.b_tile_bytes);
            for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
                int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
                int64_t kbeg; int nkb, tail; unit_k_range(p, sp, kbeg, nkb, tail);
                const int m0 = mt * BM, n0 = nt * p.bn;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (it / p.stages) & 1;
                    if (!wait_bar(&ctrl->empty[s], ph ^ 1, ctrl, p.status)) { ok = false; break; }
                    const uint32_t bar = smem_u32(&ctrl->full[s]);
                    mbar_expect_tx(bar, tx_bytes);
                    const uint32_t sa = smem_u32(stage_base + (size_t)s * p.stage_bytes + off_a_hi);
                    const uint32_t sb = smem_u32(stage_base + (size_t)s * p.stage_bytes + off_b_hi);
                    const int k0 = (int)(kbeg + (int64_t)kb * BK);
                    if (!p.a_mn) {
                        tma_load_2d(sa, &map_a, k0, m0, bar);                       // box {32 k, 128 rows}
                    } else {
                        for (int g = 0; g < BM / 32; ++g)                           // boxes {32 m, 32 k}
                            tma_load_2d(sa + g * (BK * 128), &map_a, m0 + 32 * g, k0, bar);
                    }
                    if (!p.b_mn) {
                        tma_load_2d(sb, &map_b, k0, n0, bar);                       // box {32 k, bn rows}
                    } else {
                        for (int g = 0; g < p.bn / 32; ++g)
                            tma_load_2d(sb + g * (BK * 128), &map_b, n0 + 32 * g, k0, bar);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) |
                                   ((uint32_t)(p.bn >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            // K-major (128B swizzle): 8-row groups 1024 B apart (SBO), K advance = 32 B inside the swizzled row.
            // MN-major (128B swizzle, 32-byte atoms): 32-element groups BK*128 B apart (LBO), 4-k groups 512 B apart
            // (SBO), K advance = 8 rows = 1024 B.
            const uint32_t a_lbo = p.a_mn ? BK * 128 : 16, b_lbo = p.b_mn ? BK * 128 : 16;
            const uint32_t a_sbo = p.a_mn ? 512 : 1024, b_sbo = p.b_mn ? 512 : 1024;
            const uint32_t a_lay = p.a_mn ? 1 : 2, b_lay = p.b_mn ? 1 : 2;
            const uint32_t a_kstep = p.a_mn ? 1024 : UMMA_K * 4, b_kstep = p.b_mn ? 1024 : UMMA_K * 4;
            uint32_t it = 0, tile_i = 0;
            uint32_t overwrites[2] = {0, 0};        // how often each TMEM region has been restarted
            bool ok = true;
            for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x, ++tile_i) {
                int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
                int64_t kbeg; int nkb, tail; unit_k_range(p, sp, kbeg, nkb, tail);
                const uint32_t total_reg = tile_i & 1;
                uint32_t reg = total_reg, d_tmem = 0;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const bool chunk_start = (kb % p.chunk_blocks) == 0;
                    if (chunk_start) {
                        // chunk 0 goes to the tile's total region, later chunks restart the other region
                        reg = (kb == 0) ? total_reg : (total_reg ^ 1);
                        if (!wait_bar(&ctrl->reg_free[reg], (overwrites[reg] & 1) ^ 1, ctrl, p.status)) { ok = false; break; }
                        overwrites[reg]++;
                        tc_fence_after();
                        d_tmem = tmem_base + reg * BN_MAX;
                    }
                    const int s = it % p.stages;
                    const uint32_t ph = (it / p.stages) & 1;
                    uint64_t* bar = p.split_pass ? &ctrl->ready[s] : &ctrl->full[s];
                    if (!wait_bar(bar, ph, ctrl, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t base = smem_u32(stage_base + (size_t)s * p.stage_bytes);
                    const int steps = (kb == nkb - 1) ? tail : BK / UMMA_K;
                    for (int ks = 0; ks < steps; ++ks) {
                        const uint64_t a_hi = smem_desc(base + off_a_hi + ks * a_kstep, a_lbo, a_sbo, a_lay);
                        const uint64_t b_hi = smem_desc(base + off_b_hi + ks * b_kstep, b_lbo, b_sbo, b_lay);
                        const uint32_t accumulate = (chunk_start && ks == 0) ? 0u : 1u;
                        if (p.three_x) {
                            const uint64_t a_lo = smem_desc(base + off_a_lo + ks * a_kstep, a_lbo, a_sbo, a_lay);
                            const uint64_t b_lo = smem_desc(base + off_b_lo + ks * b_kstep, b_lbo, b_sbo, b_lay);
                            umma_tf32(d_tmem, a_lo, b_hi, idesc, accumulate);
                            umma_tf32(d_tmem, a_hi, b_lo, idesc, 1u);
                            umma_tf32(d_tmem, a_hi, b_hi, idesc, 1u);
                        } else {
                            umma_tf32(d_tmem, a_hi, b_hi, idesc, accumulate);
                        }
                    }
                    umma_commit(smem_u32(&ctrl->empty[s]));      // frees the stage when these products are done
                    const bool chunk_end = ((kb + 1) % p.chunk_blocks) == 0 || kb == nkb - 1;
                    if (chunk_end) umma_commit(smem_u32(&ctrl->reg_full[reg]));
                }
            }
        }
    } else if (warp < 2 + NUM_EPI_WARPS) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;                         // TMEM lane quarter this warp may read
        const int ew = warp - 2;                        // 0..3, index of this warp among the epilogue warps
        float* tr = epi_scratch + ew * (32 * 33);       // 32x32 staging tile of this warp (padded)
        const bool c_vec = ((((uintptr_t)d.C) & 15) == 0) && ((d.ldc & 3) == 0);
        uint32_t tile_i = 0;
        uint32_t reads[2] = {0, 0};             // how often each TMEM region has been waited for
        bool ok = true;
        for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x, ++tile_i) {
            int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
            int64_t kbeg_; int nkb_, tail_; unit_k_range(p, sp, kbeg_, nkb_, tail_);
            const int n_chunks = (nkb_ + p.chunk_blocks - 1) / p.chunk_blocks;
            const uint32_t acc = tile_i & 1, oth = acc ^ 1;
            if (!wait_bar(&ctrl->reg_full[acc], reads[acc] & 1, ctrl, p.status)) { ok = false; break; }
            reads[acc]++;
            tc_fence_after();
            // chunks after the first were accumulated from zero in the other region: add them into the total
            for (int ch = 1; ch < n_chunks && ok; ++ch) {
                if (!wait_bar(&ctrl->reg_full[oth], reads[oth] & 1, ctrl, p.status)) { ok = false; break; }
                reads[oth]++;
                tc_fence_after();
                const uint32_t lane_off = (uint32_t)(q * 32) << 16;
                for (int c = 0; c < (p.bn + 31) / 32; ++c) {
                    uint32_t x[32], y[32];
                    tmem_ld32(tmem_base + oth * BN_MAX + c * 32 + lane_off, x);
                    tmem_ld32(tmem_base + acc * BN_MAX + c * 32 + lane_off, y);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) y[j] = __float_as_uint(__uint_as_float(y[j]) + __uint_as_float(x[j]));
                    tmem_st32(tmem_base + acc * BN_MAX + c * 32 + lane_off, y);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->reg_free[oth]));
            }
            if (!ok) break;
            const int64_t r = (int64_t)mt * BM + q * 32 + lane;
            const bool rv = r < d.M;
            const int64_t n0 = (int64_t)nt * p.bn;
            const int chunks = (p.bn + 31) / 32;
            float run_m = -INFINITY, run_s = 0.f, zl = 0.f;
            int64_t lab = -1;
            bool have_zl = false;
            if (EPI == EPI_LOGITS && rv) lab = (int64_t)__ldg(d.labels + r);
            for (int c = 0; c < chunks; ++c) {
                uint32_t raw[32];
                tmem_ld32(tmem_base + acc * BN_MAX + c * 32 + ((uint32_t)(q * 32) << 16), raw);
                tmem_ld_wait();
                const int64_t c0 = n0 + c * 32;
                int nvalid = (int)min((int64_t)32, min((int64_t)p.bn - c * 32, d.N - c0));
                if (nvalid < 0) nvalid = 0;
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(raw[j]);

                if (EPI == EPI_SGEMM) {
                    if (rv) {
                        float* dst = d.C + r * d.ldc + c0;
                        if (d.beta != 0.f) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (j < nvalid) v[j] = fmaf(d.beta, dst[j], d.alpha * v[j]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = d.alpha * v[j];
                        }
                        if (c_vec && nvalid == 32) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (j < nvalid) dst[j] = v[j];
                        }
                    }
                } else if (EPI == EPI_PARTIAL) {
                    if (rv) {
                        float* dst = d.partials + ((int64_t)sp * d.M + r) * d.ldp + c0;     // ldp % 4 == 0, base 256-aligned
                        if (nvalid == 32) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (j < nvalid) dst[j] = v[j];
                        }
                    }
                } else if (EPI == EPI_BIAS_TANH) {
                    if (rv) {
                        float* dst = d.C + r * d.ldc + c0;
#pragma unroll
                        for (int j = 0; j < 32; ++j) if (j < nvalid) v[j] = tanhf(v[j] + __ldg(d.bias + c0 + j));
                        if (c_vec && nvalid == 32) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (j < nvalid) dst[j] = v[j];
                        }
                    }
                } else if (EPI == EPI_LOGITS) {
                    float cm = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        v[j] = (j < nvalid) ? v[j] + __ldg(d.bias + c0 + j) : -INFINITY;
                        cm = fmaxf(cm, v[j]);
                    }
                    if (nvalid > 0) {
                        const float nm = fmaxf(run_m, cm);
                        float s = 0.f;
#pragma unroll
                        for (int j = 0; j < 32; ++j) if (j < nvalid) s += exp_mode(v[j] - nm, p.fast_math);
                        run_s = (run_m == -INFINITY ? 0.f : run_s * exp_mode(run_m - nm, p.fast_math)) + s;
                        run_m = nm;
                        if (rv) {
                            if (lab >= c0 && lab < c0 + nvalid) {
#pragma unroll
                                for (int j = 0; j < 32; ++j) if (c0 + j == lab) zl = v[j];
                                have_zl = true;
                            }
                            if (d.C) {
                                float* dst = d.C + r * d.ldc + c0;
                                if (c_vec && nvalid == 32) {
#pragma unroll
                                    for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                                } else {
#pragma unroll
                                    for (int j = 0; j < 32; ++j) if (j < nvalid) dst[j] = v[j];
                                }
                            }
                        }
                    }
                } else if (EPI == EPI_TANHP) {
                    if (rv) {
                        const float* hp = d.Hm + r * d.ldh + c0;
                        float* dst = d.C + r * d.ldc + c0;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (j < nvalid) { const float h = __ldg(hp + j); v[j] = (1.f - h * h) * v[j]; } else v[j] = 0.f;
                        }
                        if (c_vec && nvalid == 32) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (j < nvalid) dst[j] = v[j];
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = 0.f;
                    }
                    if (d.colsum_part) {
                        // column sums of this warp's 32 rows, rows added in index order
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 32; ++j) tr[lane * 33 + j] = v[j];
                        __syncwarp();
                        float s = 0.f;
#pragma unroll
                        for (int i = 0; i < 32; ++i) s += tr[i * 33 + lane];
                        // one partial row per 32-row group (4 per tile); the reduction kernel adds them in index order
                        if (lane < nvalid) d.colsum_part[((int64_t)mt * 4 + q) * d.N + c0 + lane] = s;
                    }
                }
            }
            // all TMEM reads of this accumulator stage are done: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->reg_free[acc]));

            if (EPI == EPI_LOGITS && rv) {
                d.stats[r * d.stats_ld + nt] = make_float2(run_m, run_s);
                if (have_zl) d.zlabel[r] = zl;
            }
            if (EPI == EPI_BIAS_TANH && d.ones_cols > 0 && nt == p.tiles_n - 1 && rv) {
                d.C[r * d.ldc + d.N] = 1.f;
                for (int cc = 1; cc < d.ones_cols; ++cc) d.C[r * d.ldc + d.N + cc] = 0.f;
            }
        }
    } else if (p.split_pass) {
        // ------------------------------------------------------------------ operand pass (hi/lo split, logits -> delta)
        const int st = threadIdx.x - (2 + NUM_EPI_WARPS) * 32;          // 0..255
        constexpr int NT = NUM_SPLIT_WARPS * 32;
        uint32_t it = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
            int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
            int64_t kbeg; int nkb, tail; unit_k_range(p, sp, kbeg, nkb, tail);
            const int64_t m0 = (int64_t)mt * BM;
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % p.stages;
                const uint32_t ph = (it / p.stages) & 1;
                if (!wait_bar(&ctrl->full[s], ph, ctrl, p.status)) { ok = false; break; }
                uint8_t* base = stage_base + (size_t)s * p.stage_bytes;
                const int64_t k0 = kbeg + (int64_t)kb * BK;
                // A tile: 1024 float4
                float4* a_hi = reinterpret_cast<float4*>(base + off_a_hi);
                float4* a_lo = reinterpret_cast<float4*>(base + off_a_lo);
#pragma unroll
                for (int i = 0; i < (BM * BK / 4) / NT; ++i) {
                    const int idx = st + NT * i;
                    float4 x = a_hi[idx];
                    if (d.a_transform) {
                        // un-swizzle the position of this 16-byte chunk to (pattern, class)
                        int64_t pat, cls;
                        if (!p.a_mn) {
                            const int row = idx >> 3, ch = (idx & 7) ^ (row & 7);
                            pat = d.a_pattern_is_m ? m0 + row : k0 + ch * 4;
                            cls = d.a_pattern_is_m ? k0 + ch * 4 : m0 + row;
                            // K-major: the four elements run along K
                            if (d.a_pattern_is_m) {
                                if (pat < p.n_patterns) {
                                    const float l = __ldg(d.lse + pat); const int64_t lb = (int64_t)__ldg(d.labels + pat);
                                    x.x = (cls + 0 < p.n_classes) ? exp_mode(x.x - l, p.fast_math) - (cls + 0 == lb ? 1.f : 0.f) : 0.f;
                                    x.y = (cls + 1 < p.n_classes) ? exp_mode(x.y - l, p.fast_math) - (cls + 1 == lb ? 1.f : 0.f) : 0.f;
                                    x.z = (cls + 2 < p.n_classes) ? exp_mode(x.z - l, p.fast_math) - (cls + 2 == lb ? 1.f : 0.f) : 0.f;
                                    x.w = (cls + 3 < p.n_classes) ? exp_mode(x.w - l, p.fast_math) - (cls + 3 == lb ? 1.f : 0.f) : 0.f;
                                } else x = make_float4(0.f, 0.f, 0.f, 0.f);
                            } else {
                                float e[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                                for (int t = 0; t < 4; ++t) {
                                    const int64_t pp = pat + t;
                                    if (pp < p.n_patterns && cls < p.n_classes)
                                        e[t] = exp_mode(e[t] - __ldg(d.lse + pp), p.fast_math) - (cls == (int64_t)__ldg(d.labels + pp) ? 1.f : 0.f);
                                    else e[t] = 0.f;
                                }
                                x = make_float4(e[0], e[1], e[2], e[3]);
                            }
                        } else {
                            // 32-byte units of a 128-byte row are XORed with (row & 3); a float4 is half a unit
                            const int g = idx >> 8, krow = (idx & 255) >> 3;
                            const int ch = ((((idx & 7) >> 1) ^ (krow & 3)) << 1) | (idx & 1);
                            const int64_t mn = m0 + g * 32 + ch * 4, kk = k0 + krow;
                            // MN-major: the four elements run along M
                            if (d.a_pattern_is_m) {
                                float e[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                                for (int t = 0; t < 4; ++t) {
                                    const int64_t pp = mn + t;
                                    if (pp < p.n_patterns && kk < p.n_classes)
                                        e[t] = exp_mode(e[t] - __ldg(d.lse + pp), p.fast_math) - (kk == (int64_t)__ldg(d.labels + pp) ? 1.f : 0.f);
                                    else e[t] = 0.f;
                                }
                                x = make_float4(e[0], e[1], e[2], e[3]);
                            } else {
                                pat = kk; cls = mn;
                                if (pat < p.n_patterns) {
                                    const float l = __ldg(d.lse + pat); const int64_t lb = (int64_t)__ldg(d.labels + pat);
                                    x.x = (cls + 0 < p.n_classes) ? exp_mode(x.x - l, p.fast_math) - (cls + 0 == lb ? 1.f : 0.f) : 0.f;
                                    x.y = (cls + 1 < p.n_classes) ? exp_mode(x.y - l, p.fast_math) - (cls + 1 == lb ? 1.f : 0.f) : 0.f;
                                    x.z = (cls + 2 < p.n_classes) ? exp_mode(x.z - l, p.fast_math) - (cls + 2 == lb ? 1.f : 0.f) : 0.f;
                                    x.w = (cls + 3 < p.n_classes) ? exp_mode(x.w - l, p.fast_math) - (cls + 3 == lb ? 1.f : 0.f) : 0.f;
                                } else x = make_float4(0.f, 0.f, 0.f, 0.f);
                            }
                        }
                    }
                    const float4 h = make_float4(to_tf32(x.x), to_tf32(x.y), to_tf32(x.z), to_tf32(x.w));
                    a_hi[idx] = h;
                    if (p.three_x) a_lo[idx] = make_float4(to_tf32(x.x - h.x), to_tf32(x.y - h.y), to_tf32(x.z - h.z), to_tf32(x.w - h.w));
                }
                if (p.three_x) {
                    float4* b_hi = reinterpret_cast<float4*>(base + off_b_hi);
                    float4* b_lo = reinterpret_cast<float4*>(base + off_b_lo);
                    const int nvec = p.b_tile_bytes / 16;
                    for (int idx = st; idx < nvec; idx += NT) {
                        const float4 x = b_hi[idx];
                        const float4 h = make_float4(to_tf32(x.x), to_tf32(x.y), to_tf32(x.z), to_tf32(x.w));
                        b_hi[idx] = h;
                        b_lo[idx] = make_float4(to_tf32(x.x - h.x), to_tf32(x.y - h.y), to_tf32(x.z - h.z), to_tf32(x.w - h.w));
                    }
                }
                proxy_fence_async();            // make these generic-proxy writes visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->ready[s]));
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    if (ctrl->abort) {
        // give copies that may still be in flight time to land before the shared memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

// Tensor map of a matrix whose contiguous dimension has `inner` elements and whose other dimension has `outer`
// rows `stride_elems` apart; box = {box_inner (32 floats = one swizzle row), box_outer}.
bool make_map(CUtensorMap* map, const float* base, int64_t inner, int64_t outer, int64_t stride_elems, int box_inner, int box_outer,
              bool atom32) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t gstride[1] = {(cuuint64_t)stride_elems * sizeof(float)};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, (void*)base, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool operand_ok(const float* base, int64_t s_major, int64_t s_minor_is_one_other) {
    (void)s_minor_is_one_other;
    return (((uintptr_t)base) & 15) == 0 && (s_major & 3) == 0 && s_major >= 4 && s_major < ((int64_t)1 << 38);
}

int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    }
    return n;
}

int* status_ptr() {
    static int* ptr = nullptr;
    if (!ptr) { void* p = nullptr; if (cudaGetSymbolAddress(&p, g_dev_status) == cudaSuccess) ptr = (int*)p; }
    return ptr;
}

template <int EPI>
ulsnn_status_t launch(const CUtensorMap& ma, const CUtensorMap& mb, const TcParams& p, int smem_bytes, int grid, cudaStream_t stream) {
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(tc_gemm_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET) != cudaSuccess)
            return ULSNN_ERR_CUDA;
        configured = true;
    }
    tc_gemm_kernel<EPI><<<grid, NUM_THREADS, smem_bytes, stream>>>(ma, mb, p);
    count_launch(1);
    return cuda_ok(cudaGetLastError());
}

}  // namespace

int tc_tile_m() { return BM; }
int tc_colsum_groups() { return 4; }

int tc_tile_n(const GemmDesc& d) {
    const bool b_mn = !(d.b_sk == 1);                     // B(k,j): contiguous along j unless contiguous along k
    const int gran = b_mn ? 32 : 16;
    const int64_t tiles = (d.N + BN_MAX - 1) / BN_MAX;
    int64_t bn = (d.N + tiles - 1) / tiles;
    bn = (bn + gran - 1) / gran * gran;
    if (bn < gran) bn = gran;
    if (bn > BN_MAX) bn = BN_MAX;
    return (int)bn;
}

bool tc_gemm_supported(const GemmDesc& d) {
    if (d.M <= 0 || d.N <= 0 || d.K <= 0) return false;
    if (d.M > 0x7fffffff || d.N > 0x7fffffff || d.K > 0x7fffffff) return false;
    if (!encode_fn()) return false;
    const bool a_k = (d.a_sk == 1), b_k = (d.b_sk == 1);
    if (!a_k && d.a_sm != 1) return false;
    if (!b_k && d.b_sn != 1) return false;
    if (!operand_ok(d.A, a_k ? d.a_sm : d.a_sk, 0)) return false;
    if (!operand_ok(d.B, b_k ? d.b_sn : d.b_sk, 0)) return false;
    return true;
}

ulsnn_status_t tc_gemm_launch(const GemmDesc& d, bool three_x, cudaStream_t stream) {
    if (!tc_gemm_supported(d)) return ULSNN_ERR_INVALID_ARG;
    TcParams p{};
    p.d = d;
    p.a_mn = (d.a_sk == 1) ? 0 : 1;
    p.b_mn = (d.b_sk == 1) ? 0 : 1;
    p.bn = tc_tile_n(d);
    p.tiles_m = (int)((d.M + BM - 1) / BM);
    p.tiles_n = (int)((d.N + p.bn - 1) / p.bn);
    const int splits = (d.epi == EPI_PARTIAL) ? d.splits : 1;
    const int64_t units = (int64_t)p.tiles_m * p.tiles_n * splits;
    if (units > 0x7fffffff) return ULSNN_ERR_TOO_LARGE;
    p.units = (int)units;
    p.three_x = three_x ? 1 : 0;
    p.split_pass = (three_x || d.a_transform) ? 1 : 0;
    p.fast_math = three_x ? 0 : 1;
    p.chunk_blocks = three_x ? 8 : (1 << 30);       // 256 elements of K per accumulator in the accurate mode
    p.b_tile_bytes = p.bn * 128;
    p.stage_bytes = (A_TILE_BYTES + p.b_tile_bytes) * (three_x ? 2 : 1);
    int stages = (SMEM_BUDGET - 1024 - EPI_SCRATCH_BYTES - CTRL_BYTES) / p.stage_bytes;
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    if (stages < 2) return ULSNN_ERR_INVALID_ARG;
    p.stages = stages;
    if (d.a_transform) {
        p.n_patterns = d.a_pattern_is_m ? d.M : d.K;
        p.n_classes = d.a_pattern_is_m ? d.K : d.M;
    }
    p.status = status_ptr();
    if (!p.status) return ULSNN_ERR_CUDA;

    CUtensorMap ma, mb;
    const bool oka = p.a_mn ? make_map(&ma, d.A, d.M, d.K, d.a_sk, 32, 32, true) : make_map(&ma, d.A, d.K, d.M, d.a_sm, 32, BM, false);
    const bool okb = p.b_mn ? make_map(&mb, d.B, d.N, d.K, d.b_sk, 32, 32, true) : make_map(&mb, d.B, d.K, d.N, d.b_sn, 32, p.bn, false);
    if (!oka || !okb) return ULSNN_ERR_CUDA;

    const int smem_bytes = 1024 + stages * p.stage_bytes + EPI_SCRATCH_BYTES + CTRL_BYTES;
    const int grid = p.units < sm_count() ? p.units : sm_count();
    switch (d.epi) {
        case EPI_SGEMM:     return launch<EPI_SGEMM>(ma, mb, p, smem_bytes, grid, stream);
        case EPI_BIAS_TANH: return launch<EPI_BIAS_TANH>(ma, mb, p, smem_bytes, grid, stream);
        case EPI_LOGITS:    return launch<EPI_LOGITS>(ma, mb, p, smem_bytes, grid, stream);
        case EPI_TANHP:     return launch<EPI_TANHP>(ma, mb, p, smem_bytes, grid, stream);
        case EPI_PARTIAL:   return launch<EPI_PARTIAL>(ma, mb, p, smem_bytes, grid, stream);
    }
    return ULSNN_ERR_INVALID_ARG;
}

ulsnn_status_t device_status_fetch_and_clear(cudaStream_t stream, int* word) {
    if (cudaStreamSynchronize(stream) != cudaSuccess) return ULSNN_ERR_CUDA;
    if (cudaMemcpyFromSymbol(word, g_dev_status, sizeof(int)) != cudaSuccess) return ULSNN_ERR_CUDA;
    if (*word != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_dev_status, &zero, sizeof(int)) != cudaSuccess) return ULSNN_ERR_CUDA;
    }
    return ULSNN_OK;
}

}  // namespace ulsnn
