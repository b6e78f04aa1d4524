// tcgen05 engine: TF32 tensor-core GEMM for sm_100a with TMEM accumulators, TMA-fed shared-memory ring,
// the error-compensated 3xTF32 mode (operands as TF32 hi/lo pairs, split on chip or loaded as stored pairs),
// and the fused epilogues.
//
// One persistent CTA per SM, warps with fixed roles (14 warps in the variants with an operand pass, 8 in those without):
//   warp 0 (+ 6, 7) TMA producers global -> swizzled shared-memory stages (cp.async.bulk.tensor, no multicast); in the
//                                 variants without an operand pass warp 0 fetches the A tiles, warp 6 the B tiles and
//                                 warp 7 the lo halves of stored pairs
//   warp 1      product issuer    all lanes run the loop, an elected lane issues tcgen05.mma.kind::tf32 and the
//                                 commits (in the second CTA of a pair: relays "stage ready" to the first)
//   warps 2-5   epilogue          tcgen05.ld of the 128 x BN fp32 accumulator (one row per thread), fused math, then
//                                 32x32 blocks staged in swizzled shared memory and written with TMA stores
//                                 (whole 128-byte lines, edges clipped by the tensor map)
//   warps 6-13  operand pass      (variants with a pass) for operands that do not arrive as stored pairs (3xTF32), or when A is formed
//                                 from logits: reads a landed stage, rewrites it as hi = tf32_rn(x) and writes
//                                 lo = tf32_rn(x - hi) beside it
// Tiles: 128 x BN (BN <= 256) by one CTA, or 256 x BN by the two CTAs of a cluster (tcgen05 cta_group::2): each
// CTA holds its 128 rows of A, half of the B tile and its 128 rows of the accumulator; CTA 0 issues the products.
// CTA 1 signals CTA 0 with asynchronous stores that complete transaction bytes on CTA 0's barriers; CTA 0 answers
// through multicast tcgen05.commit.
// TMEM holds two 256-column accumulator regions.  A tile's total lives in one of them, so its epilogue overlaps
// the products of the next tile, which uses the other.  The tensor core adds into an fp32 accumulator with
// truncation, an error that grows with the number of instructions chained on one accumulator; in 3xTF32 mode the
// K loop is therefore cut into chunks of 256: each chunk starts a fresh accumulator in the second region and
// the epilogue warps add it (round-to-nearest) into the tile's total, kept in TMEM.
// 3xTF32: D += lo_a*hi_b; D += hi_a*lo_b; D += hi_a*hi_b (small terms first).
// MN-major fp32 operands use the 128B swizzle with 32-byte atoms (the only one the tensor core transposes
// for 32-bit types); K-major operands the plain 128B swizzle (64B when BK = 16).
// Both operands may be K-major or MN-major in memory (transpose bits of the instruction descriptor), so the
// four forms of Section 3.1 and the three product shapes of Section 4.2 are one kernel.
// Every wait on an mbarrier is bounded: on expiry the CTA raises an abort flag, records DEV_TIMEOUT in the
// device status word, drains and frees its TMEM.
#include "common.cuh"
#include "tc_ptx.cuh"
#include <cuda.h>
#include <math.h>
#include <string.h>
#include <atomic>
#include <mutex>
#include <type_traits>

namespace ulsnn {

static __device__ int g_dev_status;

namespace {

constexpr int BM = 128;                 // rows of an output tile (TMEM lanes)
constexpr int BN_MAX = 256;             // widest column tile (TMEM columns per accumulator stage)
constexpr int BK = 32;                  // elements of K per pipeline stage (16 or 32): a K-major tile row is BK*4 bytes
constexpr int ROW_BYTES = BK * 4;       // and is swizzled in 64-byte (BK = 16) or 128-byte (BK = 32) mode
constexpr int CPR = ROW_BYTES / 16;     // 16-byte pieces per K-major row
constexpr int UMMA_K = 8;               // K of one tcgen05.mma.kind::tf32
constexpr int NUM_EPI_WARPS = 4;
constexpr int NUM_SPLIT_WARPS = 8;
constexpr int NUM_PRODUCERS = 3;         // warp 0 and the last two warps: a thread gets its next TMA copy accepted only
                                        // some hundred nanoseconds after the previous one, so the copies of a stage
                                        // are spread over three issuing threads
// Variants with an operand pass: warps 0 (producer), 1 (issuer), 2-5 (epilogue), 6-13 (operand pass): 448 threads.
// Variants without: warps 0, 1, 2-5 and the two extra producers 6-7: 256 threads, so the epilogue may use more registers.
constexpr int first_extra_producer(bool multi) { return 2 + NUM_EPI_WARPS + (multi ? 0 : NUM_SPLIT_WARPS); }
constexpr int threads_of(bool multi) { return (first_extra_producer(multi) + (multi ? NUM_PRODUCERS - 1 : 0)) * 32; }
constexpr int MAX_STAGES = 12;
constexpr int NUM_SMS = 148;               // B200; fixes the tile schedule (and with it every summation order)
constexpr int A_TILE_BYTES = BM * BK * 4;
constexpr int SMEM_BUDGET = 227 * 1024;
constexpr int EPI_STAGE_BYTES = 32 * 128;                        // one 32x32 fp32 block, 128B-swizzled
constexpr int EPI_BIAS_BYTES = BN_MAX * 4;                       // a tile's bias values, shared by the epilogue warps
constexpr int EPI_SCRATCH_BYTES = NUM_EPI_WARPS * 2 * EPI_STAGE_BYTES + EPI_BIAS_BYTES;   // two store-staging blocks per epilogue warp + the bias copy
constexpr int CTRL_BYTES = 1024;                                // barriers, TMEM base, abort flag

struct TcParams {
    GemmDesc d;
    int bn;                 // column-tile width, a multiple of 32 (the last tile of a row may use fewer columns)
    int n_gran;             // granularity of the width the tensor core is given for that last tile: 16, or 32 when B is MN-major
    int tiles_m, tiles_n;   // tiles_m counts tiles of 128*CG rows
    int units;              // tiles_m * tiles_n * splits
    int stages;
    int b_tile_bytes;       // bytes of one CTA's B tile: (bn / CG) * BK * 4
    int stage_bytes;
    int three_x, a_mn, b_mn, split_pass;
    int a_pre, b_pre;       // 3xTF32: the operand arrives as a stored (hi, lo) pair, no operand pass for it
    int c_pair;             // BIAS_TANH: the output is written as a (hi, lo) pair
    int chunk_blocks;       // k-blocks accumulated on one TMEM accumulator before it is added into the tile total
    int fast_math;          // TF32 mode: approximate exp
    int c_tma;              // the output (C or the split-K partials) is written with TMA stores
    int producers;          // producer warps that have something to fetch (1, 2 or 3)
    int direct;             // CTA pairs without an operand pass: both CTAs count their landed bytes on CTA 0's `full`
                            // barriers (cta_group::2 loads), nothing is relayed
    int64_t n_patterns, n_classes;      // bounds of the logits operand when a_transform
    unsigned long long wait_limit;      // clock cycles a device-side wait may take before the CTA gives up
    int* status;
};

struct Ctrl {
    uint64_t full[MAX_STAGES];      // TMA bytes landed
    uint64_t ready[MAX_STAGES];     // operand pass done
    uint64_t empty[MAX_STAGES];     // products that read the stage have completed
    uint64_t reg_full[2];           // the products chained on TMEM region r have completed
    uint64_t reg_free[2];           // the epilogue warps have read region r: it may be overwritten
    uint64_t relay_sink[MAX_STAGES];    // CTA 0: landing words of CTA 1's stage-ready signals
    uint64_t free_sink[2][NUM_EPI_WARPS];   // CTA 0: landing words of CTA 1's accumulator-free signals
    uint64_t bias_full, bias_free;  // the tile's bias copy has been written / read by all epilogue warps
    uint32_t tmem_base;
    volatile int abort;
    unsigned long long wait_limit;
};

// Sum over the 32 lanes of a warp of each of 32 per-lane values: lane l ends up with the total of v[l].
// A butterfly of five exchange steps, so the order of the additions is fixed.
__device__ __forceinline__ float warp_transpose_sum(float (&v)[32], int lane) {
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const bool up = lane & 16;
        const float send = up ? v[j] : v[j + 16], keep = up ? v[j + 16] : v[j];
        v[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const bool up = lane & 8;
        const float send = up ? v[j] : v[j + 8], keep = up ? v[j + 8] : v[j];
        v[j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const bool up = lane & 4;
        const float send = up ? v[j] : v[j + 4], keep = up ? v[j + 4] : v[j];
        v[j] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const bool up = lane & 2;
        const float send = up ? v[j] : v[j + 2], keep = up ? v[j + 2] : v[j];
        v[j] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
    }
    {
        const bool up = lane & 1;
        const float send = up ? v[0] : v[1], keep = up ? v[1] : v[0];
        v[0] = keep + __shfl_xor_sync(0xffffffffu, send, 1);
    }
    return v[0];
}

// softmax(z) - onehot from a stored exponential e = exp(z - m) and its chunk's factor exp(m - lse); 0 outside the matrix
__device__ __forceinline__ float delta_of(float e, float scale, int cls, int label, int n_classes) {
    return cls < n_classes ? fmaf(e, scale, cls == label ? -1.f : 0.f) : 0.f;
}

// hi = tf32_rn(x), lo = tf32_rn(x - hi).  (The tensor core ignores the low 13 mantissa bits of a stored word, so the
// landed tile could serve as hi = trunc(x) without being rewritten; but then every lo has the sign of its x, the
// truncation of the accumulator no longer averages out over the lo products, and the measured error of the
// weight gradients was 2.4 times larger.)
__device__ __forceinline__ void split4(const float4 x, float4& hi, float4& lo) {
    hi = make_float4(to_tf32(x.x), to_tf32(x.y), to_tf32(x.z), to_tf32(x.w));
    lo = make_float4(to_tf32(x.x - hi.x), to_tf32(x.y - hi.y), to_tf32(x.z - hi.z), to_tf32(x.w - hi.w));
}

// MULTI: the product has no operand pass; its copies are then issued by three warps and, in a CTA pair, counted on CTA 0's
// barriers.  Products with an operand pass are compiled without any of that (and launched without the two extra warps):
// they ran 1-4 % slower with it in the same kernel.
// THREE_X: the 3xTF32 mode (three products per k step on (hi, lo) pairs, accurate exp) against plain TF32.
template <int EPI, int CG, bool MULTI, bool THREE_X>
__global__ void __launch_bounds__(threads_of(MULTI), 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_a_lo, const __grid_constant__ CUtensorMap map_b_lo,
               const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_c_lo, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: the 128B swizzle pattern repeats every 8 rows of 128 bytes
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_base = smem;
    uint8_t* epi_scratch = smem + (size_t)p.stages * p.stage_bytes;
    Ctrl* ctrl = (Ctrl*)(epi_scratch + EPI_SCRATCH_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const GemmDesc& d = p.d;
    constexpr int FIRST_EXTRA = 2 + NUM_EPI_WARPS + (MULTI ? 0 : NUM_SPLIT_WARPS);      // first of the two extra producer warps
    constexpr bool SPLIT = !MULTI;              // an operand pass runs (warps 6-13)
    constexpr bool DIRECT = MULTI && CG == 2;   // both CTAs of a pair count their landed bytes on CTA 0's `full` barriers
    // With CG == 2 the two CTAs of a cluster work on the same sequence of tiles.  CTA 0 issues the products.  Its
    // `ready` barriers collect its own operand-pass warps and, per stage, 8 transaction bytes that warp 1 of CTA 1
    // sends over with an asynchronous store when CTA 1's stage is ready (an arrival on another CTA's barrier holds
    // its sender up for about a microsecond); its `reg_free` barriers collect its own epilogue warps and 8 bytes
    // from each epilogue warp of CTA 1 in the same way.
    const int rank = (CG == 2) ? (int)cluster_ctarank() : 0;
    const int first_unit = blockIdx.x / CG, unit_step = gridDim.x / CG;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), MULTI ? p.producers : 1);      // one arrival (with its byte count) per producer warp at work
            // CTA 0: its own operand-pass warps plus one arrival relayed from CTA 1; CTA 1: its operand-pass warps
            const int ready_count = (SPLIT ? NUM_SPLIT_WARPS : 0) + ((CG == 2 && rank == 0 && !DIRECT) ? 1 : 0);
            mbar_init(smem_u32(&ctrl->ready[s]), ready_count > 0 ? ready_count : 1);      // unused when nothing arrives on it
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&ctrl->reg_full[a]), 1);
            // CTA 0: its epilogue warps, plus (CG == 2) the issuing warp's own arrival that posts the 8 bytes each of
            // CTA 1's epilogue warps will signal
            mbar_init(smem_u32(&ctrl->reg_free[a]), NUM_EPI_WARPS + (CG == 2 ? 1 : 0));
        }
        mbar_init(smem_u32(&ctrl->bias_full), NUM_EPI_WARPS);
        mbar_init(smem_u32(&ctrl->bias_free), NUM_EPI_WARPS);
        ctrl->abort = 0;
        ctrl->wait_limit = p.wait_limit;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc<CG>(smem_u32(&ctrl->tmem_base), 512);
        tmem_relinquish<CG>();
    }
    tc_fence_before();
    if constexpr (CG == 2) cluster_sync_all(); else __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;

    // offsets inside a stage: the landed A and B tiles, then (3xTF32) their lo parts
    const int off_a_hi = 0, off_b_hi = A_TILE_BYTES;
    const int off_a_lo = A_TILE_BYTES + p.b_tile_bytes, off_b_lo = 2 * A_TILE_BYTES + p.b_tile_bytes;

    if (!MULTI && warp == 0) {
        // ------------------------------------------------------------------ TMA producer (products with an operand pass:
        // one warp fetches everything; the extra polling warps cost such products 3-5 %)
        RingPos rp{0, 0};
        bool ok = true;
        for (int u = first_unit; u < p.units && ok; u += unit_step) {
            int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
            int64_t kbeg; int nkb, tail; unit_k_range<BK, UMMA_K>(p, sp, kbeg, nkb, tail);
            // this CTA's rows of A and its share of the tile's columns of B
            const int b_cols = tile_cols(p, nt) / CG;
            const int m0 = (mt * CG + rank) * BM, n0 = nt * p.bn + rank * b_cols;
            // a K-major B tile is one box of bn/CG rows (rows past the matrix arrive as zeros); an MN-major one is
            // a box per 32 columns, and only the boxes the products read are fetched
            const int b_boxes = b_cols >> 5;
            const uint32_t b_bytes = (uint32_t)(p.b_mn ? b_boxes * (BK * 128) : p.b_tile_bytes);
            const uint32_t tx_bytes = (uint32_t)A_TILE_BYTES * (p.a_pre ? 2u : 1u) + b_bytes * (p.b_pre ? 2u : 1u);
            int k0 = (int)kbeg;
            for (int kb = 0; kb < nkb; ++kb, k0 += BK) {
                const int s = rp.stage;
                if (!wait_bar_warp(&ctrl->empty[s], rp.phase ^ 1, ctrl, p.status)) { ok = false; break; }
                rp.advance(p.stages);
                const uint32_t bar = smem_u32(&ctrl->full[s]);
                const uint32_t sa = smem_u32(stage_base + (size_t)s * p.stage_bytes + off_a_hi);
                const uint32_t sb = sa + off_b_hi;
                if (elect_one()) {
                    mbar_expect_tx(bar, tx_bytes);
                    if (!p.a_mn) {
                        tma_load_2d(sa, &map_a, k0, m0, bar);                       // box {BK k, 128 rows}
                    } else {
#pragma unroll
                        for (int g = 0; g < BM / 32; ++g)                           // boxes {32 m, BK k}
                            tma_load_2d(sa + g * (BK * 128), &map_a, m0 + 32 * g, k0, bar);
                    }
                    if (!p.b_mn) {
                        tma_load_2d(sb, &map_b, k0, n0, bar);                       // box {BK k, bn/CG rows}
                    } else {
#pragma unroll
                        for (int g = 0; g < BN_MAX / 32; ++g)
                            if (g < b_boxes) tma_load_2d(sb + g * (BK * 128), &map_b, n0 + 32 * g, k0, bar);
                    }
                    // operands stored as (hi, lo) pairs: the lo tiles land beside the hi tiles
                    if (p.a_pre) {
                        const uint32_t sal = sa + off_a_lo;
                        if (!p.a_mn) {
                            tma_load_2d(sal, &map_a_lo, k0, m0, bar);
                        } else {
#pragma unroll
                            for (int g = 0; g < BM / 32; ++g) tma_load_2d(sal + g * (BK * 128), &map_a_lo, m0 + 32 * g, k0, bar);
                        }
                    }
                    if (p.b_pre) {
                        const uint32_t sbl = sa + off_b_lo;
                        if (!p.b_mn) {
                            tma_load_2d(sbl, &map_b_lo, k0, n0, bar);
                        } else {
#pragma unroll
                            for (int g = 0; g < BN_MAX / 32; ++g)
                                if (g < b_boxes) tma_load_2d(sbl + g * (BK * 128), &map_b_lo, n0 + 32 * g, k0, bar);
                        }
                    }
                }
                __syncwarp();
            }
        }
    } else if (MULTI && (warp == 0 || warp >= FIRST_EXTRA)) {
        // ------------------------------------------------------------------ TMA producers
        // role 0: the A tiles (and their lo halves when both operands are stored pairs); role 1: the B tiles;
        // role 2: the lo halves of B, or those of A when only A is a stored pair
        const int role = warp == 0 ? 0 : warp - FIRST_EXTRA + 1;
        const bool get_a = role == 0, get_b = role == 1;
        const bool get_a_lo = p.a_pre && (p.b_pre ? role == 0 : role == 2), get_b_lo = p.b_pre && role == 2;
        RingPos rp{0, 0};
        bool ok = get_a || get_b || get_a_lo || get_b_lo;
        for (int u = first_unit; u < p.units && ok; u += unit_step) {
            int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
            int64_t kbeg; int nkb, tail; unit_k_range<BK, UMMA_K>(p, sp, kbeg, nkb, tail);
            // this CTA's rows of A and its share of the tile's columns of B
            const int b_cols = tile_cols(p, nt) / CG;
            const int m0 = (mt * CG + rank) * BM, n0 = nt * p.bn + rank * b_cols;
            // a K-major B tile is one box of bn/CG rows (rows past the matrix arrive as zeros); an MN-major one is
            // a box per 32 columns, and only the boxes the products read are fetched
            const int b_boxes = b_cols >> 5;
            const uint32_t b_bytes = (uint32_t)(p.b_mn ? b_boxes * (BK * 128) : p.b_tile_bytes);
            // what this warp fetches per stage; with direct counting CTA 0 announces the bytes of both CTAs
            const uint32_t tx_bytes = ((get_a ? (uint32_t)A_TILE_BYTES : 0u) + (get_a_lo ? (uint32_t)A_TILE_BYTES : 0u) +
                                       (get_b ? b_bytes : 0u) + (get_b_lo ? b_bytes : 0u)) * (DIRECT ? (uint32_t)CG : 1u);
            int k0 = (int)kbeg;
            for (int kb = 0; kb < nkb; ++kb, k0 += BK) {
                const int s = rp.stage;
                if (!wait_bar_warp(&ctrl->empty[s], rp.phase ^ 1, ctrl, p.status)) { ok = false; break; }
                rp.advance(p.stages);
                const uint32_t bar_local = smem_u32(&ctrl->full[s]);
                const uint32_t bar = (CG == 2 && DIRECT) ? addr_in_rank0(bar_local) : bar_local;
                const uint32_t sa = smem_u32(stage_base + (size_t)s * p.stage_bytes + off_a_hi);
                const uint32_t sb = sa + off_b_hi;
                auto load = [&](uint32_t dst, const CUtensorMap* map, int x, int y) {
                    if (CG == 2 && DIRECT) tma_load_2d_pair(dst, map, x, y, bar); else tma_load_2d(dst, map, x, y, bar);
                };
                auto load_a = [&](uint32_t dst, const CUtensorMap* map) {
                    if (!p.a_mn) {
                        load(dst, map, k0, m0);                                     // box {BK k, 128 rows}
                    } else {
#pragma unroll
                        for (int g = 0; g < BM / 32; ++g) load(dst + g * (BK * 128), map, m0 + 32 * g, k0);    // boxes {32 m, BK k}
                    }
                };
                auto load_b = [&](uint32_t dst, const CUtensorMap* map) {
                    if (!p.b_mn) {
                        load(dst, map, k0, n0);                                     // box {BK k, bn/CG rows}
                    } else {
#pragma unroll
                        for (int g = 0; g < BN_MAX / 32; ++g)
                            if (g < b_boxes) load(dst + g * (BK * 128), map, n0 + 32 * g, k0);
                    }
                };
                if (elect_one()) {
                    if (!DIRECT || rank == 0) mbar_expect_tx(bar_local, tx_bytes);
                    if (get_a) load_a(sa, &map_a);
                    if (get_b) load_b(sb, &map_b);
                    // operands stored as (hi, lo) pairs: the lo tiles land beside the hi tiles
                    if (get_a_lo) load_a(sa + off_a_lo, &map_a_lo);
                    if (get_b_lo) load_b(sa + off_b_lo, &map_b_lo);
                }
                __syncwarp();
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (rank == 0) {
            const uint32_t idesc0 = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) |
                                    ((uint32_t)((BM * CG) >> 4) << 24);
            // K-major (rows of BK*4 bytes, swizzled): 8-row groups 8*BK*4 B apart (SBO), K advance = 32 B inside the row.
            // MN-major (128B swizzle, 32-byte atoms): 32-element groups BK*128 B apart (LBO), 4-k groups 512 B apart
            // (SBO), K advance = 8 rows = 1024 B.
            const uint32_t a_lbo = p.a_mn ? BK * 128 : 16, b_lbo = p.b_mn ? BK * 128 : 16;
            constexpr uint32_t K_SBO = 8 * ROW_BYTES, K_LAY = (BK == 32) ? 2 : 4;      // 8-row groups; 128B or 64B swizzle
            const uint32_t a_sbo = p.a_mn ? 512 : K_SBO, b_sbo = p.b_mn ? 512 : K_SBO;
            const uint32_t a_lay = p.a_mn ? 1 : K_LAY, b_lay = p.b_mn ? 1 : K_LAY;
            const uint32_t a_kstep = p.a_mn ? 1024 : UMMA_K * 4, b_kstep = p.b_mn ? 1024 : UMMA_K * 4;
            // descriptors of the four tiles of stage 0; a stage or a k step only moves the 14-bit start address
            const uint32_t base0 = smem_u32(stage_base);
            const uint64_t da_hi0 = smem_desc(base0 + off_a_hi, a_lbo, a_sbo, a_lay);
            const uint64_t db_hi0 = smem_desc(base0 + off_b_hi, b_lbo, b_sbo, b_lay);
            const uint64_t da_lo0 = smem_desc(base0 + off_a_lo, a_lbo, a_sbo, a_lay);
            const uint64_t db_lo0 = smem_desc(base0 + off_b_lo, b_lbo, b_sbo, b_lay);
            const uint32_t a_kinc = a_kstep >> 4, b_kinc = b_kstep >> 4, stage_inc = (uint32_t)p.stage_bytes >> 4;
            RingPos rp{0, 0};
            uint32_t tile_i = 0;
            uint32_t overwrites[2] = {0, 0};        // how often each TMEM region has been restarted
            bool ok = true;
            for (int u = first_unit; u < p.units && ok; u += unit_step, ++tile_i) {
                int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
                int64_t kbeg; int nkb, tail; unit_k_range<BK, UMMA_K>(p, sp, kbeg, nkb, tail);
                const uint32_t idesc = idesc0 | ((uint32_t)(tile_cols(p, nt) >> 3) << 17);
                const uint32_t total_reg = tile_i & 1;
                uint32_t reg = total_reg, d_tmem = 0;
                int chunk_pos = 0;
                for (int kb = 0; kb < nkb; ++kb) {
                    const bool chunk_start = chunk_pos == 0;
                    if (chunk_start) {
                        // chunk 0 goes to the tile's total region, later chunks restart the other region
                        reg = (kb == 0) ? total_reg : (total_reg ^ 1);
                        if (overwrites[reg] > 0) {          // the region has been used: wait until both CTAs have read it
                            if (CG == 2 && elect_one()) mbar_expect_tx(smem_u32(&ctrl->reg_free[reg]), 8 * NUM_EPI_WARPS);
                            if (!wait_bar_warp(&ctrl->reg_free[reg], (overwrites[reg] - 1) & 1, ctrl, p.status)) { ok = false; break; }
                        }
                        overwrites[reg]++;
                        tc_fence_after();
                        d_tmem = tmem_base + reg * BN_MAX;
                    }
                    const int s = rp.stage;
                    if (!SPLIT && !wait_bar_warp(&ctrl->full[s], rp.phase, ctrl, p.status)) { ok = false; break; }
                    // CTA 1's signal for this stage completes 8 transaction bytes on `ready`; posting the expectation is
                    // this warp's own arrival on it (not needed when CTA 1's bytes are counted on `full` directly)
                    const bool relayed = CG == 2 && !DIRECT;
                    if (relayed && elect_one()) mbar_expect_tx(smem_u32(&ctrl->ready[s]), 8);
                    if ((SPLIT || relayed) && !wait_bar_warp(&ctrl->ready[s], rp.phase, ctrl, p.status)) { ok = false; break; }
                    rp.advance(p.stages);
                    tc_fence_after();
                    const uint32_t soff = (uint32_t)s * stage_inc;
                    const int steps = (kb == nkb - 1) ? tail : BK / UMMA_K;
#pragma unroll
                    for (int ks = 0; ks < BK / UMMA_K; ++ks) {
                        if (ks >= steps) break;
                        const uint64_t a_hi = da_hi0 + (uint64_t)(soff + ks * a_kinc);
                        const uint64_t b_hi = db_hi0 + (uint64_t)(soff + ks * b_kinc);
                        const uint32_t accumulate = (chunk_start && ks == 0) ? 0u : 1u;
                        if (THREE_X) {
                            const uint64_t a_lo = da_lo0 + (uint64_t)(soff + ks * a_kinc);
                            const uint64_t b_lo = db_lo0 + (uint64_t)(soff + ks * b_kinc);
                            umma_tf32<CG>(d_tmem, a_lo, b_hi, idesc, accumulate);
                            umma_tf32<CG>(d_tmem, a_hi, b_lo, idesc, 1u);
                            umma_tf32<CG>(d_tmem, a_hi, b_hi, idesc, 1u);
                        } else {
                            umma_tf32<CG>(d_tmem, a_hi, b_hi, idesc, accumulate);
                        }
                    }
                    umma_commit<CG>(smem_u32(&ctrl->empty[s]));      // frees the stage (in every CTA of the tile) when these products are done
                    ++chunk_pos;
                    if (chunk_pos == p.chunk_blocks || kb == nkb - 1) {
                        umma_commit<CG>(smem_u32(&ctrl->reg_full[reg]));
                        chunk_pos = 0;
                    }
                }
            }
        }
        if (CG == 2 && rank == 1 && !DIRECT) {
            // CTA 1 issues nothing: this warp tells CTA 0 when a stage of CTA 1 is ready for the products
            RingPos rp{0, 0};
            bool ok = true;
            for (int u = first_unit; u < p.units && ok; u += unit_step) {
                int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
                int64_t kbeg; int nkb, tail; unit_k_range<BK, UMMA_K>(p, sp, kbeg, nkb, tail);
                for (int kb = 0; kb < nkb; ++kb) {
                    const int s = rp.stage;
                    uint64_t* bar = SPLIT ? &ctrl->ready[s] : &ctrl->full[s];
                    if (!wait_bar_warp(bar, rp.phase, ctrl, p.status)) { ok = false; break; }
                    rp.advance(p.stages);
                    if (lane == 0) signal_rank0(smem_u32(&ctrl->relay_sink[s]), smem_u32(&ctrl->ready[s]));
                    __syncwarp();
                }
            }
        }
    } else if (warp < 2 + NUM_EPI_WARPS) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;                         // TMEM lane quarter this warp may read
        const int ew = warp - 2;                        // 0..3, index of this warp among the epilogue warps
        uint8_t* stg = epi_scratch + ew * (2 * EPI_STAGE_BYTES);     // two 32x32 store-staging blocks of this warp
        // The tile's bias values, one copy for the four epilogue warps (each writes a quarter): fetched from global
        // memory block by block they cost a third of a block's time, and shared memory has 1 KB to spare, not 4.
        float* bias_s = reinterpret_cast<float*>(epi_scratch + NUM_EPI_WARPS * (2 * EPI_STAGE_BYTES));
        constexpr bool HAS_BIAS = EPI == EPI_BIAS_TANH || EPI == EPI_LOGITS || EPI == EPI_TANH_SSE;
        const uint32_t lane_off = (uint32_t)(q * 32) << 16;
        const bool c_vec = ((((uintptr_t)d.C) & 15) == 0) && ((d.ldc & 3) == 0);
        const bool t_vec = (EPI == EPI_TANH_SSE) && ((((uintptr_t)d.T) & 15) == 0) && ((d.ldt & 3) == 0);
        const bool h_vec = (EPI == EPI_TANHP) && ((((uintptr_t)d.Hm) & 15) == 0) && ((((uintptr_t)d.Hm_lo) & 15) == 0) && ((d.ldh & 3) == 0);
        uint32_t tile_i = 0, stg_i = 0;
        uint32_t reads[2] = {0, 0};             // how often each TMEM region has been waited for
        bool ok = true;
        for (int u = first_unit; u < p.units && ok; u += unit_step, ++tile_i) {
            int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
            int64_t kbeg_; int nkb_, tail_; unit_k_range<BK, UMMA_K>(p, sp, kbeg_, nkb_, tail_);
            const int n_chunks = (nkb_ + p.chunk_blocks - 1) / p.chunk_blocks;
            const uint32_t acc = tile_i & 1, oth = acc ^ 1;
            const int n0 = nt * p.bn;
            const int chunks = (min(p.bn, (int)d.N - n0) + 31) >> 5;       // 32-column blocks of this tile inside the matrix
            if (HAS_BIAS) {
                // before the wait for the tile's products, so that the loads hide behind them; the copy may be
                // overwritten once every epilogue warp is through with the previous tile
                if (tile_i > 0 && !wait_bar(&ctrl->bias_free, (tile_i - 1) & 1, ctrl, p.status)) { ok = false; break; }
                constexpr int PER_WARP = BN_MAX / NUM_EPI_WARPS;        // 64 values per warp
#pragma unroll
                for (int j = 0; j < PER_WARP / 32; ++j) {
                    const int idx = ew * PER_WARP + j * 32 + lane;
                    bias_s[idx] = n0 + idx < (int)d.N ? __ldg(d.bias + n0 + idx) : 0.f;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->bias_full));
            }
            if (!wait_bar(&ctrl->reg_full[acc], reads[acc] & 1, ctrl, p.status)) { ok = false; break; }
            reads[acc]++;
            tc_fence_after();
            // chunks after the first were accumulated from zero in the other region: add them into the total
            for (int ch = 1; ch < n_chunks && ok; ++ch) {
                if (!wait_bar(&ctrl->reg_full[oth], reads[oth] & 1, ctrl, p.status)) { ok = false; break; }
                reads[oth]++;
                tc_fence_after();
                for (int c = 0; c < chunks; ++c) {
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
                if (lane == 0) { if (CG == 2 && rank == 1) signal_rank0(smem_u32(&ctrl->free_sink[oth][ew]), smem_u32(&ctrl->reg_free[oth])); else mbar_arrive(smem_u32(&ctrl->reg_free[oth])); }
            }
            if (!ok) break;
            if (HAS_BIAS && !wait_bar(&ctrl->bias_full, tile_i & 1, ctrl, p.status)) { ok = false; break; }
            const int r0w = (mt * CG + rank) * BM + q * 32;   // first row of this warp's 32-row block
            const int64_t r = (int64_t)r0w + lane;
            const bool rv = r < d.M;
            float run_m = -INFINITY, run_s = 0.f, zl = 0.f;
            float tile_max[BN_MAX / 32];            // LOGITS: the maximum each chunk's stored exponentials refer to
#pragma unroll
            for (int c = 0; c < BN_MAX / 32; ++c) tile_max[c] = 0.f;
            int lab = -1;
            bool have_zl = false;
            if (EPI == EPI_LOGITS && rv) lab = __ldg(d.labels + r);
            for (int c = 0; c < chunks; ++c) {
                const int c0 = n0 + c * 32;
                const int nvalid = min(32, (int)d.N - c0);      // < 32 only in the last block of a row of the matrix
                const bool full = nvalid == 32;
                uint32_t raw[32];
                tmem_ld32(tmem_base + acc * BN_MAX + c * 32 + lane_off, raw);
                tmem_ld_wait();
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(raw[j]);
                bool do_store = true;

                if (EPI == EPI_SGEMM) {
                    if (d.beta != 0.f) {
                        if (rv) {
                            const float* src = d.C + r * d.ldc + c0;
                            if (c_vec && full) {
#pragma unroll
                                for (int j = 0; j < 32; j += 4) {
                                    const float4 o = *reinterpret_cast<const float4*>(src + j);
                                    v[j] = fmaf(d.beta, o.x, d.alpha * v[j]); v[j + 1] = fmaf(d.beta, o.y, d.alpha * v[j + 1]);
                                    v[j + 2] = fmaf(d.beta, o.z, d.alpha * v[j + 2]); v[j + 3] = fmaf(d.beta, o.w, d.alpha * v[j + 3]);
                                }
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j) if (j < nvalid) v[j] = fmaf(d.beta, src[j], d.alpha * v[j]);
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = d.alpha * v[j];
                    }
                } else if (EPI == EPI_BIAS_TANH || EPI == EPI_LOGITS || EPI == EPI_TANH_SSE) {
                    {
                        const float4* bs = reinterpret_cast<const float4*>(bias_s + c * 32);      // every lane reads the same words
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 bb = bs[j >> 2];
                            v[j] += bb.x; v[j + 1] += bb.y; v[j + 2] += bb.z; v[j + 3] += bb.w;
                        }
                    }
                    if (EPI == EPI_BIAS_TANH) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = tanhf(v[j]);
                    } else if (EPI == EPI_TANH_SSE) {
                        // Eqs. 1 and 3: y = tanh(z), E += (y - t)^2, stored value dE/dz = 2 (y - t)(1 - y^2)
                        float t[32];
                        if (rv) {
                            const float* tp = d.T + r * d.ldt + c0;
                            if (t_vec && full) {
#pragma unroll
                                for (int j = 0; j < 32; j += 4) {
                                    const float4 q4 = __ldg(reinterpret_cast<const float4*>(tp + j));
                                    t[j] = q4.x; t[j + 1] = q4.y; t[j + 2] = q4.z; t[j + 3] = q4.w;
                                }
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j) t[j] = (j < nvalid) ? __ldg(tp + j) : 0.f;
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) t[j] = 0.f;
                        }
                        float s = 0.f;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float y = tanhf(v[j]);
                            const float e = (j < nvalid) ? y - t[j] : 0.f;
                            s += e * e;
                            v[j] = 2.f * e * (1.f - y * y);
                        }
                        run_s += s;
                        do_store = d.C != nullptr;
                    } else {
                        float cm = -INFINITY;
#pragma unroll
                        for (int j = 0; j < 32; ++j) { if (j >= nvalid) v[j] = -INFINITY; cm = fmaxf(cm, v[j]); }
                        const float nm = fmaxf(run_m, cm);
                        if ((unsigned)(lab - c0) < (unsigned)nvalid) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (c0 + j == lab) zl = v[j];
                            have_zl = true;
                        }
                        // the exponentials that make up the row sum are also what is stored: exp(z - nm), with nm
                        // noted per chunk, so that the delta products get softmax(z) by one multiplication
                        float s = 0.f;
                        auto sum_exp = [&](auto fast_tag) {
                            constexpr bool FAST = decltype(fast_tag)::value;
                            if (full) {
#pragma unroll
                                for (int j = 0; j < 32; ++j) { v[j] = exp_t<FAST>(v[j] - nm); s += v[j]; }
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j) { v[j] = (j < nvalid) ? exp_t<FAST>(v[j] - nm) : 0.f; s += v[j]; }
                            }
                            run_s = (run_m == -INFINITY ? 0.f : run_s * exp_t<FAST>(run_m - nm)) + s;
                        };
                        sum_exp(std::integral_constant<bool, !THREE_X>{});
                        run_m = nm;
#pragma unroll
                        for (int q8 = 0; q8 < BN_MAX / 32; ++q8) if (q8 == c) tile_max[q8] = nm;      // static indices: stays in registers
                        do_store = d.C != nullptr;
                    }
                } else if (EPI == EPI_TANHP) {
                    if (rv) {
                        const float* hp = d.Hm + r * d.ldh + c0;
                        const float* hl = d.Hm_lo ? d.Hm_lo + r * d.ldh + c0 : nullptr;
                        if (h_vec && full) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4) {
                                float4 h = __ldg(reinterpret_cast<const float4*>(hp + j));
                                if (hl) { const float4 l = __ldg(reinterpret_cast<const float4*>(hl + j)); h.x += l.x; h.y += l.y; h.z += l.z; h.w += l.w; }
                                v[j] *= (1.f - h.x * h.x); v[j + 1] *= (1.f - h.y * h.y);
                                v[j + 2] *= (1.f - h.z * h.z); v[j + 3] *= (1.f - h.w * h.w);
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                if (j < nvalid) { const float h = __ldg(hp + j) + (hl ? __ldg(hl + j) : 0.f); v[j] = (1.f - h * h) * v[j]; } else v[j] = 0.f;
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = 0.f;
                    }
                }

                // ---- store the 32x32 block (through a swizzled staging block and a TMA store, or directly)
                auto store_block = [&](const float (&w)[32], const CUtensorMap* map, float* direct_base, int64_t ld) {
                    if (p.c_tma) {
                        uint8_t* blk = stg + (stg_i & 1) * EPI_STAGE_BYTES;
                        ++stg_i;
                        if (lane == 0) bulk_wait_read_1();      // the store issued from this block two blocks ago has been read
                        __syncwarp();
                        // row `lane` of the block, 16-byte pieces XOR-swizzled with the row (128B swizzle)
                        float4* rowp = reinterpret_cast<float4*>(blk + lane * 128);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            rowp[j ^ (lane & 7)] = make_float4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                        proxy_fence_async();
                        __syncwarp();
                        if (lane == 0 && r0w < d.M) {
                            tma_store_3d(map, smem_u32(blk), c0, r0w, EPI == EPI_PARTIAL ? sp : 0);
                            bulk_commit();
                        }
                    } else {
                        // rows that TMA cannot address (a leading dimension that is not a multiple of four, a base that is
                        // not 16-byte aligned): the block goes through the same staging block, and the warp then writes
                        // it row by row, one 128-byte run per instruction
                        uint8_t* blk = stg + (stg_i & 1) * EPI_STAGE_BYTES;
                        ++stg_i;
                        __syncwarp();
                        float4* rowp = reinterpret_cast<float4*>(blk + lane * 128);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            rowp[j ^ (lane & 7)] = make_float4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                        __syncwarp();
                        const int rows_here = min(32, (int)(d.M - r0w));
                        if (lane < nvalid) {
                            float* dst = direct_base + (int64_t)r0w * ld + c0 + lane;
                            for (int rr = 0; rr < rows_here; ++rr) {
                                const float* src = reinterpret_cast<const float*>(blk + rr * 128 + ((((lane >> 2) ^ (rr & 7)) << 4) | ((lane & 3) << 2)));
                                dst[(int64_t)rr * ld] = *src;
                            }
                        }
                    }
                };
                if (do_store) {
                    if (EPI == EPI_PARTIAL) {
                        store_block(v, &map_c, d.partials + (int64_t)sp * d.M * d.ldp, d.ldp);
                    } else if ((EPI == EPI_BIAS_TANH || EPI == EPI_TANH_SSE) && p.c_pair) {
                        float lo[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) { const float h = to_tf32(v[j]); lo[j] = to_tf32(v[j] - h); v[j] = h; }
                        store_block(v, &map_c, d.C, d.ldc);
                        store_block(lo, &map_c_lo, d.C_lo, d.ldc);
                    } else {
                        store_block(v, &map_c, d.C, d.ldc);
                    }
                }
                if (EPI == EPI_TANHP && d.colsum_part) {
                    // column sums of this warp's 32 rows: one partial row per 32-row group (4 per tile); the
                    // reduction kernel adds the groups in index order
#pragma unroll
                    for (int j = 0; j < 32; ++j) if (j >= nvalid) v[j] = 0.f;
                    const float s = warp_transpose_sum(v, lane);
                    if (lane < nvalid) d.colsum_part[((int64_t)(mt * CG + rank) * 4 + q) * d.N + c0 + lane] = s;
                }
            }
            // all TMEM reads of this accumulator stage are done: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (HAS_BIAS && lane == 0) mbar_arrive(smem_u32(&ctrl->bias_free));
            if (lane == 0) { if (CG == 2 && rank == 1) signal_rank0(smem_u32(&ctrl->free_sink[acc][ew]), smem_u32(&ctrl->reg_free[acc])); else mbar_arrive(smem_u32(&ctrl->reg_free[acc])); }

            if (EPI == EPI_TANH_SSE && rv) d.stats[r * d.stats_ld + nt] = make_float2(0.f, run_s);
            if (EPI == EPI_LOGITS && rv && d.chunk_max) {
                // the tile's chunk maxima in one go: the table's rows are padded to whole tiles
                float4* dst = reinterpret_cast<float4*>(d.chunk_max + r * d.chunk_ld + (n0 >> 5));
                dst[0] = make_float4(tile_max[0], tile_max[1], tile_max[2], tile_max[3]);
                dst[1] = make_float4(tile_max[4], tile_max[5], tile_max[6], tile_max[7]);
            }
            if (EPI == EPI_LOGITS && rv) {
                d.stats[r * d.stats_ld + nt] = make_float2(run_m, run_s);
                if (have_zl) d.zlabel[r] = zl;
            }
            if (EPI == EPI_BIAS_TANH && d.ones_cols > 0 && nt == p.tiles_n - 1 && rv) {
                d.C[r * d.ldc + d.N] = 1.f;
                for (int cc = 1; cc < d.ones_cols; ++cc) d.C[r * d.ldc + d.N + cc] = 0.f;
                if (p.c_pair) for (int cc = 0; cc < d.ones_cols; ++cc) d.C_lo[r * d.ldc + d.N + cc] = 0.f;
            }
        }
        if (lane == 0) bulk_wait_all();         // every store of this warp has left shared memory and is complete
    } else if (SPLIT) {
        // ------------------------------------------------------------------ operand pass (lo parts, logits -> delta)
        const int st = threadIdx.x - (2 + NUM_EPI_WARPS) * 32;          // 0..255
        constexpr int NT = NUM_SPLIT_WARPS * 32;
        // Position of this thread's 16-byte pieces in the A tile (piece index st + 256*i, i = 0..3).
        //  K-major: row (st>>3) + 32*i of the tile, the four floats run along K from k0 + 4*kch
        //  MN-major: k row st>>3, the four floats run along M from m0 + 32*i + 4*mch
        // K-major tile: piece idx = st + NT*i sits in row idx / CPR at position idx % CPR, which holds logical piece
        // position ^ (row & 7) (128-byte rows) or position ^ ((row >> 1) & 3) (64-byte rows)
        constexpr int ROW_STEP = NT / CPR;                      // rows between a thread's consecutive pieces
        const int a_row = st / CPR;
        const int kch = (st % CPR) ^ (BK == 32 ? (a_row & 7) : ((a_row >> 1) & 3));
        // MN-major tile: 32-column groups of BK k rows of 128 bytes; piece idx sits in group idx / (BK*8), k row
        // (idx % (BK*8)) / 8; 32-byte units of a row are XORed with (k row & 3)
        constexpr int G_PIECES = BK * 8;                        // pieces per 32-column group
        const int mn_g0 = st / G_PIECES, mn_gstep = NT / G_PIECES;          // group of piece i: mn_g0 + mn_gstep*i
        const int mn_krow = (st % G_PIECES) >> 3;
        const int mch = ((((st & 7) >> 1) ^ (mn_krow & 3)) << 1) | (st & 1);
        const int n_classes = (int)p.n_classes, n_patterns = (int)p.n_patterns;
        RingPos rp{0, 0};
        bool ok = true;
        for (int u = first_unit; u < p.units && ok; u += unit_step) {
            int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
            int64_t kbeg; int nkb, tail; unit_k_range<BK, UMMA_K>(p, sp, kbeg, nkb, tail);
            const int m0 = (mt * CG + rank) * BM;
            const int b_cols = tile_cols(p, nt) / CG;
            // K-major logits (the pattern is the row): statistics of this thread's rows, once per tile
            constexpr int NA = (BM * BK / 4) / NT;          // 16-byte pieces of the A tile per thread
            int row_lab[NA];
#pragma unroll
            for (int i = 0; i < NA; ++i) row_lab[i] = -1;
            if (d.a_transform && !p.a_mn) {
#pragma unroll
                for (int i = 0; i < NA; ++i) {
                    const int pat = m0 + a_row + ROW_STEP * i;
                    if (pat < n_patterns) row_lab[i] = __ldg(d.labels + pat);
                }
            }
            int k0 = (int)kbeg;
            for (int kb = 0; kb < nkb; ++kb, k0 += BK) {
                const int s = rp.stage;
                // MN-major logits (the pattern is the k row): statistics of this thread's pattern in this block
                int k_lab = -1;
                const int kpat = k0 + mn_krow;
                // factors of the 32-class chunks this thread's pieces lie in (fetched before the wait for the stage):
                // K-major: the stage is one chunk (k0 is a multiple of 32) of each of the thread's rows;
                // MN-major: the thread's pattern is fixed and its pieces lie in consecutive chunks
                float pc_scale[NA];
#pragma unroll
                for (int i = 0; i < NA; ++i) pc_scale[i] = 0.f;
                if (d.a_transform) {
                    if (!p.a_mn) {
#pragma unroll
                        for (int i = 0; i < NA; ++i) {
                            const int pat = m0 + a_row + ROW_STEP * i;
                            if (pat < n_patterns && k0 < n_classes) pc_scale[i] = __ldg(d.scale + (int64_t)pat * d.scale_ld + (k0 >> 5));
                        }
                    } else if (kpat < n_patterns) {
                        k_lab = __ldg(d.labels + kpat);
#pragma unroll
                        for (int i = 0; i < NA; ++i) {
                            const int cls0 = m0 + 32 * (mn_g0 + mn_gstep * i);
                            if (cls0 < n_classes) pc_scale[i] = __ldg(d.scale + (int64_t)kpat * d.scale_ld + (cls0 >> 5));
                        }
                    }
                }
                if (!wait_bar(&ctrl->full[s], rp.phase, ctrl, p.status)) { ok = false; break; }
                rp.advance(p.stages);
                uint8_t* base = stage_base + (size_t)s * p.stage_bytes;
                float4* a_hi = reinterpret_cast<float4*>(base + off_a_hi);
                float4* a_lo = reinterpret_cast<float4*>(base + off_a_lo);
                float4* b_hi = reinterpret_cast<float4*>(base + off_b_hi);
                float4* b_lo = reinterpret_cast<float4*>(base + off_b_lo);
                // The body is instantiated per mode so that its unrolled loops are straight-line code.
                auto pass = [&](auto three_tag) {
                    constexpr bool THREE = decltype(three_tag)::value;
                    if (!p.a_pre) {
                    float4 x[NA];
#pragma unroll
                    for (int i = 0; i < NA; ++i) x[i] = a_hi[st + NT * i];
                    if (d.a_transform) {
                        if (!p.a_mn) {
                            const int cls = k0 + kch * 4;
#pragma unroll
                            for (int i = 0; i < NA; ++i) {
                                const bool live = m0 + a_row + ROW_STEP * i < n_patterns;
                                x[i].x = live ? delta_of(x[i].x, pc_scale[i], cls + 0, row_lab[i], n_classes) : 0.f;
                                x[i].y = live ? delta_of(x[i].y, pc_scale[i], cls + 1, row_lab[i], n_classes) : 0.f;
                                x[i].z = live ? delta_of(x[i].z, pc_scale[i], cls + 2, row_lab[i], n_classes) : 0.f;
                                x[i].w = live ? delta_of(x[i].w, pc_scale[i], cls + 3, row_lab[i], n_classes) : 0.f;
                            }
                        } else {
                            const bool live = kpat < n_patterns;
#pragma unroll
                            for (int i = 0; i < NA; ++i) {
                                const int cls = m0 + 32 * (mn_g0 + mn_gstep * i) + mch * 4;
                                x[i].x = live ? delta_of(x[i].x, pc_scale[i], cls + 0, k_lab, n_classes) : 0.f;
                                x[i].y = live ? delta_of(x[i].y, pc_scale[i], cls + 1, k_lab, n_classes) : 0.f;
                                x[i].z = live ? delta_of(x[i].z, pc_scale[i], cls + 2, k_lab, n_classes) : 0.f;
                                x[i].w = live ? delta_of(x[i].w, pc_scale[i], cls + 3, k_lab, n_classes) : 0.f;
                            }
                        }
                    }
#pragma unroll
                    for (int i = 0; i < NA; ++i) {
                        if constexpr (THREE) {
                            float4 h, l; split4(x[i], h, l);
                            a_hi[st + NT * i] = h; a_lo[st + NT * i] = l;
                        } else {
                            a_hi[st + NT * i] = x[i];       // only reached when A was transformed
                        }
                    }
                    }
                    if (THREE && !p.b_pre) {
                        const int nvec = b_cols * CPR;               // BK*4 bytes per column of the tile
#pragma unroll 4
                        for (int idx = st; idx < nvec; idx += NT) {
                            float4 h, l; split4(b_hi[idx], h, l);
                            b_hi[idx] = h; b_lo[idx] = l;
                        }
                    }
                };
                pass(std::integral_constant<bool, THREE_X>{});
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
    __syncwarp();
    tc_fence_before();
    // nobody leaves while the other CTA of the tile may still signal a barrier here or read this CTA's operands
    if constexpr (CG == 2) cluster_sync_all(); else __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<CG>(tmem_base, 512);
    }
}

// One CTA, one warp: allocates tensor memory as the product kernels do, then waits (bounded) on a barrier that
// nothing arrives on.  The wait gives up after `limit` cycles, records DEV_TIMEOUT, and the CTA leaves the way the
// product kernels leave after an abort: tensor memory freed, nothing pending.
__global__ void __launch_bounds__(32, 1) wait_probe_kernel(int* status, unsigned long long limit) {
    __shared__ Ctrl ctrl_s;
    Ctrl* ctrl = &ctrl_s;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&ctrl->full[0]), 1);
        ctrl->abort = 0;
        ctrl->wait_limit = limit;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    tmem_alloc<1>(smem_u32(&ctrl->tmem_base), 32);
    tmem_relinquish<1>();
    tc_fence_before();
    __syncwarp();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    (void)wait_bar_warp(&ctrl->full[0], 0, ctrl, status);      // phase 0 never completes
    __syncwarp();
    tc_fence_before();
    tmem_dealloc<1>(tmem_base, 32);
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
// rows `stride_elems` apart; box = {box_inner, box_outer}.
bool make_map(CUtensorMap* map, const float* base, int64_t inner, int64_t outer, int64_t stride_elems, int box_inner, int box_outer,
              bool atom32) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t gstride[1] = {(cuuint64_t)stride_elems * sizeof(float)};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, (void*)base, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : (BK == 32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B),
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of an output written with TMA stores: `slices` matrices of `rows` x `cols` floats, rows `ld` floats
// apart, one after the other; box = one 32 x 32 block (128-byte rows, 128B swizzle).  Stores are clipped at the
// edges of the matrix (rows exactly, columns at the next multiple of four).
bool make_store_map(CUtensorMap* map, const float* base, int64_t cols, int64_t rows, int64_t ld, int64_t slices) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)slices};
    cuuint64_t gstride[2] = {(cuuint64_t)ld * sizeof(float), (cuuint64_t)rows * (cuuint64_t)ld * sizeof(float)};
    cuuint32_t box[3] = {32, 32, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, (void*)base, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool operand_ok(const float* base, int64_t s_major, int64_t s_minor_is_one_other) {
    (void)s_minor_is_one_other;
    return (((uintptr_t)base) & 15) == 0 && (s_major & 3) == 0 && s_major >= 4 && s_major < ((int64_t)1 << 38);
}

int sm_count() { return sm_count_of_current_device(NUM_SMS); }

int* status_ptr() {
    static std::atomic<int*> cached[MAX_DEVICE_SLOTS];
    const int slot = current_device_slot();
    if (slot < 0) return nullptr;
    int* ptr = cached[slot].load(std::memory_order_acquire);
    if (!ptr) {
        void* q = nullptr;
        if (cudaGetSymbolAddress(&q, g_dev_status) != cudaSuccess) return nullptr;
        ptr = (int*)q;
        cached[slot].store(ptr, std::memory_order_release);
    }
    return ptr;
}

struct Maps { CUtensorMap a, b, a_lo, b_lo, c, c_lo; };

template <int EPI, int CG, bool MULTI, bool THREE_X>
ulsnn_status_t launch(const Maps& m, const TcParams& p, int smem_bytes, int grid, cudaStream_t stream) {
    static std::atomic<uint64_t> configured{0};
    if (!allow_dynamic_smem(tc_gemm_kernel<EPI, CG, MULTI, THREE_X>, SMEM_BUDGET, configured)) return ULSNN_ERR_CUDA;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(threads_of(MULTI), 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, tc_gemm_kernel<EPI, CG, MULTI, THREE_X>, m.a, m.b, m.a_lo, m.b_lo, m.c, m.c_lo, p);
    count_launch(1);
    return cuda_ok(e == cudaSuccess ? cudaGetLastError() : e);
}

template <int EPI, bool MULTI, bool THREE_X>
ulsnn_status_t launch_cg2(int cg, const Maps& m, const TcParams& p, int smem_bytes, int grid, cudaStream_t stream) {
    return cg == 2 ? launch<EPI, 2, MULTI, THREE_X>(m, p, smem_bytes, grid, stream) : launch<EPI, 1, MULTI, THREE_X>(m, p, smem_bytes, grid, stream);
}

template <int EPI>
ulsnn_status_t launch_cg(int cg, const Maps& m, const TcParams& p, int smem_bytes, int grid, cudaStream_t stream) {
    if (p.split_pass)
        return p.three_x ? launch_cg2<EPI, false, true>(cg, m, p, smem_bytes, grid, stream) : launch_cg2<EPI, false, false>(cg, m, p, smem_bytes, grid, stream);
    return p.three_x ? launch_cg2<EPI, true, true>(cg, m, p, smem_bytes, grid, stream) : launch_cg2<EPI, true, false>(cg, m, p, smem_bytes, grid, stream);
}

}  // namespace

// Products with more than one 128-row tile are computed by pairs of CTAs (256-row tiles, tcgen05 cta_group::2):
// per product instruction each SM then reads half as much of B from its shared memory.
int tc_cta_group(const GemmDesc& d) { return d.M > BM ? 2 : 1; }
int tc_tile_m(const GemmDesc& d) { return BM * tc_cta_group(d); }
int tc_slots(const GemmDesc& d) { return NUM_SMS / tc_cta_group(d); }
int tc_colsum_groups() { return 4; }

int tc_tile_n(const GemmDesc& d) {
    // 32-column blocks are the unit of the epilogue's stores (64 where two CTAs each fetch 32-column boxes of an
    // MN-major B); tiles are as wide as TMEM allows and the last one of a row is given to the tensor core at its
    // own, smaller width
    const bool b_mn = !(d.b_sk == 1);
    const int64_t g = (b_mn && tc_cta_group(d) == 2) ? 64 : 32;
    int64_t bn = (d.N + g - 1) / g * g;
    if (bn > BN_MAX) bn = BN_MAX;
    return (int)bn;
}

bool tc_operand_addressable(const float* base, int64_t ld) { return encode_fn() != nullptr && operand_ok(base, ld, 0); }

bool tc_gemm_supported(const GemmDesc& d) {
    if (d.M <= 0 || d.N <= 0 || d.K <= 0) return false;
    if (d.M > 0x7fffffff || d.N > 0x7fffffff || d.K > 0x7fffffff) return false;
    if (!encode_fn()) return false;
    const bool a_k = (d.a_sk == 1), b_k = (d.b_sk == 1);
    if (!a_k && d.a_sm != 1) return false;
    if (!b_k && d.b_sn != 1) return false;
    if (!operand_ok(d.A, a_k ? d.a_sm : d.a_sk, 0)) return false;
    if (!operand_ok(d.B, b_k ? d.b_sn : d.b_sk, 0)) return false;
    if (d.A_lo && (((uintptr_t)d.A_lo) & 15) != 0) return false;
    if (d.B_lo && (((uintptr_t)d.B_lo) & 15) != 0) return false;
    // logits as the A operand: either [pattern x class] read K-major or its transpose read MN-major
    if (d.a_transform && (a_k != (d.a_pattern_is_m != 0))) return false;
    return true;
}

ulsnn_status_t tc_gemm_launch(const GemmDesc& d, bool three_x, cudaStream_t stream) {
    if (!tc_gemm_supported(d)) return ULSNN_ERR_INVALID_ARG;
    TcParams p{};
    p.d = d;
    p.a_mn = (d.a_sk == 1) ? 0 : 1;
    p.b_mn = (d.b_sk == 1) ? 0 : 1;
    const int cg = tc_cta_group(d);
    p.bn = tc_tile_n(d);
    p.n_gran = cg * (p.b_mn ? 32 : 16);
    p.tiles_m = (int)((d.M + BM * cg - 1) / (BM * cg));
    p.tiles_n = (int)((d.N + p.bn - 1) / p.bn);
    const int splits = (d.epi == EPI_PARTIAL) ? d.splits : 1;
    const int64_t units = (int64_t)p.tiles_m * p.tiles_n * splits;
    if (units > 0x7fffffff) return ULSNN_ERR_TOO_LARGE;
    p.units = (int)units;
    p.three_x = three_x ? 1 : 0;
    p.a_pre = (three_x && d.A_lo && !d.a_transform) ? 1 : 0;
    p.b_pre = (three_x && d.B_lo) ? 1 : 0;
    p.split_pass = (d.a_transform || (three_x && !(p.a_pre && p.b_pre))) ? 1 : 0;
    p.producers = p.split_pass ? 1 : 2 + ((p.a_pre || p.b_pre) ? 1 : 0);
    p.direct = (cg == 2 && !p.split_pass) ? 1 : 0;
    p.fast_math = three_x ? 0 : 1;
    p.chunk_blocks = three_x ? 256 / BK : (1 << 30);       // 256 elements of K per accumulator in the accurate mode
    p.b_tile_bytes = (p.bn / cg) * ROW_BYTES;
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
    p.wait_limit = DEFAULT_WAIT_LIMIT_CYCLES;

    Maps m;
    memset(&m, 0, sizeof(m));
    auto map_of_a = [&](CUtensorMap* t, const float* base) {
        return p.a_mn ? make_map(t, base, d.M, d.K, d.a_sk, 32, BK, true) : make_map(t, base, d.K, d.M, d.a_sm, BK, BM, false);
    };
    auto map_of_b = [&](CUtensorMap* t, const float* base) {
        return p.b_mn ? make_map(t, base, d.N, d.K, d.b_sk, 32, BK, true) : make_map(t, base, d.K, d.N, d.b_sn, BK, p.bn / cg, false);
    };
    if (!map_of_a(&m.a, d.A) || !map_of_b(&m.b, d.B)) return ULSNN_ERR_CUDA;
    if (p.a_pre && !map_of_a(&m.a_lo, d.A_lo)) return ULSNN_ERR_CUDA;
    if (p.b_pre && !map_of_b(&m.b_lo, d.B_lo)) return ULSNN_ERR_CUDA;
    p.c_pair = ((d.epi == EPI_BIAS_TANH || d.epi == EPI_TANH_SSE) && d.C_lo) ? 1 : 0;
    // the output goes through TMA stores when its rows are 16-byte aligned; otherwise the epilogue stores directly
    if (d.epi == EPI_PARTIAL) {
        p.c_tma = make_store_map(&m.c, d.partials, d.N, d.M, d.ldp, splits) ? 1 : 0;
    } else if (d.C && (((uintptr_t)d.C) & 15) == 0 && (d.ldc & 3) == 0 && d.ldc >= 4) {
        // A TMA store clips a row at the next 16-byte boundary past the matrix edge, so a width that is not a multiple
        // of four spills up to three floats into the row's padding.  That padding is scratch in the library's own
        // logit and delta buffers; it belongs to the caller in C, and it is the ones column in an activation buffer.
        const bool pad_is_scratch = d.epi == EPI_LOGITS || d.epi == EPI_TANHP || d.epi == EPI_TANH_SSE;
        if ((d.N & 3) == 0 || pad_is_scratch) p.c_tma = make_store_map(&m.c, d.C, d.N, d.M, d.ldc, 1) ? 1 : 0;
        if (p.c_tma && p.c_pair)
            p.c_tma = ((((uintptr_t)d.C_lo) & 15) == 0 && make_store_map(&m.c_lo, d.C_lo, d.N, d.M, d.ldc, 1)) ? 1 : 0;
    }

    const int smem_bytes = 1024 + stages * p.stage_bytes + EPI_SCRATCH_BYTES + CTRL_BYTES;
    const int slots = sm_count() / cg;
    const int grid = cg * (p.units < slots ? p.units : slots);
    switch (d.epi) {
        case EPI_SGEMM:     return launch_cg<EPI_SGEMM>(cg, m, p, smem_bytes, grid, stream);
        case EPI_BIAS_TANH: return launch_cg<EPI_BIAS_TANH>(cg, m, p, smem_bytes, grid, stream);
        case EPI_LOGITS:    return launch_cg<EPI_LOGITS>(cg, m, p, smem_bytes, grid, stream);
        case EPI_TANHP:     return launch_cg<EPI_TANHP>(cg, m, p, smem_bytes, grid, stream);
        case EPI_PARTIAL:   return launch_cg<EPI_PARTIAL>(cg, m, p, smem_bytes, grid, stream);
        case EPI_TANH_SSE:  return launch_cg<EPI_TANH_SSE>(cg, m, p, smem_bytes, grid, stream);
    }
    return ULSNN_ERR_INVALID_ARG;
}

int* device_status_word() { return status_ptr(); }

ulsnn_status_t tc_wait_probe_launch(unsigned long long limit_cycles, cudaStream_t stream) {
    int* status = status_ptr();
    if (!status) return ULSNN_ERR_CUDA;
    wait_probe_kernel<<<1, 32, 0, stream>>>(status, limit_cycles);
    count_launch(2);
    return cuda_ok(cudaGetLastError());
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
