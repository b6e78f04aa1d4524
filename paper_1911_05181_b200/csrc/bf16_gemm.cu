// tcgen05 engine for operands stored as bfloat16 (the 16-bit mode: Section 1 notes that 16 bits are enough for
// smaller networks, Section 4.2 that the precision of the products is what limits the network size).
// Operands are rounded to bfloat16 once, in global memory; the products accumulate in fp32 on the tensor core
// (tcgen05.mma.kind::f16, 128 x N x 16 per instruction, twice the TF32 rate) and the activations and deltas that
// the epilogues write are bfloat16 again, so that every later product reads half the bytes.
//
// One persistent CTA per SM, 10 warps:
//   warps 0,10  TMA producers     global -> 128B-swizzled shared-memory stages (no multicast); warp 0 fetches the A
//                                 tiles and warp 10 the B tiles: a thread gets its next copy accepted only some
//                                 hundred nanoseconds after the previous one, so two issuers nearly double the rate
//   warp 1      product issuer    an elected lane issues the products and commits (idle in the second CTA of a pair)
//   warps 2-9   epilogue          two warps per TMEM lane quarter, each taking every other 64-column block of the
//                                 128 x BN fp32 accumulator: fused math, then blocks staged in swizzled shared
//                                 memory and written with TMA stores
// Tiles are 128 x BN, or 256 x BN by the two CTAs of a cluster (cta_group::2), BN <= 256: each CTA fetches its own
// halves of the operands, and both count the landed bytes on the first CTA's barrier (cta_group::2 form of the TMA
// load), so that the issuer there waits on one barrier for the whole stage.  TMEM holds two
// accumulators, so the epilogue of a tile overlaps the products of the next.  There is no operand pass: every
// byte the tensor core reads arrived by TMA.
// K-major operands: rows of 64 elements (128 bytes), 128B swizzle.  MN-major operands: boxes of 64 (M or N) x 64
// (K) elements, 128B swizzle, read by the tensor core through the transpose bits of the instruction descriptor.
// Every wait on an mbarrier is bounded, as in the TF32 engine.
#include "common.cuh"
#include "tc_ptx.cuh"
#include <cuda.h>
#include <math.h>
#include <string.h>
#include <mutex>

namespace ulsnn {

namespace {

constexpr int BM = 128;
constexpr int BN_MAX = 256;
constexpr int BK = 64;                  // elements of K per stage: a K-major tile row is 128 bytes
constexpr int UMMA_K = 16;              // K of one tcgen05.mma.kind::f16
constexpr int NUM_EPI_WARPS = 8;
constexpr int PROD_B_WARP = 2 + NUM_EPI_WARPS;      // second producer warp
constexpr int NUM_WARPS = 3 + NUM_EPI_WARPS;
constexpr int NUM_THREADS = NUM_WARPS * 32;
constexpr int MAX_STAGES = 8;
constexpr int NUM_SMS = 148;
constexpr int A_TILE_BYTES = BM * BK * 2;
constexpr int SMEM_BUDGET = 227 * 1024;
constexpr int EPI_STAGE_BYTES = 32 * 128;           // one block of 32 rows x 128 bytes (64 bf16 or 32 fp32), 128B-swizzled
constexpr int EPI_BUFS = 1;
constexpr int EPI_SCRATCH_BYTES = NUM_EPI_WARPS * EPI_BUFS * EPI_STAGE_BYTES;
constexpr int CTRL_BYTES = 1024;
constexpr float LOG2E = 1.4426950408889634f;

struct HgParams {
    HalfGemmDesc d;
    int bn, n_gran, tiles_m, tiles_n, units, stages, b_tile_bytes, stage_bytes;
    int a_mn, b_mn;
    int c_tma;
    unsigned long long wait_limit;      // clock cycles a device-side wait may take before the CTA gives up
    int* status;
};

struct Ctrl {
    uint64_t full[MAX_STAGES];      // TMA bytes landed (CTA 0 of a pair: the bytes of both CTAs)
    uint64_t empty[MAX_STAGES];     // products that read the stage have completed
    uint64_t reg_full[2];           // the products of the tile in TMEM region r have completed
    uint64_t reg_free[2];           // the epilogue warps have read region r
    uint64_t free_sink[2][NUM_EPI_WARPS];
    uint32_t tmem_base;
    volatile int abort;
    unsigned long long wait_limit;
};

template <int CG>
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    if (elect_one()) {
        if constexpr (CG == 1) {
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "setp.ne.b32 p, %4, 0;\n\t"
                "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
        } else {
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "setp.ne.b32 p, %4, 0;\n\t"
                "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
        }
    }
}

__device__ __forceinline__ float tanh_approx(float x) {
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// two floats -> one word of two bfloat16 (round to nearest even), lo in the low half
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

template <int EPI, int CG>
__global__ void __launch_bounds__(NUM_THREADS, 1)
bf16_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_c, const HgParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_base = smem;
    uint8_t* epi_scratch = smem + (size_t)p.stages * p.stage_bytes;
    Ctrl* ctrl = (Ctrl*)(epi_scratch + EPI_SCRATCH_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const HalfGemmDesc& d = p.d;
    const int rank = (CG == 2) ? (int)cluster_ctarank() : 0;
    const int first_unit = blockIdx.x / CG, unit_step = gridDim.x / CG;
    // bf16 outputs (activations, exponentials, deltas) against fp32 outputs (C of an SGEMM, split-K partials)
    constexpr bool OUT16 = (EPI == EPI_BIAS_TANH || EPI == EPI_LOGITS || EPI == EPI_TANHP || EPI == EPI_TANH_SSE);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 2);         // one arrival (with its byte count) from each producer warp
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&ctrl->reg_full[a]), 1);
            mbar_init(smem_u32(&ctrl->reg_free[a]), NUM_EPI_WARPS + (CG == 2 ? 1 : 0));
        }
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
    const int off_a = 0, off_b = A_TILE_BYTES;

    if (warp == 0 || warp == PROD_B_WARP) {
        // ------------------------------------------------------------------ TMA producers (A tiles / B tiles)
        const bool do_a = warp == 0;
        RingPos rp{0, 0};
        bool ok = true;
        for (int u = first_unit; u < p.units && ok; u += unit_step) {
            int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
            int64_t kbeg; int nkb, tail; unit_k_range<BK, UMMA_K>(p, sp, kbeg, nkb, tail);
            const int b_cols = tile_cols(p, nt) / CG;
            const int m0 = (mt * CG + rank) * BM, n0 = nt * p.bn + rank * b_cols;
            const int b_boxes = b_cols >> 6;        // MN-major B: boxes of 64 columns, only those the products read
            const uint32_t b_bytes = (uint32_t)(p.b_mn ? b_boxes * (BK * 128) : p.b_tile_bytes);
            int k0 = (int)kbeg;
            for (int kb = 0; kb < nkb; ++kb, k0 += BK) {
                const int s = rp.stage;
                if (!wait_bar_warp(&ctrl->empty[s], rp.phase ^ 1, ctrl, p.status)) { ok = false; break; }
                rp.advance(p.stages);
                const uint32_t bar_local = smem_u32(&ctrl->full[s]);
                const uint32_t bar = (CG == 2) ? addr_in_rank0(bar_local) : bar_local;
                const uint32_t sa = smem_u32(stage_base + (size_t)s * p.stage_bytes + off_a);
                const uint32_t sb = sa + off_b;
                auto load = [&](uint32_t dst, const CUtensorMap* map, int x, int y) {
                    if constexpr (CG == 2) tma_load_2d_pair(dst, map, x, y, bar); else tma_load_2d(dst, map, x, y, bar);
                };
                if (elect_one()) {
                    // CTA 0 announces the bytes of both CTAs of the pair (they fetch the same amounts)
                    if (do_a) {
                        if (rank == 0) mbar_expect_tx(bar_local, (uint32_t)A_TILE_BYTES * CG);
                        if (!p.a_mn) {
                            load(sa, &map_a, k0, m0);                                   // box {64 k, 128 rows}
                        } else {
#pragma unroll
                            for (int g = 0; g < BM / 64; ++g)                           // boxes {64 m, 64 k}
                                load(sa + g * (BK * 128), &map_a, m0 + 64 * g, k0);
                        }
                    } else {
                        if (rank == 0) mbar_expect_tx(bar_local, b_bytes * CG);
                        if (!p.b_mn) {
                            load(sb, &map_b, k0, n0);                                   // box {64 k, bn/CG rows}
                        } else {
#pragma unroll
                            for (int g = 0; g < BN_MAX / 64; ++g)
                                if (g < b_boxes) load(sb + g * (BK * 128), &map_b, n0 + 64 * g, k0);
                        }
                    }
                }
                __syncwarp();
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ product issuer
        if (rank == 0) {
            // instruction descriptor: fp32 accumulator, bf16 x bf16, transpose bits for MN-major operands, M, N
            const uint32_t idesc0 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) |
                                    ((uint32_t)((BM * CG) >> 4) << 24);
            // K-major: 8-row groups 1024 B apart (SBO), a product advances 32 B inside the 128-byte row.
            // MN-major: 64-element groups one box (BK*128 B) apart (LBO), 8-k groups 1024 B apart (SBO), a product
            // (16 k) advances 2048 B.
            const uint32_t a_lbo = p.a_mn ? BK * 128 : 16, b_lbo = p.b_mn ? BK * 128 : 16;
            const uint32_t a_kstep = p.a_mn ? 2048 : UMMA_K * 2, b_kstep = p.b_mn ? 2048 : UMMA_K * 2;
            const uint32_t base0 = smem_u32(stage_base);
            const uint64_t da0 = smem_desc(base0 + off_a, a_lbo, 1024, 2);
            const uint64_t db0 = smem_desc(base0 + off_b, b_lbo, 1024, 2);
            const uint32_t a_kinc = a_kstep >> 4, b_kinc = b_kstep >> 4, stage_inc = (uint32_t)p.stage_bytes >> 4;
            RingPos rp{0, 0};
            uint32_t tile_i = 0;
            bool ok = true;
            for (int u = first_unit; u < p.units && ok; u += unit_step, ++tile_i) {
                int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
                int64_t kbeg; int nkb, tail; unit_k_range<BK, UMMA_K>(p, sp, kbeg, nkb, tail);
                const uint32_t idesc = idesc0 | ((uint32_t)(tile_cols(p, nt) >> 3) << 17);
                const uint32_t reg = tile_i & 1;
                if (tile_i >= 2) {      // the region has held a tile before: wait until every epilogue warp has read it
                    if (CG == 2 && elect_one()) mbar_expect_tx(smem_u32(&ctrl->reg_free[reg]), 8 * NUM_EPI_WARPS);
                    if (!wait_bar_warp(&ctrl->reg_free[reg], ((tile_i >> 1) - 1) & 1, ctrl, p.status)) { ok = false; break; }
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + reg * BN_MAX;
                for (int kb = 0; kb < nkb; ++kb) {
                    const int s = rp.stage;
                    if (!wait_bar_warp(&ctrl->full[s], rp.phase, ctrl, p.status)) { ok = false; break; }
                    rp.advance(p.stages);
                    tc_fence_after();
                    const uint32_t soff = (uint32_t)s * stage_inc;
                    const int steps = (kb == nkb - 1) ? tail : BK / UMMA_K;
#pragma unroll
                    for (int ks = 0; ks < BK / UMMA_K; ++ks) {
                        if (ks >= steps) break;
                        umma_bf16<CG>(d_tmem, da0 + (uint64_t)(soff + ks * a_kinc), db0 + (uint64_t)(soff + ks * b_kinc), idesc,
                                      (kb == 0 && ks == 0) ? 0u : 1u);
                    }
                    umma_commit<CG>(smem_u32(&ctrl->empty[s]));
                }
                if (ok) umma_commit<CG>(smem_u32(&ctrl->reg_full[reg]));
            }
        }
    } else if (warp < 2 + NUM_EPI_WARPS) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;                         // TMEM lane quarter this warp may read
        const int ew = warp - 2;                        // 0..7
        const int half = ew >> 2;                       // which 64-column blocks of a tile this warp takes
        uint8_t* stg = epi_scratch + ew * (EPI_BUFS * EPI_STAGE_BYTES);
        const uint32_t lane_off = (uint32_t)(q * 32) << 16;
        const bool c_vec = ((((uintptr_t)d.C) & 15) == 0) && ((d.ldc & 3) == 0);
        const bool bias_vec = (EPI == EPI_BIAS_TANH || EPI == EPI_LOGITS || EPI == EPI_TANH_SSE) && ((((uintptr_t)d.bias) & 15) == 0);
        const bool t_vec = (EPI == EPI_TANH_SSE) && ((((uintptr_t)d.T) & 15) == 0) && ((d.ldt & 3) == 0);
        const bool ch_vec = ((((uintptr_t)d.Ch) & 15) == 0) && ((d.ldch & 7) == 0);
        const bool h_vec = (EPI == EPI_TANHP) && ((((uintptr_t)d.Hm) & 15) == 0) && ((d.ldh & 7) == 0);
        uint32_t tile_i = 0, stg_i = 0;
        bool ok = true;
        for (int u = first_unit; u < p.units && ok; u += unit_step, ++tile_i) {
            int mt, nt, sp; unit_coords(p, u, mt, nt, sp);
            const uint32_t acc = tile_i & 1;
            const int n0 = nt * p.bn;
            const int cols_in = min(p.bn, (int)d.N - n0);
            const int nblk = (cols_in + 63) >> 6;           // 64-column blocks of this tile inside the matrix
            const int r0w = (mt * CG + rank) * BM + q * 32;
            const int64_t r = (int64_t)r0w + lane;
            const bool rv = r < d.M;
            float run_m = -INFINITY, run_s = 0.f, zl = 0.f;
            bool have_zl = false;
            int lab = -1;
            if (EPI == EPI_LOGITS && rv) lab = __ldg(d.labels + r);        // asked for before the wait for the products
            // TANH_SSE: the targets of a 64-column block are brought into L2 one block ahead of their use
            auto prefetch_targets = [&](int b64) {
                const int c0 = n0 + b64 * 64;
                if (EPI == EPI_TANH_SSE && rv && b64 < nblk) {
                    const float* tp = d.T + r * d.ldt + c0;
                    const int last = min(63, (int)d.N - c0 - 1);
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(tp));
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(tp + (last >> 1)));
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(tp + last));
                }
            };
            prefetch_targets(half);
            if (!wait_bar(&ctrl->reg_full[acc], (tile_i >> 1) & 1, ctrl, p.status)) { ok = false; break; }
            tc_fence_after();

            // next staging block of this warp, free to be written
            auto next_block = [&]() -> uint8_t* {
                uint8_t* blk = stg + (stg_i % EPI_BUFS) * EPI_STAGE_BYTES;
                ++stg_i;
                if (lane == 0) { if (EPI_BUFS == 2) bulk_wait_read_1(); else bulk_wait_read_0(); }
                __syncwarp();
                return blk;
            };

            for (int blk64 = half; blk64 < nblk; blk64 += 2) {
                uint32_t packed[32];                    // OUT16: this thread's 64 values of the block, as bf16 pairs
                float cmax[2] = {0.f, 0.f};
                // both 32-column chunks of the block and their biases are asked for before the first is used
                uint32_t raw[2][32];
                float bv[2][32];
                const int nv64 = min(64, (int)d.N - (n0 + blk64 * 64));
                prefetch_targets(blk64 + 2);
                tmem_ld32(tmem_base + acc * BN_MAX + (2 * blk64) * 32 + lane_off, raw[0]);
                if (nv64 > 32) tmem_ld32(tmem_base + acc * BN_MAX + (2 * blk64 + 1) * 32 + lane_off, raw[1]);
                if (EPI == EPI_BIAS_TANH || EPI == EPI_LOGITS || EPI == EPI_TANH_SSE) {
#pragma unroll
                    for (int cc = 0; cc < 2; ++cc) {
                        const int c0 = n0 + (2 * blk64 + cc) * 32;
                        const int nvalid = max(0, min(32, (int)d.N - c0));
                        if (bias_vec && nvalid == 32) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4) {
                                const float4 bb = __ldg(reinterpret_cast<const float4*>(d.bias + c0 + j));
                                bv[cc][j] = bb.x; bv[cc][j + 1] = bb.y; bv[cc][j + 2] = bb.z; bv[cc][j + 3] = bb.w;
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) bv[cc][j] = (j < nvalid) ? __ldg(d.bias + c0 + j) : 0.f;
                        }
                    }
                }
                tmem_ld_wait();
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    const int c = 2 * blk64 + cc;
                    const int c0 = n0 + c * 32;
                    const int nvalid = max(0, min(32, (int)d.N - c0));
                    const bool full = nvalid == 32;
                    float v[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = (nvalid > 0) ? __uint_as_float(raw[cc][j]) : 0.f;

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
                    } else if (EPI == EPI_TANH_SSE) {
                        // Eqs. 1 and 3: y = tanh(z), E += (y - t)^2, stored value dE/dz = 2 (y - t)(1 - y^2)
                        float s = 0.f;
                        if (rv && nvalid > 0) {
                            const float* tp = d.T + r * d.ldt + c0;
#pragma unroll
                            for (int j = 0; j < 32; j += 4) {
                                float4 t4;
                                if (t_vec && full) t4 = __ldg(reinterpret_cast<const float4*>(tp + j));
                                else t4 = make_float4(j < nvalid ? __ldg(tp + j) : 0.f, j + 1 < nvalid ? __ldg(tp + j + 1) : 0.f,
                                                      j + 2 < nvalid ? __ldg(tp + j + 2) : 0.f, j + 3 < nvalid ? __ldg(tp + j + 3) : 0.f);
                                const float tt[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
                                for (int t = 0; t < 4; ++t) {
                                    const float y = tanh_approx(v[j + t] + bv[cc][j + t]);
                                    const float e = (j + t < nvalid) ? y - tt[t] : 0.f;
                                    s += e * e;
                                    v[j + t] = 2.f * e * (1.f - y * y);
                                }
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = 0.f;
                        }
                        run_s += s;
                    } else if (EPI == EPI_BIAS_TANH || EPI == EPI_LOGITS) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] += bv[cc][j];
                        if (EPI == EPI_BIAS_TANH) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = (j < nvalid) ? tanh_approx(v[j]) : 0.f;
                        } else if (nvalid > 0) {
                            // four interleaved chains each for the maximum and the sum (fixed order)
                            float cm4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                            for (int j = 0; j < 32; ++j) { if (j >= nvalid) v[j] = -INFINITY; cm4[j & 3] = fmaxf(cm4[j & 3], v[j]); }
                            const float cm = fmaxf(fmaxf(cm4[0], cm4[1]), fmaxf(cm4[2], cm4[3]));
                            const float nm = fmaxf(run_m, cm);
                            if ((unsigned)(lab - c0) < (unsigned)nvalid) {
#pragma unroll
                                for (int j = 0; j < 32; ++j) if (c0 + j == lab) zl = v[j];
                                have_zl = true;
                            }
                            // stored: exp(z - nm), nm noted per 32-class chunk; the same values make up the row sum
                            const float nm2 = nm * LOG2E;
                            float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                            for (int j = 0; j < 32; ++j) { v[j] = (j < nvalid) ? ex2_approx(fmaf(v[j], LOG2E, -nm2)) : 0.f; s4[j & 3] += v[j]; }
                            const float s = (s4[0] + s4[1]) + (s4[2] + s4[3]);
                            run_s = (run_m == -INFINITY ? 0.f : run_s * ex2_approx((run_m - nm) * LOG2E)) + s;
                            run_m = nm;
                            cmax[cc] = nm;
                        }
                    } else if (EPI == EPI_TANHP) {
                        if (rv && nvalid > 0) {
                            const __nv_bfloat16* hp = d.Hm + r * d.ldh + c0;
                            if (h_vec && full) {
#pragma unroll
                                for (int j = 0; j < 32; j += 8) {
                                    const uint4 w = __ldg(reinterpret_cast<const uint4*>(hp + j));
                                    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                                    for (int t = 0; t < 4; ++t) {
                                        const float h0 = bf16_lo(ww[t]), h1 = bf16_hi(ww[t]);
                                        v[j + 2 * t] *= (1.f - h0 * h0);
                                        v[j + 2 * t + 1] *= (1.f - h1 * h1);
                                    }
                                }
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j) {
                                    if (j < nvalid) { const float h = __bfloat162float(hp[j]); v[j] = (1.f - h * h) * v[j]; } else v[j] = 0.f;
                                }
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = 0.f;
                        }
                    }

                    if constexpr (OUT16) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) packed[cc * 16 + j] = pack_bf16(v[2 * j], v[2 * j + 1]);
                    } else if (nvalid > 0) {
                        // fp32 output: a 32 x 32 block per chunk
                        float* base = (EPI == EPI_PARTIAL) ? d.partials + (int64_t)sp * d.M * d.ldp : d.C;
                        const int64_t ld = (EPI == EPI_PARTIAL) ? d.ldp : d.ldc;
                        if (p.c_tma) {
                            uint8_t* blk = next_block();
                            float4* rowp = reinterpret_cast<float4*>(blk + lane * 128);
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                rowp[j ^ (lane & 7)] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                            proxy_fence_async();
                            __syncwarp();
                            if (lane == 0 && r0w < d.M) {
                                tma_store_3d(&map_c, smem_u32(blk), c0, r0w, EPI == EPI_PARTIAL ? sp : 0);
                                bulk_commit();
                            }
                        } else {
                            // rows TMA cannot address (a leading dimension that is not a multiple of four, a base that is not
                            // 16-byte aligned): through the same staging block, then row by row in 128-byte runs by the warp
                            uint8_t* blk = next_block();
                            float4* rowp = reinterpret_cast<float4*>(blk + lane * 128);
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                rowp[j ^ (lane & 7)] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                            __syncwarp();
                            const int rows_here = min(32, (int)(d.M - r0w));
                            if (lane < nvalid) {
                                float* dst = base + (int64_t)r0w * ld + c0 + lane;
                                for (int rr = 0; rr < rows_here; ++rr) {
                                    const float* src = reinterpret_cast<const float*>(blk + rr * 128 + ((((lane >> 2) ^ (rr & 7)) << 4) | ((lane & 3) << 2)));
                                    dst[(int64_t)rr * ld] = *src;
                                }
                            }
                            __syncwarp();
                        }
                    }
                }
                if constexpr (OUT16) {
                    const int c0 = n0 + blk64 * 64;
                    if (d.Ch) {
                        if (p.c_tma) {
                            uint8_t* blk = next_block();
                            uint4* rowp = reinterpret_cast<uint4*>(blk + lane * 128);
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                rowp[j ^ (lane & 7)] = make_uint4(packed[4 * j], packed[4 * j + 1], packed[4 * j + 2], packed[4 * j + 3]);
                            proxy_fence_async();
                            __syncwarp();
                            if (lane == 0 && r0w < d.M) {
                                tma_store_2d(&map_c, smem_u32(blk), c0, r0w);
                                bulk_commit();
                            }
                        } else if (rv) {
                            __nv_bfloat16* dst = d.Ch + r * d.ldch + c0;
                            if (ch_vec && nv64 == 64) {
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    reinterpret_cast<uint4*>(dst)[j] = make_uint4(packed[4 * j], packed[4 * j + 1], packed[4 * j + 2], packed[4 * j + 3]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j) {
                                    if (2 * j < nv64) dst[2 * j] = __ushort_as_bfloat16((unsigned short)(packed[j] & 0xFFFFu));
                                    if (2 * j + 1 < nv64) dst[2 * j + 1] = __ushort_as_bfloat16((unsigned short)(packed[j] >> 16));
                                }
                            }
                        }
                    }
                    if (EPI == EPI_LOGITS && rv && d.chunk_max)
                        *reinterpret_cast<float2*>(d.chunk_max + r * d.chunk_ld + (c0 >> 5)) = make_float2(cmax[0], cmax[1]);
                }
            }
            // all TMEM reads of this accumulator are done: hand it back to the issuing warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { if (CG == 2 && rank == 1) signal_rank0(smem_u32(&ctrl->free_sink[acc][ew]), smem_u32(&ctrl->reg_free[acc])); else mbar_arrive(smem_u32(&ctrl->reg_free[acc])); }

            if (EPI == EPI_LOGITS && rv) {
                d.stats[r * d.stats_ld + nt * 2 + half] = make_float2(run_m, run_s);
                if (have_zl) d.zlabel[r] = zl;
            }
            if (EPI == EPI_TANH_SSE && rv) d.stats[r * d.stats_ld + nt * 2 + half] = make_float2(0.f, run_s);
            if (EPI == EPI_BIAS_TANH && d.ones_cols > 0 && nt == p.tiles_n - 1 && half == 0 && rv) {
                d.Ch[r * d.ldch + d.N] = __float2bfloat16_rn(1.f);
                for (int cc = 1; cc < d.ones_cols; ++cc) d.Ch[r * d.ldch + d.N + cc] = __float2bfloat16_rn(0.f);
            }
        }
        if (lane == 0) bulk_wait_all();
    }

    // ---------------------------------------------------------------------- teardown
    if (ctrl->abort) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    __syncwarp();
    tc_fence_before();
    if constexpr (CG == 2) cluster_sync_all(); else __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<CG>(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------------ small kernels

// dst[r][j] = bf16(src[r][j]) for j < cols; dst[r][cols] = 1 when `ones`; the rest of the row (up to ldd) = 0.
// One thread per 8 output elements (one 16-byte store).
__global__ void to_bf16_kernel(const float* __restrict__ src, int64_t rows, int64_t cols, int64_t lds,
                               __nv_bfloat16* __restrict__ dst, int64_t ldd, int ones) {
    const int64_t groups = ldd >> 3;
    const int64_t total = rows * groups;
    const bool vec = ((((uintptr_t)src) & 15) == 0) && ((lds & 3) == 0);
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = e / groups, j0 = (e - r * groups) << 3;
        float v[8];
        const float* s = src + r * lds + j0;
        if (vec && j0 + 8 <= cols) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(s)), b = __ldg(reinterpret_cast<const float4*>(s) + 1);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
        } else {
#pragma unroll
            for (int t = 0; t < 8; ++t) v[t] = (j0 + t < cols) ? __ldg(s + t) : ((ones && j0 + t == cols) ? 1.f : 0.f);
        }
        *reinterpret_cast<uint4*>(dst + r * ldd + j0) =
            make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
    }
}

// In place: E[p][j] (= exp(z - m) as the LOGITS epilogue left it) -> bf16(E[p][j] * scale[p][j/32] - [label_p == j]),
// zero for j >= n_classes.  One thread per 8 elements, which lie in one 32-class chunk.
__global__ void delta_bf16_kernel(__nv_bfloat16* __restrict__ E, int64_t lde, const float* __restrict__ scale, int64_t scale_ld,
                                  const int32_t* __restrict__ labels, int64_t n, int n_classes) {
    const int64_t groups = lde >> 3;
    const int64_t total = n * groups;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t pat = e / groups;
        const int j0 = (int)(e - pat * groups) << 3;
        uint4* ptr = reinterpret_cast<uint4*>(E + pat * lde + j0);
        uint4 w = *ptr;
        const float f = (j0 < n_classes) ? __ldg(scale + pat * scale_ld + (j0 >> 5)) : 0.f;
        const int lab = __ldg(labels + pat);
        uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int j = j0 + 2 * t;
            const float d0 = (j < n_classes) ? fmaf(bf16_lo(ww[t]), f, j == lab ? -1.f : 0.f) : 0.f;
            const float d1 = (j + 1 < n_classes) ? fmaf(bf16_hi(ww[t]), f, j + 1 == lab ? -1.f : 0.f) : 0.f;
            ww[t] = pack_bf16(d0, d1);
        }
        *ptr = make_uint4(ww[0], ww[1], ww[2], ww[3]);
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

// bf16 matrix whose contiguous dimension has `inner` elements, `outer` rows `stride_elems` apart; 128B swizzle
bool make_map16(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t stride_elems, int box_inner, int box_outer,
                bool store) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t gstride[1] = {(cuuint64_t)stride_elems * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)base, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, store ? CU_TENSOR_MAP_L2_PROMOTION_NONE : CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 output written with TMA stores: `slices` matrices of rows x cols, box = one 32 x 32 block
bool make_store_map32(CUtensorMap* map, const float* base, int64_t cols, int64_t rows, int64_t ld, int64_t slices) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)slices};
    cuuint64_t gstride[2] = {(cuuint64_t)ld * sizeof(float), (cuuint64_t)rows * (cuuint64_t)ld * sizeof(float)};
    cuuint32_t box[3] = {32, 32, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, (void*)base, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool operand_ok(const void* base, int64_t ld) {
    return (((uintptr_t)base) & 15) == 0 && (ld & 7) == 0 && ld >= 8 && ld < ((int64_t)1 << 38);
}

int sm_count() { return sm_count_of_current_device(NUM_SMS); }

template <int EPI, int CG>
ulsnn_status_t launch(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const HgParams& p, int smem_bytes,
                      int grid, cudaStream_t stream) {
    static std::atomic<uint64_t> configured{0};
    if (!allow_dynamic_smem(bf16_gemm_kernel<EPI, CG>, SMEM_BUDGET, configured)) return ULSNN_ERR_CUDA;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, bf16_gemm_kernel<EPI, CG>, ma, mb, mc, p);
    count_launch(1);
    return cuda_ok(e == cudaSuccess ? cudaGetLastError() : e);
}

template <int EPI>
ulsnn_status_t launch_cg(int cg, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const HgParams& p,
                         int smem_bytes, int grid, cudaStream_t stream) {
    return cg == 2 ? launch<EPI, 2>(ma, mb, mc, p, smem_bytes, grid, stream) : launch<EPI, 1>(ma, mb, mc, p, smem_bytes, grid, stream);
}

inline int cta_group(const HalfGemmDesc& d) { return d.M > BM ? 2 : 1; }

}  // namespace

int hg_tile_m(const HalfGemmDesc& d) { return BM * cta_group(d); }
int hg_slots(const HalfGemmDesc& d) { return NUM_SMS / cta_group(d); }
int hg_k_granule() { return BK; }

int hg_tile_n(const HalfGemmDesc& d) {
    // 64-column blocks are the unit of the epilogue's bf16 stores and of an MN-major B box (one per CTA of a pair)
    const bool b_mn = !(d.b_sk == 1);
    const int64_t g = (b_mn && cta_group(d) == 2) ? 128 : 64;
    int64_t bn = (d.N + g - 1) / g * g;
    if (bn > BN_MAX) bn = BN_MAX;
    return (int)bn;
}

bool hg_gemm_supported(const HalfGemmDesc& d) {
    if (d.M <= 0 || d.N <= 0 || d.K <= 0) return false;
    if (d.M > 0x7fffffff || d.N > 0x7fffffff || d.K > 0x7fffffff) return false;
    if (!encode_fn()) return false;
    const bool a_k = (d.a_sk == 1), b_k = (d.b_sk == 1);
    if (!a_k && d.a_sm != 1) return false;
    if (!b_k && d.b_sn != 1) return false;
    if (!operand_ok(d.A, a_k ? d.a_sm : d.a_sk)) return false;
    if (!operand_ok(d.B, b_k ? d.b_sn : d.b_sk)) return false;
    if (d.epi == EPI_PARTIAL && (d.k_per_split % BK) != 0) return false;
    return true;
}

ulsnn_status_t hg_gemm_launch(const HalfGemmDesc& d, cudaStream_t stream) {
    if (!hg_gemm_supported(d)) return ULSNN_ERR_INVALID_ARG;
    HgParams p{};
    p.d = d;
    p.a_mn = (d.a_sk == 1) ? 0 : 1;
    p.b_mn = (d.b_sk == 1) ? 0 : 1;
    const int cg = cta_group(d);
    p.bn = hg_tile_n(d);
    p.n_gran = cg * (p.b_mn ? 64 : 16);
    p.tiles_m = (int)((d.M + BM * cg - 1) / (BM * cg));
    p.tiles_n = (int)((d.N + p.bn - 1) / p.bn);
    const int splits = (d.epi == EPI_PARTIAL) ? d.splits : 1;
    const int64_t units = (int64_t)p.tiles_m * p.tiles_n * splits;
    if (units > 0x7fffffff) return ULSNN_ERR_TOO_LARGE;
    p.units = (int)units;
    p.b_tile_bytes = (p.bn / cg) * BK * 2;
    p.stage_bytes = A_TILE_BYTES + p.b_tile_bytes;
    int stages = (SMEM_BUDGET - 1024 - EPI_SCRATCH_BYTES - CTRL_BYTES) / p.stage_bytes;
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    if (stages < 2) return ULSNN_ERR_INVALID_ARG;
    p.stages = stages;
    p.status = device_status_word();
    p.wait_limit = DEFAULT_WAIT_LIMIT_CYCLES;
    if (!p.status) return ULSNN_ERR_CUDA;

    CUtensorMap ma, mb, mc;
    memset(&ma, 0, sizeof(ma)); memset(&mb, 0, sizeof(mb)); memset(&mc, 0, sizeof(mc));
    const bool a_made = p.a_mn ? make_map16(&ma, d.A, d.M, d.K, d.a_sk, 64, BK, false) : make_map16(&ma, d.A, d.K, d.M, d.a_sm, BK, BM, false);
    const bool b_made = p.b_mn ? make_map16(&mb, d.B, d.N, d.K, d.b_sk, 64, BK, false) : make_map16(&mb, d.B, d.K, d.N, d.b_sn, BK, p.bn / cg, false);
    if (!a_made || !b_made) return ULSNN_ERR_CUDA;

    const bool out16 = d.epi == EPI_BIAS_TANH || d.epi == EPI_LOGITS || d.epi == EPI_TANHP || d.epi == EPI_TANH_SSE;
    if (d.epi == EPI_PARTIAL) {
        p.c_tma = make_store_map32(&mc, d.partials, d.N, d.M, d.ldp, splits) ? 1 : 0;
    } else if (d.epi == EPI_SGEMM) {
        if (d.C && (((uintptr_t)d.C) & 15) == 0 && (d.ldc & 3) == 0 && d.ldc >= 4 && (d.N & 3) == 0)
            p.c_tma = make_store_map32(&mc, d.C, d.N, d.M, d.ldc, 1) ? 1 : 0;
    } else if (out16 && d.Ch && (((uintptr_t)d.Ch) & 15) == 0 && (d.ldch & 7) == 0 && d.ldch >= 8) {
        // A TMA store clips a row at the next 16-byte boundary past the matrix edge: a width that is not a multiple of
        // eight spills into the row's padding.  That is scratch in the exponential and delta buffers, but it is the
        // ones column of an activation buffer.
        if ((d.N & 7) == 0 || d.epi != EPI_BIAS_TANH) p.c_tma = make_map16(&mc, d.Ch, d.N, d.M, d.ldch, 64, 32, true) ? 1 : 0;
    }

    const int smem_bytes = 1024 + stages * p.stage_bytes + EPI_SCRATCH_BYTES + CTRL_BYTES;
    const int slots = sm_count() / cg;
    const int grid = cg * (p.units < slots ? p.units : slots);
    switch (d.epi) {
        case EPI_SGEMM:     return launch_cg<EPI_SGEMM>(cg, ma, mb, mc, p, smem_bytes, grid, stream);
        case EPI_BIAS_TANH: return launch_cg<EPI_BIAS_TANH>(cg, ma, mb, mc, p, smem_bytes, grid, stream);
        case EPI_LOGITS:    return launch_cg<EPI_LOGITS>(cg, ma, mb, mc, p, smem_bytes, grid, stream);
        case EPI_TANHP:     return launch_cg<EPI_TANHP>(cg, ma, mb, mc, p, smem_bytes, grid, stream);
        case EPI_PARTIAL:   return launch_cg<EPI_PARTIAL>(cg, ma, mb, mc, p, smem_bytes, grid, stream);
        case EPI_TANH_SSE:  return launch_cg<EPI_TANH_SSE>(cg, ma, mb, mc, p, smem_bytes, grid, stream);
    }
    return ULSNN_ERR_INVALID_ARG;
}

ulsnn_status_t launch_to_bf16(const float* src, int64_t rows, int64_t cols, int64_t lds, __nv_bfloat16* dst, int64_t ldd,
                              int ones, cudaStream_t stream) {
    if (rows <= 0 || cols <= 0) return ULSNN_OK;
    if ((ldd & 7) != 0 || ldd < cols + (ones ? 1 : 0) || (((uintptr_t)dst) & 15) != 0) return ULSNN_ERR_INVALID_ARG;
    const int64_t total = rows * (ldd >> 3);
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    to_bf16_kernel<<<(unsigned)blocks, 256, 0, stream>>>(src, rows, cols, lds, dst, ldd, ones);
    count_launch(2);
    return cuda_ok(cudaGetLastError());
}

ulsnn_status_t launch_delta_bf16(__nv_bfloat16* E, int64_t lde, const float* scale, int64_t scale_ld, const int32_t* labels,
                                 int64_t n, int64_t n_classes, cudaStream_t stream) {
    if (n <= 0) return ULSNN_OK;
    if ((lde & 7) != 0 || (((uintptr_t)E) & 15) != 0) return ULSNN_ERR_INVALID_ARG;
    const int64_t total = n * (lde >> 3);
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    delta_bf16_kernel<<<(unsigned)blocks, 256, 0, stream>>>(E, lde, scale, scale_ld, labels, n, (int)n_classes);
    count_launch(2);
    return cuda_ok(cudaGetLastError());
}

}  // namespace ulsnn
