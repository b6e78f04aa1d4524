// PTX wrappers shared by the tensor-core engines: mbarriers, TMA copies, cluster signals, tcgen05 allocation,
// commits and TMEM access, shared-memory matrix descriptors.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <atomic>
#include "common.cuh"

namespace ulsnn {
namespace {

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
// One lane of a converged warp (always the same one for the full mask).  The warps that issue TMA copies and
// tensor-core products run their loops with all 32 lanes and elect the issuing lane around the instruction
// itself: addresses and descriptors then stay warp-uniform values.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred = 0;
    asm volatile("{\n\t.reg .pred px;\n\telect.sync _|px, 0xffffffff;\n\t@px mov.s32 %0, 1;\n\t}" : "+r"(pred));
    return pred != 0;
}
// Asynchronous signal to CTA 0: stores 8 bytes into CTA 0's shared memory at the offset of `sink` and completes 8
// transaction bytes on CTA 0's barrier at the offset of `bar`.  Unlike an arrival on a remote barrier it does not
// hold up the sending thread.
__device__ __forceinline__ void signal_rank0(uint32_t sink, uint32_t bar) {
    asm volatile(
        "{\n\t.reg .b32 rs, rb;\n\t.reg .b64 v;\n\t"
        "mapa.shared::cluster.u32 rs, %0, 0;\n\t"
        "mapa.shared::cluster.u32 rb, %1, 0;\n\t"
        "mov.b64 v, 0;\n\t"
        "st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b64 [rs], v, [rb];\n\t}"
        ::"r"(sink), "r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
// The same copy issued by a CTA of a pair (tcgen05 cta_group::2): the data lands in the issuing CTA's shared memory, the
// bytes are counted on the barrier at shared::cluster address `bar`, which may belong to the other CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
// shared::cluster address of CTA 0's copy of a shared-memory location of this CTA
__device__ __forceinline__ uint32_t addr_in_rank0(uint32_t local) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(r) : "r"(local));
    return r;
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_wait_read_0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// CG = number of CTAs (1 or 2) that share one tile: with 2, one tcgen05.mma spans the tensor cores of both SMs of
// a cluster, each CTA holding its 128 rows of A, its half of the B tile and its 128 rows of the accumulator
template <int CG> __device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    if constexpr (CG == 1) asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    else asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
template <int CG> __device__ __forceinline__ void tmem_relinquish() {
    if constexpr (CG == 1) asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    else asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
template <int CG> __device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    if constexpr (CG == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
template <int CG>
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    if (elect_one()) {
        if constexpr (CG == 1) {
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "setp.ne.b32 p, %4, 0;\n\t"
                "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
        } else {
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "setp.ne.b32 p, %4, 0;\n\t"
                "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
        }
    }
}
// The barrier (at this offset in every CTA of the tile) gets one arrival when the products issued so far are done.
template <int CG>
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    if (elect_one()) {
        if constexpr (CG == 1) {
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
        } else {
            asm volatile(
                "{\n\t.reg .b16 m;\n\tmov.b16 m, 3;\n\t"
                "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n\t}"
                ::"r"(bar) : "memory");
        }
    }
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
// Round to the nearest TF32 value (10 mantissa bits), ties away from zero, as cvt.rna.tf32.f32 does, but with two
// integer instructions at full rate: the conversion instruction runs at a fraction of it, and the operand pass
// applies this to every element of every landed tile.
__device__ __forceinline__ float to_tf32(float x) {
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u);
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
template <bool FAST> __device__ __forceinline__ float exp_t(float x) { return FAST ? __expf(x) : exp_fast_accurate(x); }

// Shared-memory matrix descriptor of a swizzled tile (sm_100 format: version 1 at bit 46; layout type at bits
// 61-63: 2 = 128B swizzle of 16-byte units, 1 = 128B swizzle of 32-byte units).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | ((uint64_t)layout << 61);
}

// Ring position: stage index and the parity of the pass over the ring.
struct RingPos {
    int stage; uint32_t phase;
    __device__ __forceinline__ void advance(int stages) { if (++stage == stages) { stage = 0; phase ^= 1u; } }
};

// Default limit of a device-side wait, in SM clock cycles (~1.5 s at 2 GHz): a kernel parameter, so that a test can
// make a wait run out within microseconds.
constexpr unsigned long long DEFAULT_WAIT_LIMIT_CYCLES = 3000000000ull;

// Bounded wait on an mbarrier of a CTA whose control block `ctrl` has the fields `abort` and `wait_limit`.  Returns
// false (after raising the abort flag and recording DEV_TIMEOUT in the device status word) if the phase did not
// complete within the limit, or if another thread of the CTA has given up already.
template <class CtrlT>
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, CtrlT* ctrl, int* status) {
    const uint32_t b = smem_u32(bar);
    if (mbar_try_wait(b, parity)) return true;
    const unsigned long long t0 = clock64();
    const unsigned long long limit = ctrl->wait_limit;
    uint32_t spins = 0;
    while (!mbar_try_wait(b, parity)) {
        if ((++spins & 255u) == 0) {
            if (ctrl->abort) return false;
            if ((unsigned long long)clock64() - t0 > limit) {
                ctrl->abort = 1;
                atomicExch(status, DEV_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}
// wait_bar by all lanes of a converged warp, with one outcome for the warp
template <class CtrlT>
__device__ __forceinline__ bool wait_bar_warp(uint64_t* bar, uint32_t parity, CtrlT* ctrl, int* status) {
    const bool ok = wait_bar(bar, parity, ctrl, status);
    return __all_sync(0xffffffffu, ok);
}

// Work units of a persistent kernel: unit u = (column tile nt, row tile mt, split-K slice sp), nt fastest.  P has the
// fields tiles_m, tiles_n, bn, n_gran and the product description d.
template <class P>
__device__ __forceinline__ void unit_coords(const P& p, int u, int& mt, int& nt, int& sp) {
    nt = u % p.tiles_n;
    const int r = u / p.tiles_n;
    mt = r % p.tiles_m;
    sp = r / p.tiles_m;
}
// columns of column tile nt that the products cover: the whole tile, or what is left of the matrix rounded up
template <class P>
__device__ __forceinline__ int tile_cols(const P& p, int nt) {
    const int left = (int)p.d.N - nt * p.bn;
    return left >= p.bn ? p.bn : (left + p.n_gran - 1) / p.n_gran * p.n_gran;
}
// k range of slice sp in blocks of BLOCK_K elements; tail_steps = product instructions (STEP_K elements each) of the last block
template <int BLOCK_K, int STEP_K, class P>
__device__ __forceinline__ void unit_k_range(const P& p, int sp, int64_t& kbeg, int& nkb, int& tail_steps) {
    kbeg = (p.d.epi == EPI_PARTIAL) ? (int64_t)sp * p.d.k_per_split : 0;
    int64_t kend = (p.d.epi == EPI_PARTIAL) ? kbeg + p.d.k_per_split : p.d.K;
    if (kend > p.d.K) kend = p.d.K;
    const int64_t len = kend - kbeg;
    nkb = (int)((len + BLOCK_K - 1) / BLOCK_K);
    const int rem = (int)(len - (int64_t)(nkb - 1) * BLOCK_K);      // 1..BLOCK_K elements in the last block
    tail_steps = (rem + STEP_K - 1) / STEP_K;
}

// ------------------------------------------------------------------------------------------ per-device host state
// One process may drive several GPUs, so whatever the host remembers about "the device" is kept per device ordinal.
inline int current_device_slot() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    return device_cache_slot(dev);
}
inline int sm_count_of_current_device(int fallback) {
    static std::atomic<int> cached[MAX_DEVICE_SLOTS];
    const int slot = current_device_slot();
    if (slot < 0) return fallback;
    int n = cached[slot].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, slot) != cudaSuccess || n <= 0) n = fallback;
        cached[slot].store(n, std::memory_order_relaxed);
    }
    return n;
}
// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) applies to the current device only: once per kernel and device.
// `done` is the kernel's own bit mask over the device slots.
template <class Kernel>
inline bool allow_dynamic_smem(Kernel kernel, int bytes, std::atomic<uint64_t>& done) {
    const int slot = current_device_slot();
    if (slot < 0) return false;
    const uint64_t bit = 1ull << slot;
    if (done.load(std::memory_order_acquire) & bit) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    done.fetch_or(bit, std::memory_order_release);
    return true;
}

}  // namespace
}  // namespace ulsnn
