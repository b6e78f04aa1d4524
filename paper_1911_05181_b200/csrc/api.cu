// C-ABI of the library: argument validation, workspace layout, and the stream-ordered sequence of
// kernel launches that makes up one error / gradient evaluation (Section 4.2).
#include "common.cuh"
#include <atomic>
#include <mutex>
#include <new>
#include <vector>

namespace ulsnn {

static std::atomic<int64_t> g_counts[4];
void count_launch(int kind) { g_counts[kind & 3].fetch_add(1, std::memory_order_relaxed); }

namespace {

constexpr int MAX_LAYERS = 16;
constexpr int TIMING_SLOTS = 64;        // per-product timings are kept for this many most recent calls
constexpr int64_t SLICE_CAP = 4096;     // longest run of patterns summed in one fp32 accumulator
constexpr int64_t SLICE_CAP_BF16 = 8192;    // 16-bit mode: the operands' rounding dwarfs the accumulator's, fewer partials to reduce

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }
inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

bool parse_trans(char c, bool* t) {
    if (c == 'N' || c == 'n') { *t = false; return true; }
    if (c == 'T' || c == 't') { *t = true; return true; }
    return false;
}

ulsnn_status_t check_arch() {
    static std::mutex mu;
    static int cached[MAX_DEVICE_SLOTS];          // 0 unknown, 1 ok, 2 unsupported
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ULSNN_ERR_CUDA;
    if (device_cache_slot(dev) < 0) return ULSNN_ERR_UNSUPPORTED_ARCH;
    std::lock_guard<std::mutex> lk(mu);
    if (cached[dev] == 0) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return ULSNN_ERR_CUDA;
        cached[dev] = (major == 10) ? 1 : 2;
    }
    return cached[dev] == 1 ? ULSNN_OK : ULSNN_ERR_UNSUPPORTED_ARCH;
}

// Which engine computes a product asked for in `math`.
bool use_tc(const GemmDesc& d, ulsnn_math_t math) {
    return math != ULSNN_MATH_FP32_SIMT && tc_gemm_supported(d);
}

ulsnn_status_t run_gemm(const GemmDesc& d, ulsnn_math_t math, cudaStream_t stream) {
    if (use_tc(d, math)) return tc_gemm_launch(d, math == ULSNN_MATH_3XTF32, stream);
    return simt_gemm_launch(d, stream);
}

struct SplitPlan { int splits; int64_t k_per_split; };

// Fixed by the shapes only.  Slices are at most SLICE_CAP long once K is large (bounds the fp32 rounding of a
// long sum), and short-and-wide products get enough slices to fill the GPU.
SplitPlan plan_splits(int64_t tiles, int64_t K, int64_t slots, int64_t granule = 32, int64_t cap = SLICE_CAP) {
    int64_t s_acc = (K > 2 * cap) ? (K + cap - 1) / cap : 1;
    int64_t s_fill = 1;
    if (tiles < slots && K >= 1024) {
        s_fill = (2 * slots + tiles - 1) / tiles;
        if (s_fill > K / 512) s_fill = K / 512;
        if (s_fill < 1) s_fill = 1;
    }
    int64_t s = s_acc > s_fill ? s_acc : s_fill;
    int64_t kps = round_up((K + s - 1) / s, granule);
    if (kps < granule) kps = granule;
    s = (K + kps - 1) / kps;
    if (s < 1) s = 1;
    return SplitPlan{(int)s, kps};
}

int64_t slots_of(const GemmDesc& d, bool tc) { return tc ? tc_slots(d) : simt_slots(); }

int64_t tiles_of(const GemmDesc& d, bool tc) {
    const int64_t bm = tc ? tc_tile_m(d) : simt_tile_m();
    const int64_t bn = tc ? tc_tile_n(d) : simt_tile_n();
    return ((d.M + bm - 1) / bm) * ((d.N + bn - 1) / bn);
}

// ------------------------------------------------------------------------------------------- SGEMM

struct SgemmArgs {
    bool ta, tb; int64_t M, N, K; float alpha, beta;
    const float* A; int64_t lda; const float* B; int64_t ldb; float* C; int64_t ldc;
};

ulsnn_status_t validate_sgemm(char transA, char transB, int64_t M, int64_t N, int64_t K,
                              int64_t lda, int64_t ldb, int64_t ldc, bool* ta, bool* tb) {
    if (!parse_trans(transA, ta) || !parse_trans(transB, tb)) return ULSNN_ERR_INVALID_ARG;
    if (M < 0 || N < 0 || K < 0) return ULSNN_ERR_INVALID_ARG;
    const int64_t a_cols = *ta ? M : K, b_cols = *tb ? K : N;
    if (lda < (a_cols > 1 ? a_cols : 1) || ldb < (b_cols > 1 ? b_cols : 1) || ldc < (N > 1 ? N : 1)) return ULSNN_ERR_INVALID_ARG;
    return ULSNN_OK;
}

GemmDesc sgemm_desc(const SgemmArgs& a) {
    GemmDesc d{};
    d.M = a.M; d.N = a.N; d.K = a.K;
    d.A = a.A; d.a_sm = a.ta ? 1 : a.lda; d.a_sk = a.ta ? a.lda : 1;
    d.B = a.B; d.b_sk = a.tb ? 1 : a.ldb; d.b_sn = a.tb ? a.ldb : 1;
    d.C = a.C; d.ldc = a.ldc; d.alpha = a.alpha; d.beta = a.beta;
    d.epi = EPI_SGEMM; d.splits = 1; d.k_per_split = a.K;
    return d;
}

size_t sgemm_ws_for(const GemmDesc& d, bool tc) {
    const SplitPlan p = plan_splits(tiles_of(d, tc), d.K, slots_of(d, tc));
    if (p.splits <= 1) return 0;
    return align256((size_t)p.splits * (size_t)d.M * (size_t)round_up(d.N, 4) * sizeof(float));
}

ulsnn_status_t half_sgemm_impl(const SgemmArgs& a, void* ws, size_t ws_bytes, cudaStream_t stream);

// Re-buffering of operands the tensor-core path cannot address with TMA (Section 3.3 copies B' into a buffer laid out
// for the kernel): an operand whose base is not 16-byte aligned or whose leading dimension is not a multiple of 4 is
// copied into the workspace with its rows padded to a multiple of four floats; the product then runs on the tensor
// cores as for any other operand.  The workspace holds [copy of A][copy of B][split-K partials].
struct PackPlan {
    bool a, b;                      // which operands are copied
    int64_t a_rows, a_cols, lda, b_rows, b_cols, ldb;
    size_t a_bytes, b_bytes;
};

PackPlan pack_plan(const SgemmArgs& a) {
    PackPlan pl{};
    pl.a_rows = a.ta ? a.K : a.M; pl.a_cols = a.ta ? a.M : a.K; pl.lda = round_up(pl.a_cols, 4);
    pl.b_rows = a.tb ? a.N : a.K; pl.b_cols = a.tb ? a.K : a.N; pl.ldb = round_up(pl.b_cols, 4);
    pl.a = !tc_operand_addressable(a.A, a.lda);
    pl.b = !tc_operand_addressable(a.B, a.ldb);
    pl.a_bytes = pl.a ? align256((size_t)pl.a_rows * pl.lda * sizeof(float)) : 0;
    pl.b_bytes = pl.b ? align256((size_t)pl.b_rows * pl.ldb * sizeof(float)) : 0;
    return pl;
}

// the product with its re-buffered operands at `ws`
SgemmArgs packed_args(const SgemmArgs& a, const PackPlan& pl, void* ws) {
    SgemmArgs t = a;
    if (pl.a) { t.A = (const float*)ws; t.lda = pl.lda; }
    if (pl.b) { t.B = (const float*)((char*)ws + pl.a_bytes); t.ldb = pl.ldb; }
    return t;
}

// Scratch the re-buffered tensor-core route needs for these operands (0 when they need no re-buffering or the route
// does not exist for them).
size_t sgemm_packed_need(const SgemmArgs& a, ulsnn_math_t math) {
    if (math != ULSNN_MATH_3XTF32 && math != ULSNN_MATH_TF32) return 0;
    const PackPlan pl = pack_plan(a);
    if (!pl.a && !pl.b) return 0;
    // a stand-in address with the alignment the copies will have
    const SgemmArgs t = packed_args(a, pl, (void*)(uintptr_t)256);
    const GemmDesc d = sgemm_desc(t);
    if (!tc_gemm_supported(d)) return 0;
    return pl.a_bytes + pl.b_bytes + sgemm_ws_for(d, true);
}

ulsnn_status_t sgemm_impl(const SgemmArgs& a_in, ulsnn_math_t math, void* ws, size_t ws_bytes, cudaStream_t stream) {
    if (a_in.M == 0 || a_in.N == 0) return ULSNN_OK;
    if (!a_in.C) return ULSNN_ERR_INVALID_ARG;
    if (a_in.K == 0 || a_in.alpha == 0.f) {
        if (a_in.beta == 1.f) return ULSNN_OK;
        return launch_scale_rows(a_in.C, a_in.M, a_in.N, a_in.ldc, a_in.beta, stream);
    }
    if (!a_in.A || !a_in.B) return ULSNN_ERR_INVALID_ARG;
    if (math == ULSNN_MATH_BF16) return half_sgemm_impl(a_in, ws, ws_bytes, stream);
    SgemmArgs a = a_in;
    if (!use_tc(sgemm_desc(a), math)) {
        // the re-buffered route, when the workspace has room for it; otherwise the FFMA kernel takes the operands as they are
        const size_t need = sgemm_packed_need(a, math);
        if (need > 0 && ws && ws_bytes >= need && ((uintptr_t)ws & 255) == 0) {
            const PackPlan pl = pack_plan(a);
            a = packed_args(a_in, pl, ws);
            ulsnn_status_t st = ULSNN_OK;
            if (pl.a && (st = launch_pack_rows(a_in.A, pl.a_rows, pl.a_cols, a_in.lda, (float*)a.A, pl.lda, stream)) != ULSNN_OK) return st;
            if (pl.b && (st = launch_pack_rows(a_in.B, pl.b_rows, pl.b_cols, a_in.ldb, (float*)a.B, pl.ldb, stream)) != ULSNN_OK) return st;
            ws = (char*)ws + pl.a_bytes + pl.b_bytes;
            ws_bytes -= pl.a_bytes + pl.b_bytes;
        }
    }
    GemmDesc d = sgemm_desc(a);
    const bool tc = use_tc(d, math);
    const SplitPlan p = plan_splits(tiles_of(d, tc), d.K, slots_of(d, tc));
    if (p.splits <= 1) return run_gemm(d, math, stream);
    const int64_t ldp = round_up(d.N, 4);
    const size_t need = (size_t)p.splits * (size_t)d.M * (size_t)ldp * sizeof(float);
    if (!ws || ws_bytes < need) return ULSNN_ERR_WORKSPACE_TOO_SMALL;
    if (((uintptr_t)ws & 255) != 0) return ULSNN_ERR_INVALID_ARG;
    d.epi = EPI_PARTIAL; d.splits = p.splits; d.k_per_split = p.k_per_split;
    d.partials = (float*)ws; d.ldp = ldp;
    ulsnn_status_t st = run_gemm(d, math, stream);
    if (st != ULSNN_OK) return st;
    return launch_splitk_reduce(d.partials, p.splits, d.M, d.N, ldp, a.alpha, a.beta, a.C, a.ldc, nullptr, stream);
}

// 16-bit mode: the operands are first rounded to bfloat16 into the workspace (rows padded to 8 elements), which
// therefore holds [A as bf16][B as bf16][split-K partials].
struct HalfSgemmPlan {
    int64_t a_rows, a_cols, lda, b_rows, b_cols, ldb;
    size_t a_bytes, b_bytes, part_bytes;
    SplitPlan sp; int64_t ldp;
};

HalfGemmDesc half_sgemm_desc(const SgemmArgs& a, const HalfSgemmPlan& pl, const __nv_bfloat16* Ab, const __nv_bfloat16* Bb) {
    HalfGemmDesc d{};
    d.M = a.M; d.N = a.N; d.K = a.K;
    d.A = Ab; d.a_sm = a.ta ? 1 : pl.lda; d.a_sk = a.ta ? pl.lda : 1;
    d.B = Bb; d.b_sk = a.tb ? 1 : pl.ldb; d.b_sn = a.tb ? pl.ldb : 1;
    d.C = a.C; d.ldc = a.ldc; d.alpha = a.alpha; d.beta = a.beta;
    d.epi = EPI_SGEMM; d.splits = 1; d.k_per_split = a.K;
    return d;
}

HalfSgemmPlan half_sgemm_plan(const SgemmArgs& a) {
    HalfSgemmPlan pl{};
    pl.a_rows = a.ta ? a.K : a.M; pl.a_cols = a.ta ? a.M : a.K; pl.lda = round_up(pl.a_cols, 8);
    pl.b_rows = a.tb ? a.N : a.K; pl.b_cols = a.tb ? a.K : a.N; pl.ldb = round_up(pl.b_cols, 8);
    pl.a_bytes = align256((size_t)pl.a_rows * pl.lda * 2);
    pl.b_bytes = align256((size_t)pl.b_rows * pl.ldb * 2);
    const HalfGemmDesc d = half_sgemm_desc(a, pl, nullptr, nullptr);
    const int64_t tiles = ((d.M + hg_tile_m(d) - 1) / hg_tile_m(d)) * ((d.N + hg_tile_n(d) - 1) / hg_tile_n(d));
    pl.sp = plan_splits(tiles, d.K, hg_slots(d), hg_k_granule(), SLICE_CAP_BF16);
    pl.ldp = round_up(d.N, 4);
    pl.part_bytes = pl.sp.splits <= 1 ? 0 : align256((size_t)pl.sp.splits * (size_t)d.M * (size_t)pl.ldp * sizeof(float));
    return pl;
}

ulsnn_status_t half_sgemm_impl(const SgemmArgs& a, void* ws, size_t ws_bytes, cudaStream_t stream) {
    const HalfSgemmPlan pl = half_sgemm_plan(a);
    const size_t need = pl.a_bytes + pl.b_bytes + pl.part_bytes;
    if (!ws || ws_bytes < need) return ULSNN_ERR_WORKSPACE_TOO_SMALL;
    if (((uintptr_t)ws & 255) != 0) return ULSNN_ERR_INVALID_ARG;
    __nv_bfloat16* Ab = (__nv_bfloat16*)ws;
    __nv_bfloat16* Bb = (__nv_bfloat16*)((char*)ws + pl.a_bytes);
    ulsnn_status_t st = launch_to_bf16(a.A, pl.a_rows, pl.a_cols, a.lda, Ab, pl.lda, 0, stream);
    if (st != ULSNN_OK) return st;
    if ((st = launch_to_bf16(a.B, pl.b_rows, pl.b_cols, a.ldb, Bb, pl.ldb, 0, stream)) != ULSNN_OK) return st;
    HalfGemmDesc d = half_sgemm_desc(a, pl, Ab, Bb);
    if (pl.sp.splits <= 1) return hg_gemm_launch(d, stream);
    d.epi = EPI_PARTIAL; d.splits = pl.sp.splits; d.k_per_split = pl.sp.k_per_split;
    d.partials = (float*)((char*)ws + pl.a_bytes + pl.b_bytes); d.ldp = pl.ldp;
    if ((st = hg_gemm_launch(d, stream)) != ULSNN_OK) return st;
    return launch_splitk_reduce(d.partials, pl.sp.splits, d.M, d.N, pl.ldp, a.alpha, a.beta, a.C, a.ldc, nullptr, stream);
}

// scratch a product needs in `math` (operands as given)
size_t sgemm_need(const SgemmArgs& a, ulsnn_math_t math) {
    if (math == ULSNN_MATH_BF16) { const HalfSgemmPlan pl = half_sgemm_plan(a); return pl.a_bytes + pl.b_bytes + pl.part_bytes; }
    const GemmDesc d = sgemm_desc(a);
    return sgemm_ws_for(d, use_tc(d, math));
}

// Scratch of ulsnn_sgemm, one per device.  It only grows, and a buffer that has been handed to a call is never freed
// before the process exits (a larger one is allocated beside it): a product enqueued by another host thread may still
// be reading it.
struct DevScratch { void* p = nullptr; size_t bytes = 0; std::vector<void*> retired; };
DevScratch g_scratch[MAX_DEVICE_SLOTS];
std::mutex g_scratch_mu;

}  // namespace
}  // namespace ulsnn

using namespace ulsnn;

// ----------------------------------------------------------------------------------------------- misc

extern "C" const char* ulsnn_status_string(ulsnn_status_t s) {
    switch (s) {
        case ULSNN_OK: return "ok";
        case ULSNN_ERR_INVALID_ARG: return "invalid argument";
        case ULSNN_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x (B200)";
        case ULSNN_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case ULSNN_ERR_CUDA: return "CUDA runtime error";
        case ULSNN_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case ULSNN_ERR_TOO_LARGE: return "size exceeds a fixed maximum";
    }
    return "unknown status";
}

extern "C" int ulsnn_version(void) { return 109; }

extern "C" void ulsnn_launch_counts(int64_t counts[4]) {
    for (int i = 0; i < 4; ++i) counts[i] = g_counts[i].load(std::memory_order_relaxed);
}

// ----------------------------------------------------------------------------------------------- SGEMM

extern "C" ulsnn_status_t ulsnn_sgemm_workspace_bytes(char transA, char transB, int64_t M, int64_t N, int64_t K,
                                                      ulsnn_math_t math, size_t* bytes) {
    bool ta, tb;
    if (!bytes || !parse_trans(transA, &ta) || !parse_trans(transB, &tb) || M < 0 || N < 0 || K < 0) return ULSNN_ERR_INVALID_ARG;
    if ((int)math < 0 || (int)math > 3) return ULSNN_ERR_INVALID_ARG;
    *bytes = 0;
    if (M == 0 || N == 0 || K == 0) return ULSNN_OK;
    SgemmArgs a{ta, tb, M, N, K, 1.f, 0.f, nullptr, ta ? M : K, nullptr, tb ? K : N, nullptr, N};
    if (math == ULSNN_MATH_BF16) { *bytes = sgemm_need(a, math); return ULSNN_OK; }
    a.lda = round_up(a.lda, 4); a.ldb = round_up(a.ldb, 4);       // an addressable stand-in for the tile-width query
    GemmDesc d = sgemm_desc(a);
    size_t w = sgemm_ws_for(d, false);
    if (math != ULSNN_MATH_FP32_SIMT) { const size_t w2 = sgemm_ws_for(d, true); if (w2 > w) w = w2; }
    *bytes = w;
    return ULSNN_OK;
}

extern "C" ulsnn_status_t ulsnn_sgemm_workspace_bytes_for(char transA, char transB, int64_t M, int64_t N, int64_t K,
                                                          const float* A, int64_t lda, const float* B, int64_t ldb,
                                                          ulsnn_math_t math, size_t* bytes) {
    SgemmArgs a{false, false, M, N, K, 1.f, 0.f, A, lda, B, ldb, nullptr, N > 1 ? N : 1};
    if (!bytes) return ULSNN_ERR_INVALID_ARG;
    ulsnn_status_t st = validate_sgemm(transA, transB, M, N, K, lda, ldb, a.ldc, &a.ta, &a.tb);
    if (st != ULSNN_OK) return st;
    if ((int)math < 0 || (int)math > 3) return ULSNN_ERR_INVALID_ARG;
    *bytes = 0;
    if (M == 0 || N == 0 || K == 0) return ULSNN_OK;
    size_t w = sgemm_need(a, math);
    const size_t packed = sgemm_packed_need(a, math);
    if (packed > w) w = packed;
    *bytes = w;
    return ULSNN_OK;
}

extern "C" ulsnn_status_t ulsnn_sgemm_ex(char transA, char transB, int64_t M, int64_t N, int64_t K, float alpha,
                                         const float* A, int64_t lda, const float* B, int64_t ldb,
                                         float beta, float* C, int64_t ldc, ulsnn_math_t math,
                                         void* workspace, size_t workspace_bytes, ulsnn_stream_t stream) {
    SgemmArgs a{false, false, M, N, K, alpha, beta, A, lda, B, ldb, C, ldc};
    ulsnn_status_t st = validate_sgemm(transA, transB, M, N, K, lda, ldb, ldc, &a.ta, &a.tb);
    if (st != ULSNN_OK) return st;
    if ((int)math < 0 || (int)math > 3) return ULSNN_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return ULSNN_OK;
    if ((st = check_arch()) != ULSNN_OK) return st;
    return sgemm_impl(a, math, workspace, workspace_bytes, (cudaStream_t)stream);
}

extern "C" ulsnn_status_t ulsnn_sgemm(char transA, char transB, int64_t M, int64_t N, int64_t K, float alpha,
                                      const float* A, int64_t lda, const float* B, int64_t ldb,
                                      float beta, float* C, int64_t ldc, ulsnn_stream_t stream) {
    SgemmArgs a{false, false, M, N, K, alpha, beta, A, lda, B, ldb, C, ldc};
    ulsnn_status_t st = validate_sgemm(transA, transB, M, N, K, lda, ldb, ldc, &a.ta, &a.tb);
    if (st != ULSNN_OK) return st;
    if (M == 0 || N == 0) return ULSNN_OK;
    if ((st = check_arch()) != ULSNN_OK) return st;
    void* ws = nullptr; size_t have = 0;
    if (K > 0 && alpha != 0.f && A && B && C) {
        GemmDesc d = sgemm_desc(a);
        size_t need = sgemm_ws_for(d, use_tc(d, ULSNN_MATH_3XTF32));
        const size_t packed = sgemm_packed_need(a, ULSNN_MATH_3XTF32);
        if (packed > need) need = packed;
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || device_cache_slot(dev) < 0) return ULSNN_ERR_CUDA;
        std::lock_guard<std::mutex> lk(g_scratch_mu);
        DevScratch& sc = g_scratch[device_cache_slot(dev)];
        if (need > sc.bytes) {
            void* bigger = nullptr;
            if (cudaMalloc(&bigger, need) != cudaSuccess) return ULSNN_ERR_CUDA;
            if (sc.p) sc.retired.push_back(sc.p);
            sc.p = bigger; sc.bytes = need;
        }
        ws = sc.p; have = sc.bytes;
    }
    return sgemm_impl(a, ULSNN_MATH_3XTF32, ws, have, (cudaStream_t)stream);
}

// ----------------------------------------------------------------------------------------------- SGEMM without allocation

// Split-K scratch of ulsnn_sgemm_noalloc.  It lives in the library's image: every device that loads the library
// holds these bytes until the process exits, which is why the size is kept modest.
#define ULSNN_NOALLOC_SCRATCH_BYTES (8u << 20)
static __device__ __align__(256) unsigned char g_noalloc_scratch[ULSNN_NOALLOC_SCRATCH_BYTES];

namespace ulsnn {
namespace {
// In host code `g_noalloc_scratch` is only a handle of the symbol; the address a kernel can use has to be asked for,
// per device, with that device current.
std::mutex g_noalloc_mu;
void* g_noalloc_ptr[MAX_DEVICE_SLOTS];

ulsnn_status_t noalloc_scratch(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || device_cache_slot(dev) < 0) return ULSNN_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_noalloc_mu);
    if (!g_noalloc_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return ULSNN_ERR_CUDA;
        g_noalloc_ptr[dev] = p;
    }
    *out = g_noalloc_ptr[dev];
    return ULSNN_OK;
}
}  // namespace
}  // namespace ulsnn

extern "C" size_t ulsnn_sgemm_noalloc_max_scratch_bytes(void) { return (size_t)ULSNN_NOALLOC_SCRATCH_BYTES; }

extern "C" ulsnn_status_t ulsnn_sgemm_noalloc(char transA, char transB, int64_t M, int64_t N, int64_t K, float alpha,
                                              const float* A, int64_t lda, const float* B, int64_t ldb,
                                              float beta, float* C, int64_t ldc, ulsnn_math_t math,
                                              ulsnn_stream_t stream) {
    SgemmArgs a{false, false, M, N, K, alpha, beta, A, lda, B, ldb, C, ldc};
    ulsnn_status_t st = validate_sgemm(transA, transB, M, N, K, lda, ldb, ldc, &a.ta, &a.tb);
    if (st != ULSNN_OK) return st;
    if ((int)math < 0 || (int)math > 3) return ULSNN_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return ULSNN_OK;
    size_t need = 0;
    if (K > 0 && alpha != 0.f && A && B && C) {
        // the same route and slice plan as ulsnn_sgemm_ex takes for these operands when it is given the workspace
        // ulsnn_sgemm_workspace_bytes_for asks for, so the two give the same bits: operands TMA cannot address are
        // re-buffered in the array when copies and partials fit, and go to the FFMA kernel when they do not
        need = sgemm_need(a, math);
        const size_t packed = sgemm_packed_need(a, math);
        if (packed > need && packed <= (size_t)ULSNN_NOALLOC_SCRATCH_BYTES) need = packed;
    }
    if (need > (size_t)ULSNN_NOALLOC_SCRATCH_BYTES) return ULSNN_ERR_TOO_LARGE;
    if ((st = check_arch()) != ULSNN_OK) return st;
    void* ws = nullptr;
    if (need > 0 && (st = noalloc_scratch(&ws)) != ULSNN_OK) return st;
    // Every slice writes all the entries of its partial product that the reduction reads, so the scratch needs
    // no clearing although it still holds what the previous call left there.
    return sgemm_impl(a, math, ws, need, (cudaStream_t)stream);
}

// ----------------------------------------------------------------------------------------------- network

struct ulsnn_mlp {
    int L;
    int32_t sizes[MAX_LAYERS + 1];
    ulsnn_math_t math;
    int64_t max_patterns;
    // strides of the library-owned matrices
    int64_t ldh[MAX_LAYERS + 1];    // H_l (output of weight l-1, l = 1..L-1): sizes[l] + a ones column, padded to 4
    int64_t ldd[MAX_LAYERS + 1];    // delta_l, l = 1..L-1
    int64_t ldz;                    // logits
    int64_t stats_ld;
    // workspace carve-up
    float* H[MAX_LAYERS + 1];
    float* Hlo[MAX_LAYERS + 1];     // 3xTF32: H_l is kept as a pair, H = tf32_rn(h) and Hlo the rounded remainder
    float* Whi[MAX_LAYERS];         // 3xTF32: the same pair for every weight matrix, rebuilt at the start of a call
    float* Wlo[MAX_LAYERS];
    float* D[MAX_LAYERS + 1];
    float* Z;
    float* Zlo;                     // 3xTF32, squared-error head: lo half of the output deltas (Z holds the hi half)
    float2* stats;
    float* lse;
    float* chunk_tab; int64_t chunk_ld;     // per pattern and 32-class chunk: chunk maximum, then the factor exp(m - lse)
    float* zlabel;
    double* loss_parts;
    float* colsum_parts;
    float* partials;
    size_t partials_bytes;
    size_t total_bytes;
    // 16-bit mode: bfloat16 copies of the batch and the weights (rebuilt every call), activations, deltas and stored
    // exponentials.  Activation rows (the batch included) end in a ones column, so that every bias gradient is a
    // column of a weight-gradient product.
    __nv_bfloat16* Xb; int64_t ldxb;
    __nv_bfloat16* Wb[MAX_LAYERS]; int64_t ldwb[MAX_LAYERS];
    __nv_bfloat16* Hb[MAX_LAYERS + 1]; int64_t ldhb[MAX_LAYERS + 1];
    __nv_bfloat16* Db[MAX_LAYERS + 1]; int64_t lddb[MAX_LAYERS + 1];
    __nv_bfloat16* Eb; int64_t ldeb;
    // optional: events recorded when the gradient of a weight matrix (dW_w and db_w) is final
    cudaEvent_t grad_done[MAX_LAYERS];
    bool have_grad_events;
    // optional per-product timing
    bool timing;
    int n_phases;                       // products launched so far by the call in flight
    int64_t timed_calls;                // calls recorded since timing was switched on
    std::vector<cudaEvent_t> ev;        // [TIMING_SLOTS][3*MAX_LAYERS][2], slot = call index modulo TIMING_SLOTS
    int64_t phase_mnk[3 * (3 * MAX_LAYERS)];
};

namespace {

// Upper bound, over every batch length n <= B, of the split-K scratch for dW_w: M = sizes[w+1], N = sizes[w]
// (+1 ones column when w >= 1).  plan_splits never returns more than max(ceil(n/SLICE_CAP), fill slices), and
// both terms grow with n.
size_t wgrad_partial_bound(const int32_t* sizes, int w, int64_t B) {
    GemmDesc d{};
    d.M = sizes[w + 1]; d.N = sizes[w] + (w >= 1 ? 1 : 0); d.K = B;
    d.a_sm = 1; d.a_sk = 4; d.b_sk = 4; d.b_sn = 1;
    const int64_t ldp = round_up(d.N, 4);
    int64_t smax = (B + SLICE_CAP - 1) / SLICE_CAP;
    for (int tc = 0; tc < 2; ++tc) {
        const int64_t tiles = tiles_of(d, tc != 0), slots = slots_of(d, tc != 0);
        if (tiles < slots && B >= 1024) {
            int64_t f = (2 * slots + tiles - 1) / tiles;
            if (f > B / 512) f = B / 512;
            if (f > smax) smax = f;
        }
    }
    if (smax < 1) smax = 1;
    return (size_t)smax * (size_t)d.M * (size_t)ldp * sizeof(float);
}

// 16-bit mode: split-K scratch bound for dW_w, M = sizes[w+1], N = sizes[w] + 1 (ones column), any n <= B
size_t wgrad_partial_bound_bf16(const int32_t* sizes, int w, int64_t B) {
    HalfGemmDesc d{};
    d.M = sizes[w + 1]; d.N = sizes[w] + 1; d.K = B;
    d.a_sm = 1; d.a_sk = 8; d.b_sk = 8; d.b_sn = 1;
    const int64_t ldp = round_up(d.N, 4);
    int64_t smax = (B + SLICE_CAP_BF16 - 1) / SLICE_CAP_BF16;
    const int64_t tiles = ((d.M + hg_tile_m(d) - 1) / hg_tile_m(d)) * ((d.N + hg_tile_n(d) - 1) / hg_tile_n(d));
    const int64_t slots = hg_slots(d);
    if (tiles < slots && B >= 1024) {
        int64_t f = (2 * slots + tiles - 1) / tiles;
        if (f > B / 512) f = B / 512;
        if (f > smax) smax = f;
    }
    if (smax < 1) smax = 1;
    return (size_t)smax * (size_t)d.M * (size_t)ldp * sizeof(float);
}

ulsnn_status_t layout_bf16(ulsnn_mlp* h, char* base) {
    const int L = h->L; const int64_t B = h->max_patterns;
    size_t off = 0;
    auto take = [&](size_t bytes) { char* p = base ? base + off : nullptr; off += align256(bytes); return p; };
    h->ldxb = round_up((int64_t)h->sizes[0] + 1, 8);
    h->Xb = (__nv_bfloat16*)take((size_t)B * h->ldxb * 2);
    for (int l = 1; l < L; ++l) {
        h->ldhb[l] = round_up((int64_t)h->sizes[l] + 1, 8);
        h->lddb[l] = round_up((int64_t)h->sizes[l], 8);
        h->Hb[l] = (__nv_bfloat16*)take((size_t)B * h->ldhb[l] * 2);
        h->Db[l] = (__nv_bfloat16*)take((size_t)B * h->lddb[l] * 2);
    }
    for (int l = 0; l < L; ++l) {
        h->ldwb[l] = round_up((int64_t)h->sizes[l], 8);
        h->Wb[l] = (__nv_bfloat16*)take((size_t)h->sizes[l + 1] * h->ldwb[l] * 2);
    }
    h->ldeb = round_up((int64_t)h->sizes[L], 8);
    h->Eb = (__nv_bfloat16*)take((size_t)B * h->ldeb * 2);
    h->stats_ld = 2 * (((int64_t)h->sizes[L] + 63) / 64);       // two entries per column tile, tiles at least 64 wide
    h->stats = (float2*)take((size_t)B * h->stats_ld * sizeof(float2));
    h->lse = (float*)take((size_t)B * sizeof(float));
    h->chunk_ld = round_up(((int64_t)h->sizes[L] + 31) / 32, 8);
    h->chunk_tab = (float*)take((size_t)B * h->chunk_ld * sizeof(float));
    h->zlabel = (float*)take((size_t)B * sizeof(float));
    h->loss_parts = (double*)take((size_t)(rowstats_blocks(B) + 1) * sizeof(double));
    size_t pb = 0;
    for (int w = 0; w < L; ++w) { const size_t b = wgrad_partial_bound_bf16(h->sizes, w, B); if (b > pb) pb = b; }
    h->partials_bytes = align256(pb);
    h->partials = (float*)take(pb);
    h->total_bytes = off;
    return ULSNN_OK;
}

ulsnn_status_t layout(ulsnn_mlp* h, char* base) {
    if (h->math == ULSNN_MATH_BF16) return layout_bf16(h, base);
    const int L = h->L; const int64_t B = h->max_patterns;
    size_t off = 0;
    auto take = [&](size_t bytes) { char* p = base ? base + off : nullptr; off += align256(bytes); return p; };
    for (int l = 1; l < L; ++l) {
        h->ldh[l] = round_up((int64_t)h->sizes[l] + 1, 4);
        h->ldd[l] = round_up((int64_t)h->sizes[l], 4);
        h->H[l] = (float*)take((size_t)B * h->ldh[l] * sizeof(float));
        h->Hlo[l] = (h->math == ULSNN_MATH_3XTF32) ? (float*)take((size_t)B * h->ldh[l] * sizeof(float)) : nullptr;
        h->D[l] = (float*)take((size_t)B * h->ldd[l] * sizeof(float));
    }
    for (int l = 0; l < L; ++l) {
        const size_t wbytes = (size_t)h->sizes[l] * h->sizes[l + 1] * sizeof(float);
        h->Whi[l] = (h->math == ULSNN_MATH_3XTF32) ? (float*)take(wbytes) : nullptr;
        h->Wlo[l] = (h->math == ULSNN_MATH_3XTF32) ? (float*)take(wbytes) : nullptr;
    }
    h->ldz = round_up((int64_t)h->sizes[L], 4);
    h->Z = (float*)take((size_t)B * h->ldz * sizeof(float));
    h->Zlo = (h->math == ULSNN_MATH_3XTF32) ? (float*)take((size_t)B * h->ldz * sizeof(float)) : nullptr;
    h->stats_ld = ((int64_t)h->sizes[L] + 63) / 64;          // enough for any column-tile width >= 64
    h->stats = (float2*)take((size_t)B * h->stats_ld * sizeof(float2));
    h->lse = (float*)take((size_t)B * sizeof(float));
    h->chunk_ld = round_up(((int64_t)h->sizes[L] + 31) / 32, 8);      // whole 256-column tiles: the epilogue writes eight at a time
    h->chunk_tab = (float*)take((size_t)B * h->chunk_ld * sizeof(float));
    h->zlabel = (float*)take((size_t)B * sizeof(float));
    h->loss_parts = (double*)take((size_t)(rowstats_blocks(B) + 1) * sizeof(double));
    size_t cs = 0;
    if (L >= 2) cs = (size_t)((B + 127) / 128) * 4 * (size_t)h->sizes[1] * sizeof(float);
    else cs = (size_t)delta_colsum_tiles(B) * (size_t)h->sizes[1] * sizeof(float);
    h->colsum_parts = (float*)take(cs);
    size_t pb = 0;
    for (int w = 0; w < L; ++w) { const size_t b = wgrad_partial_bound(h->sizes, w, B); if (b > pb) pb = b; }
    h->partials_bytes = align256(pb);
    h->partials = (float*)take(pb);
    h->total_bytes = off;
    return ULSNN_OK;
}

ulsnn_status_t check_desc(const ulsnn_mlp_desc_t* d) {
    if (!d || !d->sizes || d->n_layers < 1 || d->n_layers > MAX_LAYERS || d->max_patterns < 1) return ULSNN_ERR_INVALID_ARG;
    if ((int)d->math < 0 || (int)d->math > 3) return ULSNN_ERR_INVALID_ARG;
    for (int l = 0; l <= d->n_layers; ++l) if (d->sizes[l] < 1 || d->sizes[l] > (1 << 20)) return ULSNN_ERR_INVALID_ARG;
    if (d->max_patterns > ((int64_t)1 << 31) - 256) return ULSNN_ERR_TOO_LARGE;
    return ULSNN_OK;
}

void fill_handle(ulsnn_mlp* h, const ulsnn_mlp_desc_t* d) {
    *h = ulsnn_mlp{};
    h->L = d->n_layers; h->math = d->math; h->max_patterns = d->max_patterns;
    for (int l = 0; l <= h->L; ++l) h->sizes[l] = d->sizes[l];
}

// B operand = weight matrix w (strides already set): the stored (hi, lo) pair where the tensor-core engine can take
// it, the caller's matrix otherwise (the FFMA engine multiplies exact fp32 values anyway)
void set_weight_operand(ulsnn_mlp* h, GemmDesc& d, const float* const* W, int w) {
    d.B = W[w]; d.B_lo = nullptr;
    if (h->math == ULSNN_MATH_3XTF32) {
        GemmDesc t = d;
        t.B = h->Whi[w]; t.B_lo = h->Wlo[w];
        if (tc_gemm_supported(t)) d = t;
    }
}

// a product's launch bracketed by events when the handle's timing is on
template <class Launch>
ulsnn_status_t timed_product(ulsnn_mlp* h, int64_t M, int64_t N, int64_t K, cudaStream_t stream, Launch launch) {
    if (!h->timing || h->n_phases >= 3 * MAX_LAYERS) return launch();
    const int i = h->n_phases++;
    h->phase_mnk[3 * i] = M; h->phase_mnk[3 * i + 1] = N; h->phase_mnk[3 * i + 2] = K;
    const size_t slot = (size_t)((h->timed_calls - 1) % TIMING_SLOTS);
    cudaEvent_t* e = &h->ev[(slot * 3 * MAX_LAYERS + i) * 2];
    if (cudaEventRecord(e[0], stream) != cudaSuccess) return ULSNN_ERR_CUDA;
    ulsnn_status_t st = launch();
    if (cudaEventRecord(e[1], stream) != cudaSuccess) return ULSNN_ERR_CUDA;
    return st;
}
ulsnn_status_t timed_gemm(ulsnn_mlp* h, const GemmDesc& d, cudaStream_t stream) {
    return timed_product(h, d.M, d.N, d.K, stream, [&] { return run_gemm(d, h->math, stream); });
}
ulsnn_status_t timed_gemm(ulsnn_mlp* h, const HalfGemmDesc& d, cudaStream_t stream) {
    return timed_product(h, d.M, d.N, d.K, stream, [&] { return hg_gemm_launch(d, stream); });
}

// dW_w and db_w of this call are final on the stream: tell whoever waits for them (the gradient exchange between
// several GPUs starts on a layer's gradient while the products of the layers below still run)
ulsnn_status_t mark_gradient_done(ulsnn_mlp* h, int w, cudaStream_t stream) {
    if (!h->have_grad_events || !h->grad_done[w]) return ULSNN_OK;
    return cuda_ok(cudaEventRecord(h->grad_done[w], stream));
}

// The forward products: hidden layers with bias + tanh fused, then the logits with their row statistics.
// What the outputs are compared with: integer labels (softmax + cross-entropy) or, when T is not null, a dense
// target matrix (the paper's tanh outputs with summed squared error, Eqs. 1 and 3).
struct Targets { const int32_t* labels; const float* T; int64_t ldt; };

ulsnn_status_t forward(ulsnn_mlp* h, const float* const* W, const float* const* b, const float* X, int64_t ldx,
                       const Targets& tg, int64_t n, bool keep_logits, int accumulate, double* loss_out,
                       cudaStream_t stream) {
    const int32_t* labels = tg.labels;
    const int L = h->L;
    h->n_phases = 0;
    if (h->timing) h->timed_calls++;
    // 3xTF32: every weight matrix is split once per call into its TF32 (hi, lo) pair, and the activations are
    // written as such pairs, so that the products which read them need no operand pass for them
    const bool pairs = h->math == ULSNN_MATH_3XTF32;
    if (pairs) {
        for (int l = 0; l < L; ++l) {
            ulsnn_status_t st = launch_split_hilo(W[l], (int64_t)h->sizes[l] * h->sizes[l + 1], h->Whi[l], h->Wlo[l], stream);
            if (st != ULSNN_OK) return st;
        }
    }
    const float* in = X; const float* in_lo = nullptr; int64_t ld_in = ldx;
    for (int l = 1; l < L; ++l) {
        GemmDesc d{};
        d.M = n; d.N = h->sizes[l]; d.K = h->sizes[l - 1];
        d.A = in; d.A_lo = in_lo; d.a_sm = ld_in; d.a_sk = 1;
        d.b_sk = 1; d.b_sn = d.K;
        set_weight_operand(h, d, W, l - 1);
        d.C = h->H[l]; d.C_lo = pairs ? h->Hlo[l] : nullptr; d.ldc = h->ldh[l]; d.alpha = 1.f; d.beta = 0.f;
        d.epi = EPI_BIAS_TANH; d.bias = b[l - 1]; d.ones_cols = (int)(h->ldh[l] - d.N);
        d.splits = 1; d.k_per_split = d.K;
        ulsnn_status_t st = timed_gemm(h, d, stream);
        if (st != ULSNN_OK) return st;
        in = h->H[l]; in_lo = d.C_lo; ld_in = h->ldh[l];
    }
    GemmDesc d{};
    d.M = n; d.N = h->sizes[L]; d.K = h->sizes[L - 1];
    d.A = in; d.A_lo = in_lo; d.a_sm = ld_in; d.a_sk = 1;
    d.b_sk = 1; d.b_sn = d.K;
    set_weight_operand(h, d, W, L - 1);
    d.C = keep_logits ? h->Z : nullptr; d.ldc = h->ldz; d.alpha = 1.f; d.beta = 0.f;
    d.epi = EPI_LOGITS; d.bias = b[L - 1]; d.labels = labels;
    if (tg.T) {         // the output deltas dE/dz go where the logits would, as a pair in 3xTF32 mode
        d.epi = EPI_TANH_SSE; d.T = tg.T; d.ldt = tg.ldt;
        d.C_lo = keep_logits ? h->Zlo : nullptr;
    }
    d.stats = h->stats; d.stats_ld = h->stats_ld; d.zlabel = h->zlabel;
    d.chunk_max = (keep_logits && !tg.T) ? h->chunk_tab : nullptr; d.chunk_ld = h->chunk_ld;
    d.splits = 1; d.k_per_split = d.K;
    const bool tc = use_tc(d, h->math);
    const int64_t bn = tc ? tc_tile_n(d) : simt_tile_n();
    const int tiles = (int)((d.N + bn - 1) / bn);
    if (tiles > h->stats_ld) return ULSNN_ERR_WORKSPACE_TOO_SMALL;
    ulsnn_status_t st = timed_gemm(h, d, stream);
    if (st != ULSNN_OK) return st;
    if (tg.T) return launch_rowsums(h->stats, h->stats_ld, tiles, n, h->loss_parts, accumulate, loss_out, stream);
    return launch_rowstats(h->stats, h->stats_ld, tiles, h->zlabel, n, h->lse, d.chunk_max, h->chunk_ld,
                           (int)(((int64_t)h->sizes[L] + 31) / 32), h->loss_parts, accumulate, loss_out, stream);
}

// ---- 16-bit mode (softmax head).  The batch and the weights are rounded to bfloat16 first; every product then reads
// and writes bfloat16 (fp32 accumulators, fp32 statistics, loss and gradients).
ulsnn_status_t forward_bf16(ulsnn_mlp* h, const float* const* W, const float* const* b, const float* X, int64_t ldx,
                            const Targets& tg, int64_t n, bool keep, int accumulate, double* loss_out, cudaStream_t stream) {
    const int L = h->L;
    const int32_t* labels = tg.labels;
    h->n_phases = 0;
    if (h->timing) h->timed_calls++;
    ulsnn_status_t st = launch_to_bf16(X, n, h->sizes[0], ldx, h->Xb, h->ldxb, 1, stream);
    if (st != ULSNN_OK) return st;
    for (int l = 0; l < L; ++l)
        if ((st = launch_to_bf16(W[l], h->sizes[l + 1], h->sizes[l], h->sizes[l], h->Wb[l], h->ldwb[l], 0, stream)) != ULSNN_OK) return st;
    const __nv_bfloat16* in = h->Xb; int64_t ld_in = h->ldxb;
    for (int l = 1; l < L; ++l) {
        HalfGemmDesc d{};
        d.M = n; d.N = h->sizes[l]; d.K = h->sizes[l - 1];
        d.A = in; d.a_sm = ld_in; d.a_sk = 1;
        d.B = h->Wb[l - 1]; d.b_sk = 1; d.b_sn = h->ldwb[l - 1];
        d.Ch = h->Hb[l]; d.ldch = h->ldhb[l];
        d.epi = EPI_BIAS_TANH; d.bias = b[l - 1]; d.ones_cols = (int)(h->ldhb[l] - d.N);
        d.splits = 1; d.k_per_split = d.K;
        if ((st = timed_gemm(h, d, stream)) != ULSNN_OK) return st;
        in = h->Hb[l]; ld_in = h->ldhb[l];
    }
    HalfGemmDesc d{};
    d.M = n; d.N = h->sizes[L]; d.K = h->sizes[L - 1];
    d.A = in; d.a_sm = ld_in; d.a_sk = 1;
    d.B = h->Wb[L - 1]; d.b_sk = 1; d.b_sn = h->ldwb[L - 1];
    d.Ch = keep ? h->Eb : nullptr; d.ldch = h->ldeb;
    d.epi = EPI_LOGITS; d.bias = b[L - 1]; d.labels = labels;
    d.stats = h->stats; d.stats_ld = h->stats_ld; d.zlabel = h->zlabel;
    d.chunk_max = (keep && !tg.T) ? h->chunk_tab : nullptr; d.chunk_ld = h->chunk_ld;
    if (tg.T) { d.epi = EPI_TANH_SSE; d.T = tg.T; d.ldt = tg.ldt; }     // the output deltas dE/dz go where the exponentials would
    d.splits = 1; d.k_per_split = d.K;
    const int entries = 2 * (int)((d.N + hg_tile_n(d) - 1) / hg_tile_n(d));
    if (entries > h->stats_ld) return ULSNN_ERR_WORKSPACE_TOO_SMALL;
    if ((st = timed_gemm(h, d, stream)) != ULSNN_OK) return st;
    if (tg.T) return launch_rowsums(h->stats, h->stats_ld, entries, n, h->loss_parts, accumulate, loss_out, stream);
    return launch_rowstats(h->stats, h->stats_ld, entries, h->zlabel, n, h->lse, d.chunk_max, h->chunk_ld,
                           (int)(((int64_t)h->sizes[L] + 31) / 32), h->loss_parts, accumulate, loss_out, stream);
}

ulsnn_status_t gradient_bf16(ulsnn_mlp* h, const float* const* W, const float* const* b, const float* X, int64_t ldx,
                             const Targets& tg, int64_t n, int accumulate, float* const* dW, float* const* db,
                             double* loss_out, cudaStream_t stream) {
    const int L = h->L;
    ulsnn_status_t st = forward_bf16(h, W, b, X, ldx, tg, n, true, accumulate, loss_out, stream);
    if (st != ULSNN_OK) return st;
    // softmax head: delta_L = softmax - onehot, in place over the stored exponentials (the squared-error epilogue has
    // written its deltas already)
    if (!tg.T && (st = launch_delta_bf16(h->Eb, h->ldeb, h->chunk_tab, h->chunk_ld, tg.labels, n, h->sizes[L], stream)) != ULSNN_OK) return st;
    // delta_l = (1 - H_l*H_l) * (delta_{l+1} W_{l+1})   (H_D of Section 4.2)
    for (int l = L - 1; l >= 1; --l) {
        HalfGemmDesc d{};
        d.M = n; d.N = h->sizes[l]; d.K = h->sizes[l + 1];
        if (l + 1 == L) { d.A = h->Eb; d.a_sm = h->ldeb; } else { d.A = h->Db[l + 1]; d.a_sm = h->lddb[l + 1]; }
        d.a_sk = 1;
        d.B = h->Wb[l]; d.b_sk = h->ldwb[l]; d.b_sn = 1;
        d.Ch = h->Db[l]; d.ldch = h->lddb[l];
        d.epi = EPI_TANHP; d.Hm = h->Hb[l]; d.ldh = h->ldhb[l];
        d.splits = 1; d.k_per_split = d.K;
        if ((st = timed_gemm(h, d, stream)) != ULSNN_OK) return st;
    }
    // dW_w = delta_{w+1}^T [act_w | 1]: the last column is db_w
    const float beta = accumulate ? 1.f : 0.f;
    for (int w = L - 1; w >= 0; --w) {
        HalfGemmDesc d{};
        d.M = h->sizes[w + 1]; d.N = h->sizes[w] + 1; d.K = n;
        if (w + 1 == L) { d.A = h->Eb; d.a_sk = h->ldeb; } else { d.A = h->Db[w + 1]; d.a_sk = h->lddb[w + 1]; }
        d.a_sm = 1;
        if (w >= 1) { d.B = h->Hb[w]; d.b_sk = h->ldhb[w]; } else { d.B = h->Xb; d.b_sk = h->ldxb; }
        d.b_sn = 1;
        d.epi = EPI_PARTIAL;
        const int64_t tiles = ((d.M + hg_tile_m(d) - 1) / hg_tile_m(d)) * ((d.N + hg_tile_n(d) - 1) / hg_tile_n(d));
        const SplitPlan p = plan_splits(tiles, d.K, hg_slots(d), hg_k_granule(), SLICE_CAP_BF16);
        d.splits = p.splits; d.k_per_split = p.k_per_split;
        d.ldp = round_up(d.N, 4); d.partials = h->partials;
        if ((size_t)p.splits * (size_t)d.M * (size_t)d.ldp * sizeof(float) > h->partials_bytes) return ULSNN_ERR_WORKSPACE_TOO_SMALL;
        if ((st = timed_gemm(h, d, stream)) != ULSNN_OK) return st;
        if ((st = launch_splitk_reduce(d.partials, p.splits, d.M, h->sizes[w], d.ldp, 1.f, beta, dW[w], h->sizes[w], db[w], stream)) != ULSNN_OK) return st;
        if ((st = mark_gradient_done(h, w, stream)) != ULSNN_OK) return st;
    }
    return ULSNN_OK;
}

ulsnn_status_t check_call(ulsnn_mlp* h, const float* const* W, const float* const* b, const float* X, int64_t ldx,
                          const void* targets, int64_t n, double* loss_out) {
    if (!h || !W || !b || !loss_out || n < 0 || n > h->max_patterns) return ULSNN_ERR_INVALID_ARG;
    if (n > 0 && (!X || !targets || ldx < h->sizes[0])) return ULSNN_ERR_INVALID_ARG;
    for (int l = 0; l < h->L; ++l) if (!W[l] || !b[l]) return ULSNN_ERR_INVALID_ARG;
    return ULSNN_OK;
}

}  // namespace

extern "C" ulsnn_status_t ulsnn_mlp_workspace_bytes(const ulsnn_mlp_desc_t* desc, size_t* bytes) {
    ulsnn_status_t st = check_desc(desc);
    if (st != ULSNN_OK || !bytes) return st != ULSNN_OK ? st : ULSNN_ERR_INVALID_ARG;
    ulsnn_mlp tmp; fill_handle(&tmp, desc);
    layout(&tmp, nullptr);
    *bytes = tmp.total_bytes;
    return ULSNN_OK;
}

extern "C" ulsnn_status_t ulsnn_mlp_create(ulsnn_mlp_t** handle, const ulsnn_mlp_desc_t* desc, void* workspace, size_t workspace_bytes) {
    if (!handle) return ULSNN_ERR_INVALID_ARG;
    *handle = nullptr;
    ulsnn_status_t st = check_desc(desc);
    if (st != ULSNN_OK) return st;
    if (!workspace || ((uintptr_t)workspace & 255) != 0) return ULSNN_ERR_INVALID_ARG;
    ulsnn_mlp* h = new (std::nothrow) ulsnn_mlp;
    if (!h) return ULSNN_ERR_CUDA;
    fill_handle(h, desc);
    layout(h, (char*)workspace);
    if (h->total_bytes > workspace_bytes) { delete h; return ULSNN_ERR_WORKSPACE_TOO_SMALL; }
    *handle = h;
    return ULSNN_OK;
}

extern "C" void ulsnn_mlp_destroy(ulsnn_mlp_t* handle) {
    if (!handle) return;
    for (cudaEvent_t e : handle->ev) if (e) cudaEventDestroy(e);
    delete handle;
}

extern "C" ulsnn_status_t ulsnn_mlp_set_gradient_events(ulsnn_mlp_t* h, void* const* events) {
    if (!h) return ULSNN_ERR_INVALID_ARG;
    h->have_grad_events = false;
    for (int w = 0; w < MAX_LAYERS; ++w) h->grad_done[w] = nullptr;
    if (!events) return ULSNN_OK;
    for (int w = 0; w < h->L; ++w) {
        h->grad_done[w] = (cudaEvent_t)events[w];
        if (events[w]) h->have_grad_events = true;
    }
    return ULSNN_OK;
}

extern "C" ulsnn_status_t ulsnn_mlp_enable_timing(ulsnn_mlp_t* h, int on) {
    if (!h) return ULSNN_ERR_INVALID_ARG;
    if (on && h->ev.empty()) {
        h->ev.assign((size_t)TIMING_SLOTS * 3 * MAX_LAYERS * 2, nullptr);
        const size_t used = (size_t)(3 * h->L - 1) * 2;
        for (int slot = 0; slot < TIMING_SLOTS; ++slot)
            for (size_t i = 0; i < used; ++i)
                if (cudaEventCreate(&h->ev[(size_t)slot * 3 * MAX_LAYERS * 2 + i]) != cudaSuccess) return ULSNN_ERR_CUDA;
    }
    h->timing = on != 0;
    h->n_phases = 0;
    h->timed_calls = 0;
    return ULSNN_OK;
}

extern "C" ulsnn_status_t ulsnn_mlp_phase_times(ulsnn_mlp_t* h, int* n, float* ms, int64_t* mnk) {
    if (!h || !n || !ms || !mnk || *n < 0) return ULSNN_ERR_INVALID_ARG;
    const int cap = *n;
    *n = 0;
    if (!h->timing || h->timed_calls == 0) return ULSNN_OK;
    const int cnt = h->n_phases < cap ? h->n_phases : cap;
    const int64_t calls = h->timed_calls < TIMING_SLOTS ? h->timed_calls : TIMING_SLOTS;
    for (int i = 0; i < cnt; ++i) {
        double sum = 0.0;
        for (int64_t c = 0; c < calls; ++c) {
            const size_t slot = (size_t)((h->timed_calls - 1 - c) % TIMING_SLOTS);
            cudaEvent_t* e = &h->ev[(slot * 3 * MAX_LAYERS + i) * 2];
            float t = 0.f;
            if (cudaEventSynchronize(e[1]) != cudaSuccess) return ULSNN_ERR_CUDA;
            if (cudaEventElapsedTime(&t, e[0], e[1]) != cudaSuccess) return ULSNN_ERR_CUDA;
            sum += t;
        }
        ms[i] = (float)(sum / (double)calls);
        for (int j = 0; j < 3; ++j) mnk[3 * i + j] = h->phase_mnk[3 * i + j];
    }
    *n = cnt;
    return ULSNN_OK;
}

namespace {

ulsnn_status_t forward_call(ulsnn_mlp_t* h, const float* const* W, const float* const* b, const float* X, int64_t ldx,
                            const Targets& tg, int64_t n, double* loss_out, cudaStream_t stream) {
    ulsnn_status_t st = check_call(h, W, b, X, ldx, tg.T ? (const void*)tg.T : (const void*)tg.labels, n, loss_out);
    if (st != ULSNN_OK) return st;
    if (tg.T && n > 0 && tg.ldt < h->sizes[h->L]) return ULSNN_ERR_INVALID_ARG;
    if ((st = check_arch()) != ULSNN_OK) return st;
    if (n == 0) return launch_zero_f64(loss_out, 1, stream);
    if (h->math == ULSNN_MATH_BF16) return forward_bf16(h, W, b, X, ldx, tg, n, false, 0, loss_out, stream);
    return forward(h, W, b, X, ldx, tg, n, false, 0, loss_out, stream);
}

ulsnn_status_t gradient_call(ulsnn_mlp_t* h, const float* const* W, const float* const* b, const float* X, int64_t ldx,
                             const Targets& tg, int64_t n, int accumulate, float* const* dW, float* const* db,
                             double* loss_out, cudaStream_t stream) {
    ulsnn_status_t st = check_call(h, W, b, X, ldx, tg.T ? (const void*)tg.T : (const void*)tg.labels, n, loss_out);
    if (st != ULSNN_OK) return st;
    if (tg.T && n > 0 && tg.ldt < h->sizes[h->L]) return ULSNN_ERR_INVALID_ARG;
    if (!dW || !db) return ULSNN_ERR_INVALID_ARG;
    const int L = h->L;
    const bool sse = tg.T != nullptr;
    const int32_t* labels = tg.labels;
    for (int l = 0; l < L; ++l) if (!dW[l] || !db[l]) return ULSNN_ERR_INVALID_ARG;
    if ((st = check_arch()) != ULSNN_OK) return st;
    if (n == 0) {
        if (accumulate) return ULSNN_OK;
        for (int l = 0; l < L; ++l) {
            if ((st = launch_zero(dW[l], (int64_t)h->sizes[l] * h->sizes[l + 1], stream)) != ULSNN_OK) return st;
            if ((st = launch_zero(db[l], h->sizes[l + 1], stream)) != ULSNN_OK) return st;
        }
        return launch_zero_f64(loss_out, 1, stream);
    }
    if (h->math == ULSNN_MATH_BF16) return gradient_bf16(h, W, b, X, ldx, tg, n, accumulate, dW, db, loss_out, stream);
    if ((st = forward(h, W, b, X, ldx, tg, n, true, accumulate, loss_out, stream)) != ULSNN_OK) return st;

    int64_t colsum_rows = 0;
    // Deltas of the hidden layers, top down: delta_l = (1 - H_l*H_l) * (delta_{l+1} W_{l+1})   (H_D of Section 4.2).
    // Softmax head, 3xTF32 and FFMA modes: delta_L is not stored, the kernels form softmax(z) - onehot from the stored
    // exponentials as they load them (the operand pass that splits them into TF32 pairs is there anyway).
    // Softmax head, TF32 mode: a kernel turns the stored exponentials into delta_L in place, so that the two products
    // that read it need no operand pass at all.
    // Squared-error head: the output epilogue has written delta_L = dE/dz where the exponentials would be.
    const bool stored_delta = sse || h->math == ULSNN_MATH_TF32;
    if (!sse && stored_delta &&
        (st = launch_delta_inplace(h->Z, h->ldz, h->chunk_tab, h->chunk_ld, labels, n, h->sizes[L], stream)) != ULSNN_OK) return st;
    for (int l = L - 1; l >= 1; --l) {
        GemmDesc d{};
        d.M = n; d.N = h->sizes[l]; d.K = h->sizes[l + 1];
        if (l + 1 == L && stored_delta) {
            d.A = h->Z; d.A_lo = h->Zlo; d.a_sm = h->ldz;
        } else if (l + 1 == L) {
            d.A = h->Z; d.a_sm = h->ldz; d.a_transform = 1; d.scale = h->chunk_tab; d.scale_ld = h->chunk_ld; d.labels = labels; d.a_pattern_is_m = 1;
        }
        else            { d.A = h->D[l + 1]; d.a_sm = h->ldd[l + 1]; }
        d.a_sk = 1;
        d.b_sk = d.N; d.b_sn = 1;
        set_weight_operand(h, d, W, l);
        d.C = h->D[l]; d.ldc = h->ldd[l]; d.alpha = 1.f; d.beta = 0.f;
        d.epi = EPI_TANHP; d.Hm = h->H[l]; d.Hm_lo = h->Hlo[l]; d.ldh = h->ldh[l];
        d.colsum_part = (l == 1) ? h->colsum_parts : nullptr;
        d.splits = 1; d.k_per_split = d.K;
        if (l == 1) colsum_rows = ((n + 127) / 128) * (use_tc(d, h->math) ? tc_colsum_groups() : simt_colsum_groups());
        if ((st = timed_gemm(h, d, stream)) != ULSNN_OK) return st;
    }

    // Weight gradients dW_w = delta_{w+1}^T * act_w: the sum over patterns is the K dimension (Section 4.2), cut into
    // slices of a fixed length whose partial products are combined in slice order.
    const float beta = accumulate ? 1.f : 0.f;
    for (int w = L - 1; w >= 0; --w) {
        GemmDesc d{};
        d.M = h->sizes[w + 1]; d.N = h->sizes[w] + (w >= 1 ? 1 : 0); d.K = n;
        if (w + 1 == L && stored_delta) { d.A = h->Z; d.A_lo = h->Zlo; d.a_sk = h->ldz; }
        else if (w + 1 == L) { d.A = h->Z; d.a_sk = h->ldz; d.a_transform = 1; d.scale = h->chunk_tab; d.scale_ld = h->chunk_ld; d.labels = labels; d.a_pattern_is_m = 0; }
        else            { d.A = h->D[w + 1]; d.a_sk = h->ldd[w + 1]; }
        d.a_sm = 1;
        if (w >= 1) { d.B = h->H[w]; d.B_lo = h->Hlo[w]; d.b_sk = h->ldh[w]; } else { d.B = X; d.b_sk = ldx; }
        d.b_sn = 1;
        d.alpha = 1.f; d.beta = 0.f; d.epi = EPI_PARTIAL;
        const bool tc = use_tc(d, h->math);
        const SplitPlan p = plan_splits(tiles_of(d, tc), d.K, slots_of(d, tc));
        d.splits = p.splits; d.k_per_split = p.k_per_split;
        d.ldp = round_up(d.N, 4); d.partials = h->partials;
        if ((size_t)p.splits * (size_t)d.M * (size_t)d.ldp * sizeof(float) > h->partials_bytes) return ULSNN_ERR_WORKSPACE_TOO_SMALL;
        if ((st = timed_gemm(h, d, stream)) != ULSNN_OK) return st;
        if ((st = launch_splitk_reduce(d.partials, p.splits, d.M, h->sizes[w], d.ldp, 1.f, beta, dW[w], h->sizes[w],
                                       w >= 1 ? db[w] : nullptr, stream)) != ULSNN_OK) return st;
        if (w >= 1 && (st = mark_gradient_done(h, w, stream)) != ULSNN_OK) return st;
    }
    // bias gradient of the first layer: column sums of delta_1 (both engines use 128-row tiles)
    if (L >= 2) {
        st = launch_colsum_reduce(h->colsum_parts, colsum_rows, h->sizes[1], accumulate, db[0], stream);
    } else if (stored_delta) {
        st = launch_matrix_colsum(h->Z, h->Zlo, h->ldz, n, h->sizes[1], h->colsum_parts, accumulate, db[0], stream);
    } else {
        st = launch_delta_colsum(h->Z, h->ldz, h->chunk_tab, h->chunk_ld, labels, n, h->sizes[1], h->colsum_parts, accumulate, db[0], stream);
    }
    if (st != ULSNN_OK) return st;
    return mark_gradient_done(h, 0, stream);      // db_0 comes last
}

}  // namespace

extern "C" ulsnn_status_t ulsnn_mlp_forward_loss(ulsnn_mlp_t* h, const float* const* W, const float* const* b,
                                                 const float* X, int64_t ldx, const int32_t* labels, int64_t n,
                                                 double* loss_out, ulsnn_stream_t stream) {
    return forward_call(h, W, b, X, ldx, Targets{labels, nullptr, 0}, n, loss_out, (cudaStream_t)stream);
}

extern "C" ulsnn_status_t ulsnn_mlp_gradient(ulsnn_mlp_t* h, const float* const* W, const float* const* b,
                                             const float* X, int64_t ldx, const int32_t* labels, int64_t n,
                                             int accumulate, float* const* dW, float* const* db, double* loss_out,
                                             ulsnn_stream_t stream) {
    return gradient_call(h, W, b, X, ldx, Targets{labels, nullptr, 0}, n, accumulate, dW, db, loss_out, (cudaStream_t)stream);
}

extern "C" ulsnn_status_t ulsnn_mlp_forward_sse(ulsnn_mlp_t* h, const float* const* W, const float* const* b,
                                                const float* X, int64_t ldx, const float* T, int64_t ldt, int64_t n,
                                                double* loss_out, ulsnn_stream_t stream) {
    if (n > 0 && !T) return ULSNN_ERR_INVALID_ARG;
    static const float dummy = 0.f;
    return forward_call(h, W, b, X, ldx, Targets{nullptr, T ? T : &dummy, ldt}, n, loss_out, (cudaStream_t)stream);
}

extern "C" ulsnn_status_t ulsnn_mlp_gradient_sse(ulsnn_mlp_t* h, const float* const* W, const float* const* b,
                                                 const float* X, int64_t ldx, const float* T, int64_t ldt, int64_t n,
                                                 int accumulate, float* const* dW, float* const* db, double* loss_out,
                                                 ulsnn_stream_t stream) {
    if (n > 0 && !T) return ULSNN_ERR_INVALID_ARG;
    static const float dummy = 0.f;
    return gradient_call(h, W, b, X, ldx, Targets{nullptr, T ? T : &dummy, ldt}, n, accumulate, dW, db, loss_out, (cudaStream_t)stream);
}

extern "C" ulsnn_status_t ulsnn_sgd_step(ulsnn_mlp_t* h, float* const* W, float* const* b,
                                         const float* const* dW, const float* const* db, float lr, ulsnn_stream_t stream) {
    if (!h || !W || !b || !dW || !db) return ULSNN_ERR_INVALID_ARG;
    for (int l = 0; l < h->L; ++l) if (!W[l] || !b[l] || !dW[l] || !db[l]) return ULSNN_ERR_INVALID_ARG;
    ulsnn_status_t st = check_arch();
    if (st != ULSNN_OK) return st;
    SgdBatch batch{};
    for (int l = 0; l < h->L; ++l) {
        batch.w[2 * l] = W[l]; batch.g[2 * l] = dW[l]; batch.n[2 * l] = (int64_t)h->sizes[l] * h->sizes[l + 1];
        batch.w[2 * l + 1] = b[l]; batch.g[2 * l + 1] = db[l]; batch.n[2 * l + 1] = h->sizes[l + 1];
    }
    batch.count = 2 * h->L;
    return launch_sgd_multi(batch, lr, (cudaStream_t)stream);
}

extern "C" ulsnn_status_t ulsnn_vec_dot_workspace_bytes(int64_t n, size_t* bytes) {
    if (!bytes || n < 0) return ULSNN_ERR_INVALID_ARG;
    *bytes = align256((size_t)(dot_parts(n) + 1) * sizeof(double));
    return ULSNN_OK;
}

extern "C" ulsnn_status_t ulsnn_vec_dot(int64_t n, const float* x, const float* y, double* out, void* workspace,
                                        size_t workspace_bytes, ulsnn_stream_t stream) {
    if (n < 0 || !out || (n > 0 && (!x || !y))) return ULSNN_ERR_INVALID_ARG;
    if (n > 0 && (!workspace || ((uintptr_t)workspace & 7) != 0)) return ULSNN_ERR_INVALID_ARG;
    if ((size_t)(dot_parts(n) + 1) * sizeof(double) > workspace_bytes && n > 0) return ULSNN_ERR_WORKSPACE_TOO_SMALL;
    ulsnn_status_t st = check_arch();
    if (st != ULSNN_OK) return st;
    return launch_dot(n, x, y, out, (double*)workspace, (cudaStream_t)stream);
}

extern "C" ulsnn_status_t ulsnn_vec_axpby(int64_t n, float a, const float* x, float b, const float* y, float* out,
                                          ulsnn_stream_t stream) {
    if (n < 0 || (n > 0 && (!x || !y || !out))) return ULSNN_ERR_INVALID_ARG;
    if (n == 0) return ULSNN_OK;
    ulsnn_status_t st = check_arch();
    if (st != ULSNN_OK) return st;
    return launch_axpby(n, a, x, b, y, out, (cudaStream_t)stream);
}

extern "C" int ulsnn_debug_device_cache_slot(int device) { return device_cache_slot(device); }

extern "C" ulsnn_status_t ulsnn_debug_wait_timeout(uint64_t limit_cycles, ulsnn_stream_t stream) {
    if (limit_cycles == 0 || limit_cycles > 2000000000ull) return ULSNN_ERR_INVALID_ARG;
    ulsnn_status_t st = check_arch();
    if (st != ULSNN_OK) return st;
    return tc_wait_probe_launch((unsigned long long)limit_cycles, (cudaStream_t)stream);
}

extern "C" ulsnn_status_t ulsnn_last_device_status(ulsnn_mlp_t* h, ulsnn_stream_t stream) {
    (void)h;        // the status word belongs to the device, not to a handle
    int word = 0;
    ulsnn_status_t st = device_status_fetch_and_clear((cudaStream_t)stream, &word);
    if (st != ULSNN_OK) return st;
    return word == DEV_OK ? ULSNN_OK : ULSNN_ERR_DEVICE_TIMEOUT;
}
