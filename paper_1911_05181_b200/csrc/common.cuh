// Shared declarations of the library's translation units (host + device).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/ulsnn.h"

namespace ulsnn {

// What a GEMM kernel does with its accumulator tile.
enum Epilogue : int {
    EPI_SGEMM     = 0,  // C = alpha*acc + beta*C                                   (Section 3.1)
    EPI_BIAS_TANH = 1,  // C = tanh(acc + bias[col]); optionally C[:, N] = 1         (Eq. 2 / H = tanh(X W^T))
    EPI_LOGITS    = 2,  // z = acc + bias[col]; per-(row, column-tile) softmax statistics, z at the label; stored: exp(z - m)
                        // with m the running maximum of the row when its 32-column chunk was reached (chunk_max)
    EPI_TANHP     = 3,  // C = (1 - h*h) * acc, h = Hm[row][col]; per-row-tile column sums (H_D of Section 4.2)
    EPI_PARTIAL   = 4,  // split-K slice: raw accumulator into partials[slice]
    EPI_TANH_SSE  = 5   // the paper's output layer (Eqs. 1, 3): y = tanh(acc + bias); per-(row, column-tile) sums of
                        // (y - t)^2; C = 2 (y - t)(1 - y^2) = dE/dz (optionally as a (hi, lo) pair)
};

// One product D = op(A) op(B) plus its fused epilogue; both engines (FFMA and tcgen05) take this.
struct GemmDesc {
    int64_t M, N, K;
    const float* A; int64_t a_sm, a_sk;   // A(i,k) = A[i*a_sm + k*a_sk]  (one of the strides is 1)
    const float* B; int64_t b_sk, b_sn;   // B(k,j) = B[k*b_sk + j*b_sn]
    // Operands stored as a pair: when A_lo (B_lo) is not null the operand's value is A + A_lo, where A holds the
    // values rounded to TF32 and A_lo the rounded remainders, with the strides of A (B).  The tensor-core engine
    // then needs no operand pass for it in 3xTF32 mode; the FFMA engine adds the two.
    const float* A_lo; const float* B_lo;
    float* C; int64_t ldc;
    float* C_lo;              // BIAS_TANH, TANH_SSE: not null -> C gets tf32_rn(v) and C_lo the rounded remainder (same ldc)
    float alpha, beta;
    int epi;
    // epilogue operands
    const float* bias;        // [N]                 BIAS_TANH, LOGITS
    int ones_cols;            // BIAS_TANH: write C[:, N] = 1 and C[:, N+1 .. N+ones_cols) = 0 (0: nothing)
    const float* Hm; int64_t ldh;        // TANHP
    const float* Hm_lo;       // TANHP: not null -> h = Hm + Hm_lo
    float* colsum_part;       // TANHP: [row_tiles * groups][N] partial column sums (may be null)
    const int32_t* labels;    // LOGITS and the A transform: label of each pattern
    const float* T; int64_t ldt;         // TANH_SSE: targets [M x N], rows ldt apart
    float2* stats; int64_t stats_ld;     // LOGITS: stats[row*stats_ld + col_tile] = (max, sum exp(z - max)); TANH_SSE: (0, sum (y-t)^2)
    float* zlabel;            // LOGITS: z[row][label[row]]
    float* chunk_max; int64_t chunk_ld;  // LOGITS: chunk_max[row*chunk_ld + col/32] = the m that chunk's stored values refer to
    // A transform: the stored operand holds e = exp(z - m) as left by the LOGITS epilogue; the product uses
    // softmax(z) - onehot(label) = e * scale - onehot, scale[pattern*scale_ld + class/32] = exp(m - logsumexp)
    int a_transform;
    const float* scale; int64_t scale_ld;
    int a_pattern_is_m;       // 1: the M index of A is the pattern (K is the class); 0: K is the pattern
    // split-K (EPI_PARTIAL): slice s covers k in [s*k_per_split, min(K, (s+1)*k_per_split))
    int splits; int64_t k_per_split;
    float* partials; int64_t ldp;        // partials[(s*M + i)*ldp + j]
};

// One product of the 16-bit engine: operands stored as bfloat16, fp32 accumulation.  The epilogues are those of
// GemmDesc, except that activations, stored exponentials and deltas (BIAS_TANH, LOGITS, TANHP) are written as
// bfloat16 to Ch, and that the transcendental functions are the hardware approximations.
struct HalfGemmDesc {
    int64_t M, N, K;
    const __nv_bfloat16* A; int64_t a_sm, a_sk;   // A(i,k) = A[i*a_sm + k*a_sk]  (one of the strides is 1)
    const __nv_bfloat16* B; int64_t b_sk, b_sn;   // B(k,j) = B[k*b_sk + j*b_sn]
    int epi;                  // any Epilogue
    float* C; int64_t ldc;    // SGEMM: fp32 output
    float alpha, beta;
    __nv_bfloat16* Ch; int64_t ldch;     // BIAS_TANH, LOGITS and TANH_SSE (may be null: statistics only), TANHP: bfloat16 output
    const float* bias;        // [N]  BIAS_TANH, LOGITS
    int ones_cols;            // BIAS_TANH: Ch[:, N] = 1 and Ch[:, N+1 .. N+ones_cols) = 0
    const __nv_bfloat16* Hm; int64_t ldh;        // TANHP
    const int32_t* labels;    // LOGITS
    const float* T; int64_t ldt;         // TANH_SSE: fp32 targets [M x N]
    float2* stats; int64_t stats_ld;     // LOGITS: stats[row*stats_ld + 2*col_tile + h], h = 0, 1: (max, sum exp(z - max)) over
                                         // the even (odd) 64-column blocks of the tile; (-inf, 0) when there is none.
                                         // TANH_SSE: (0, sum (y - t)^2) at the same places
    float* zlabel;
    float* chunk_max; int64_t chunk_ld;  // LOGITS: as in GemmDesc
    int splits; int64_t k_per_split;     // EPI_PARTIAL; k_per_split is a multiple of hg_k_granule()
    float* partials; int64_t ldp;
};

// Device status word values (0 = fine).
enum : int { DEV_OK = 0, DEV_TIMEOUT = 1 };

// Host-side caches of per-device facts (architecture check, SM count, symbol addresses, kernel attributes, scratch
// buffers) are arrays indexed by this slot: the device ordinal, or -1 when it is outside the table.
constexpr int MAX_DEVICE_SLOTS = 64;
inline int device_cache_slot(int device) { return (device >= 0 && device < MAX_DEVICE_SLOTS) ? device : -1; }

// engines
ulsnn_status_t simt_gemm_launch(const GemmDesc& d, cudaStream_t stream);
int simt_tile_m();
int simt_tile_n();
// tcgen05 engine (tc_gemm.cu).  tc_gemm_supported: can TMA address these operands (16-byte aligned bases, leading
// dimensions that are multiples of 4 floats)?  tc_tile_n: the column-tile width it will use for this product.
bool tc_gemm_supported(const GemmDesc& d);
int tc_tile_m(const GemmDesc& d);
int tc_tile_n(const GemmDesc& d);
// how many tiles each engine works on at a time (CTAs, or CTA pairs): what a split-K plan has to fill
int tc_slots(const GemmDesc& d);
int simt_slots();
// EPI_TANHP writes this many partial column-sum rows per 128-row tile (row index = tile*groups + group)
int tc_colsum_groups();
int simt_colsum_groups();
ulsnn_status_t tc_gemm_launch(const GemmDesc& d, bool three_x, cudaStream_t stream);
// device status word shared by all kernels of the library on the current device
int* device_status_word();      // its address on the current device (null if it cannot be had)
// One CTA that waits, with the given limit in clock cycles, on a barrier nothing ever arrives on: the wait runs out,
// the CTA records DEV_TIMEOUT, frees its tensor memory and returns.  For the test of the bounded-wait path.
ulsnn_status_t tc_wait_probe_launch(unsigned long long limit_cycles, cudaStream_t stream);
ulsnn_status_t device_status_fetch_and_clear(cudaStream_t stream, int* word);

// 16-bit tcgen05 engine (bf16_gemm.cu): operands need 16-byte aligned bases and leading dimensions that are
// multiples of 8 elements
bool hg_gemm_supported(const HalfGemmDesc& d);
int hg_tile_m(const HalfGemmDesc& d);
int hg_tile_n(const HalfGemmDesc& d);
int hg_slots(const HalfGemmDesc& d);
int hg_k_granule();
ulsnn_status_t hg_gemm_launch(const HalfGemmDesc& d, cudaStream_t stream);
// dst[r][j] = bf16(src[r][j]), j < cols; dst[r][cols] = 1 when `ones`; the rest of each row up to ldd (a multiple of 8) = 0
ulsnn_status_t launch_to_bf16(const float* src, int64_t rows, int64_t cols, int64_t lds, __nv_bfloat16* dst, int64_t ldd,
                              int ones, cudaStream_t stream);
// in place: stored exponentials -> bf16(e * scale[pattern][class/32] - [label == class]), zero beyond n_classes
ulsnn_status_t launch_delta_bf16(__nv_bfloat16* E, int64_t lde, const float* scale, int64_t scale_ld, const int32_t* labels,
                                 int64_t n, int64_t n_classes, cudaStream_t stream);

// reductions and small kernels (reduce.cu)
// out[i*ldo + j] = alpha * sum_s parts[(s*M + i)*ldp + j] + beta*out   for j < N;   if bias_out: column N goes to
// bias_out[i] (= sum_s parts[..][N], scaled the same way) -- the "ones column" that carries the bias gradient.
ulsnn_status_t launch_splitk_reduce(const float* parts, int splits, int64_t M, int64_t N, int64_t ldp,
                                    float alpha, float beta, float* out, int64_t ldo, float* bias_out,
                                    cudaStream_t stream);
// out[j] = sum_t parts[t*N + j] (+ out[j] if accumulate), t in fixed order
ulsnn_status_t launch_colsum_reduce(const float* parts, int64_t tiles, int64_t N, int accumulate, float* out,
                                    cudaStream_t stream);
// lse[p] from the per-tile statistics; loss = sum_p (lse[p] - zlabel[p]) in a fixed order, in double
// chunk_tab (may be null): [n x chunk_ld] chunk maxima written by the LOGITS epilogue, turned in place into the
// factors exp(m - lse) that the delta products multiply the stored exponentials with
ulsnn_status_t launch_rowstats(const float2* stats, int64_t stats_ld, int tiles, const float* zlabel, int64_t n,
                               float* lse, float* chunk_tab, int64_t chunk_ld, int n_chunks, double* block_partials,
                               int accumulate, double* loss_out, cudaStream_t stream);
int rowstats_blocks(int64_t n);
// loss = sum_p sum_t stats[p*stats_ld + t].y in a fixed order, in double (the squared-error head)
ulsnn_status_t launch_rowsums(const float2* stats, int64_t stats_ld, int tiles, int64_t n, double* block_partials,
                              int accumulate, double* loss_out, cudaStream_t stream);
// out[j] = sum_p (A[p*lda + j] + A_lo[p*lda + j])  (A_lo may be null), rows added in a fixed order
ulsnn_status_t launch_matrix_colsum(const float* A, const float* A_lo, int64_t lda, int64_t n, int64_t cols, float* parts,
                                    int accumulate, float* out, cudaStream_t stream);
// db[j] = sum_p softmax(z_p)_j - [label_p == j]   (only for networks without a hidden layer); Z holds the stored
// exponentials, scale their per-chunk factors
ulsnn_status_t launch_delta_colsum(const float* Z, int64_t ldz, const float* scale, int64_t scale_ld, const int32_t* labels,
                                   int64_t n, int64_t n_classes, float* parts, int accumulate, float* out,
                                   cudaStream_t stream);
int delta_colsum_tiles(int64_t n);
// in place: stored exponentials Z [n x ldz] (ldz a multiple of 4, 16-byte aligned) -> Z * scale[pattern][class/32] - onehot,
// zero in the row padding
ulsnn_status_t launch_delta_inplace(float* Z, int64_t ldz, const float* scale, int64_t scale_ld, const int32_t* labels,
                                    int64_t n, int64_t n_classes, cudaStream_t stream);
// hi[i] = tf32_rn(x[i]), lo[i] = tf32_rn(x[i] - hi[i])   (round to nearest, ties away from zero, 10 mantissa bits)
ulsnn_status_t launch_split_hilo(const float* x, int64_t n, float* hi, float* lo, cudaStream_t stream);
// out = a*x + b*y (out may alias x or y); *out = sum_i x[i]*y[i] in double, blocks of 1024 elements in index order
ulsnn_status_t launch_axpby(int64_t n, float a, const float* x, float b, const float* y, float* out, cudaStream_t stream);
ulsnn_status_t launch_dot(int64_t n, const float* x, const float* y, double* out, double* parts, cudaStream_t stream);
int64_t dot_parts(int64_t n);
// w[t][i] -= lr * g[t][i] for `count` tensors in one launch
struct SgdBatch { static constexpr int MAX = 32; float* w[MAX]; const float* g[MAX]; int64_t n[MAX]; int count; };
ulsnn_status_t launch_sgd_multi(const SgdBatch& b, float lr, cudaStream_t stream);
ulsnn_status_t launch_zero(float* p, int64_t n, cudaStream_t stream);
ulsnn_status_t launch_zero_f64(double* p, int64_t n, cudaStream_t stream);
ulsnn_status_t launch_scale_rows(float* C, int64_t M, int64_t N, int64_t ldc, float beta, cudaStream_t stream);
// dst[r][c] = src[r][c] (c < cols), 0 for cols <= c < ldd; dst 16-byte aligned, ldd a multiple of 4
ulsnn_status_t launch_pack_rows(const float* src, int64_t rows, int64_t cols, int64_t lds, float* dst, int64_t ldd,
                                cudaStream_t stream);
// can TMA address a row-major fp32 operand with this base and leading dimension?
bool tc_operand_addressable(const float* base, int64_t ld);

// launch accounting: kind 0 FFMA GEMM, 1 tcgen05 GEMM, 2 reductions/small kernels, 3 fills
void count_launch(int kind);

static inline ulsnn_status_t cuda_ok(cudaError_t e) { return e == cudaSuccess ? ULSNN_OK : ULSNN_ERR_CUDA; }

}  // namespace ulsnn
