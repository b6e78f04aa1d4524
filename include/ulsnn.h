/*
 * ulsnn — error-and-gradient evaluation of large fully connected networks by
 * single-precision matrix products, on one NVIDIA B200 (sm_100a).
 *
 * The calls follow the problem statement of "Ultra-Large-Scale Neural-Network
 * Training on a PIII Cluster": a Level-3-BLAS SGEMM (Section 3.1), the error and
 * the gradient of a block of training patterns (Sections
 * 4.2-4.3, 6.2) and the plain step W := W - alpha*grad (Section 4.2).
 *
 * Conventions that hold for every call
 *  - Matrices are ROW-MAJOR fp32; a leading dimension (lda, ldx, ...) is the
 *    distance in elements between consecutive rows (the "stride" of Section 3.4).
 *  - Every data pointer is DEVICE memory owned by the caller, unless a comment
 *    says "host".  Arrays of pointers (W, b, dW, db) are HOST arrays of device
 *    pointers.  The library never frees or keeps a caller's buffer after the
 *    work enqueued by a call has finished.
 *  - Calls enqueue work on `stream` and return without synchronising.  They
 *    never exit, throw or trap.  Argument errors are detected on the host
 *    before anything is launched and reported through the return value.
 *  - Results are bitwise reproducible from run to run: every reduction (split
 *    K, column sums, loss) is done in an order fixed by the shapes only.
 *  - Device-side waits are bounded; if one expires the kernel records it in a
 *    status word and returns; ulsnn_last_device_status() reports it.
 */
#ifndef ULSNN_H
#define ULSNN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int ulsnn_status_t;
#define ULSNN_OK                        0
#define ULSNN_ERR_INVALID_ARG          (-1)   /* bad trans, negative size, ld too small, null pointer, bad label range ... */
#define ULSNN_ERR_UNSUPPORTED_ARCH     (-2)   /* current device is not compute capability 10.x */
#define ULSNN_ERR_WORKSPACE_TOO_SMALL  (-3)
#define ULSNN_ERR_CUDA                 (-4)   /* a CUDA runtime call failed (launch, attribute, allocation) */
#define ULSNN_ERR_DEVICE_TIMEOUT       (-5)   /* a bounded device-side wait expired */
#define ULSNN_ERR_TOO_LARGE            (-6)   /* a size exceeds a stated fixed maximum */

/* How products of fp32 numbers are formed.  Accumulation is fp32 in all modes. */
typedef enum {
    ULSNN_MATH_3XTF32    = 0,  /* tensor cores, each operand split hi+lo in TF32, three products: fp32-level accuracy */
    ULSNN_MATH_TF32      = 1,  /* tensor cores, operands truncated to TF32 (10-bit mantissa): fast mode */
    ULSNN_MATH_FP32_SIMT = 2,  /* FFMA on the CUDA cores: exact fp32 products, the comparison kernel */
    ULSNN_MATH_BF16      = 3   /* tensor cores, operands and stored activations / deltas rounded to bfloat16 (8-bit
                                  mantissa), hardware tanh and exp approximations: the 16-bit mode (Section 1: 16 bits
                                  are enough for smaller networks), twice the tensor rate and half the bytes of TF32 */
} ulsnn_math_t;

/* A CUDA stream (cudaStream_t / CUstream); 0 is the legacy default stream. */
typedef struct CUstream_st* ulsnn_stream_t;

const char* ulsnn_status_string(ulsnn_status_t status);
/* Packed version: major*10000 + minor*100 + patch. */
int ulsnn_version(void);

/* ------------------------------------------------------------------------------------------------
 * SGEMM (Section 3.1: "C <- alpha*A*B + beta*C", 2MNK flops, Level-3 BLAS interface).
 *
 *   C = alpha * op(A) * op(B) + beta * C,   op(X) = X ('N'/'n') or X^T ('T'/'t')
 *   op(A) is M x K, op(B) is K x N, C is M x N; row-major, so A is stored M x K with lda >= K when
 *   transA == 'N' and K x M with lda >= M when transA == 'T' (likewise B with ldb >= N or >= K); ldc >= N.
 *   beta == 0: C is overwritten and never read (it may hold NaN).  alpha == 0: A and B are not read.
 *   M, N or K == 0 are valid (K == 0 gives C = beta*C).  A, B, C must not overlap.
 *
 * ulsnn_sgemm uses ULSNN_MATH_3XTF32.  For shapes with few output tiles and a long K it splits K and
 * needs scratch memory: it takes it from a per-device buffer that the library allocates with cudaMalloc
 * on first need and grows on demand (so that first call may synchronise the device, and must not happen
 * inside a stream capture).  ulsnn_sgemm_ex never allocates: the caller passes the scratch
 * (ulsnn_sgemm_workspace_bytes tells how much; workspace may be NULL when that is 0).  The workspace must be
 * 256-byte aligned and may be reused by the next call on the same stream.
 * Operands that the tensor-core path cannot address with TMA (a base pointer not 16-byte aligned, or a leading
 * dimension that is not a multiple of 4) are first copied into the workspace with their rows padded to a multiple of
 * four floats (the re-buffering of Section 3.3), and the product then runs on the tensor cores like any other.  The
 * copies need room: ulsnn_sgemm_workspace_bytes_for, which is given the operands, includes it; ulsnn_sgemm_workspace_bytes,
 * which is not, covers addressable operands only.  ulsnn_sgemm_ex takes the re-buffered route when the workspace it is
 * given is large enough for it and computes such a product with the FFMA kernel (at least as accurate, several times
 * slower) when it is not; C may have any alignment and ldc on either route.
 * ulsnn_sgemm's own scratch is shared by all its calls on a device: calls on one device must be ordered with respect
 * to each other (one stream, or events), and any call that needs more scratch than every earlier one may synchronise.
 * ULSNN_MATH_BF16: op(A) and op(B) are first rounded to bfloat16 (round to nearest even) into the workspace, which
 * therefore is never empty in this mode (two bfloat16 copies with rows padded to 8 elements, then the split-K
 * partials); any lda / ldb is accepted.  C, alpha and beta stay fp32.  Expect a relative error of about 2e-3.
 * Errors: ULSNN_ERR_INVALID_ARG (nothing launched), ULSNN_ERR_WORKSPACE_TOO_SMALL, ULSNN_ERR_UNSUPPORTED_ARCH, ULSNN_ERR_CUDA.
 */
ulsnn_status_t ulsnn_sgemm(char transA, char transB, int64_t M, int64_t N, int64_t K, float alpha,
                           const float* A, int64_t lda, const float* B, int64_t ldb,
                           float beta, float* C, int64_t ldc, ulsnn_stream_t stream);
ulsnn_status_t ulsnn_sgemm_ex(char transA, char transB, int64_t M, int64_t N, int64_t K, float alpha,
                              const float* A, int64_t lda, const float* B, int64_t ldb,
                              float beta, float* C, int64_t ldc, ulsnn_math_t math,
                              void* workspace, size_t workspace_bytes, ulsnn_stream_t stream);
ulsnn_status_t ulsnn_sgemm_workspace_bytes(char transA, char transB, int64_t M, int64_t N, int64_t K,
                                           ulsnn_math_t math, size_t* bytes /* host, out */);
/* The same for given operands: A, B (device pointers, inspected for their alignment only, never read) and their leading
 * dimensions.  Includes the room for re-buffered copies of operands TMA cannot address (Section 3.3). */
ulsnn_status_t ulsnn_sgemm_workspace_bytes_for(char transA, char transB, int64_t M, int64_t N, int64_t K,
                                               const float* A, int64_t lda, const float* B, int64_t ldb,
                                               ulsnn_math_t math, size_t* bytes /* host, out */);

/*
 * SGEMM for callers that cannot allocate device memory (the paper has no counterpart of this call).
 *
 * Some callers have no way to provide scratch: code that runs where cudaMalloc is off limits (inside a region
 * whose memory budget is fixed up front, under a host framework that owns every allocation, in a callback that
 * must not synchronise the device) cannot size and pass the workspace ulsnn_sgemm_ex wants, and cannot accept
 * the allocate-on-first-need of ulsnn_sgemm.  ulsnn_sgemm_noalloc computes the same product as ulsnn_sgemm_ex with
 * the same `math`, but takes its split-K scratch from a fixed array of ulsnn_sgemm_noalloc_max_scratch_bytes()
 * (8 MiB) that is part of the library's image on every GPU that loads it.  It calls neither cudaMalloc nor
 * cudaFree nor any allocating routine.
 *  - A product whose scratch does not fit is rejected with ULSNN_ERR_TOO_LARGE and nothing is launched.  What is
 *    compared with the maximum is the scratch the product actually needs on the route it takes (split-K partials;
 *    in ULSNN_MATH_BF16 also the two bfloat16 copies; for operands TMA cannot address their re-buffered copies when
 *    those fit, else the FFMA kernel's partials), which can be less than ulsnn_sgemm_workspace_bytes reports.
 *    Products that need no scratch never touch the array.
 *  - The first call on each device that needs the array looks up the array's device address (with that device
 *    current); make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps the previous call's contents (nothing has to start
 *    at zero: every slice overwrites what the reduction reads).  Calls that could overlap on the GPU (different
 *    streams without an ordering between them) race on it: keep them on one stream or order them yourself.
 * Other arguments, conventions and errors are those of ulsnn_sgemm_ex.
 */
size_t         ulsnn_sgemm_noalloc_max_scratch_bytes(void);
ulsnn_status_t ulsnn_sgemm_noalloc(char transA, char transB, int64_t M, int64_t N, int64_t K, float alpha,
                                   const float* A, int64_t lda, const float* B, int64_t ldb,
                                   float beta, float* C, int64_t ldc, ulsnn_math_t math, ulsnn_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * Network evaluation (Section 4.1, Eq. 2 for the tanh hidden layers; Section 4.2 for the matrix form
 * H = tanh(X W^T), H_D = (1 - H*H)*(Y_D W), grad = H_D^T X, Y_D^T H; Section 4.3 for additivity over
 * patterns).  The output layer is softmax with cross-entropy on integer labels, and every layer has a
 * bias; with all biases zero the hidden layers are exactly Eq. 2.
 *
 * sizes[0..n_layers]: sizes[0] inputs, sizes[n_layers] classes, n_layers >= 1 weight matrices (<= 16).
 * W[l] is [sizes[l+1] x sizes[l]] row-major dense (w_jk: j = unit of layer l+1, k = unit of layer l);
 * b[l] is [sizes[l+1]].  max_patterns bounds n_patterns of every later call on the handle.
 */
typedef struct {
    int32_t        n_layers;
    const int32_t* sizes;         /* host, n_layers + 1 entries, each in [1, 2^20] */
    ulsnn_math_t   math;
    int64_t        max_patterns;  /* >= 1 */
} ulsnn_mlp_desc_t;

typedef struct ulsnn_mlp ulsnn_mlp_t;   /* opaque host object; owns no device memory */

/* Device scratch the handle needs (activations, logits, deltas, split-K partials, row statistics). */
ulsnn_status_t ulsnn_mlp_workspace_bytes(const ulsnn_mlp_desc_t* desc, size_t* bytes /* host, out */);
/* workspace: device memory, 256-byte aligned, at least the size above; owned by the caller and borrowed by the
 * handle until ulsnn_mlp_destroy.  Its contents are scratch between calls.  Calls on one handle must be
 * stream-ordered with respect to each other (they share the workspace). */
ulsnn_status_t ulsnn_mlp_create(ulsnn_mlp_t** handle /* host, out */, const ulsnn_mlp_desc_t* desc,
                                void* workspace, size_t workspace_bytes);
void           ulsnn_mlp_destroy(ulsnn_mlp_t* handle);

/*
 * "Compute the error": loss = sum_p [ logsumexp_j z_pj - z_{p,label_p} ], z = W_L h + b_L, SUMMED over the
 * n_patterns patterns (no 1/n, as Eq. 3).  X is [n_patterns x sizes[0]] with ldx >= sizes[0]; labels are int32
 * in [0, sizes[L]) (not checked: with an out-of-range label the results are unspecified, but nothing is
 * read or written out of bounds).
 * loss_out: device pointer to ONE double, written on the stream.  n_patterns == 0 writes 0.
 * Costs 2*n_p*sum_l sizes[l]*sizes[l+1] flops (Section 6.2).
 */
ulsnn_status_t ulsnn_mlp_forward_loss(ulsnn_mlp_t* handle, const float* const* W, const float* const* b,
                                      const float* X, int64_t ldx, const int32_t* labels, int64_t n_patterns,
                                      double* loss_out, ulsnn_stream_t stream);
/*
 * "Compute the gradient": the loss above and its derivative with respect to every W[l] and b[l], summed over
 * the patterns: dW[l] is [sizes[l+1] x sizes[l]] dense, db[l] is [sizes[l+1]].
 * accumulate == 0: dW, db and *loss_out are overwritten.  accumulate != 0: the results of this block of patterns
 * are ADDED to what dW, db and *loss_out hold (Section 4.3: error and gradient are additive over disjoint
 * subsets of the training set); a caller sweeping a large training set chunk by chunk in a fixed order gets a
 * bitwise reproducible total.  n_patterns == 0 with accumulate == 0 writes zeros.
 */
ulsnn_status_t ulsnn_mlp_gradient(ulsnn_mlp_t* handle, const float* const* W, const float* const* b,
                                  const float* X, int64_t ldx, const int32_t* labels, int64_t n_patterns,
                                  int accumulate, float* const* dW, float* const* db, double* loss_out,
                                  ulsnn_stream_t stream);
/*
 * The paper's own output layer and error (Section 4.1): tanh output units, Eq. 1, and the summed squared error of
 * Eq. 3, E = sum_p sum_j (y_pj - t_pj)^2 with y = tanh(W_L h + b_L), against a dense target matrix.
 * T is [n_patterns x sizes[L]] fp32 device memory, row-major, ldt >= sizes[L] (any values: +-1 codes, 0/1 codes ...).
 * ulsnn_mlp_forward_sse writes E to *loss_out; ulsnn_mlp_gradient_sse also returns dE/dW[l] and dE/db[l], the true
 * derivatives of Eq. 3: the matrices of Section 4.2 built from Y_D = (1 - Y*Y)*(T - Y) equal -1/2 times these.
 * Everything else (hidden layers, accumulate, summation over patterns, n_patterns == 0, errors) is as in
 * ulsnn_mlp_forward_loss / ulsnn_mlp_gradient; the flop count is the same (Section 6.2).
 */
ulsnn_status_t ulsnn_mlp_forward_sse(ulsnn_mlp_t* handle, const float* const* W, const float* const* b,
                                     const float* X, int64_t ldx, const float* T, int64_t ldt, int64_t n_patterns,
                                     double* loss_out, ulsnn_stream_t stream);
ulsnn_status_t ulsnn_mlp_gradient_sse(ulsnn_mlp_t* handle, const float* const* W, const float* const* b,
                                      const float* X, int64_t ldx, const float* T, int64_t ldt, int64_t n_patterns,
                                      int accumulate, float* const* dW, float* const* db, double* loss_out,
                                      ulsnn_stream_t stream);
/* Section 4.2: W := W - lr * dW, b := b - lr * db, in place, one fused multiply-add per element. */
/*
 * Training-set parallelism over several GPUs (Section 4.3: the patterns are partitioned, every worker evaluates its
 * share, the per-worker gradients are summed).  events: host array of n_layers CUDA events (cudaEvent_t, created by
 * the caller; entries may be NULL), or NULL to switch this off.  Every later ulsnn_mlp_gradient[_sse] on the handle
 * records events[w] on its stream as soon as dW[w] and db[w] of that call are final: the top layer's come first, the
 * first layer's last, so the exchange of a layer's gradient with the other GPUs can run on a second stream while the
 * products of the layers below still compute (the reduce overlapped with computation, Section 5.2).  The events stay
 * the caller's; the handle keeps the array's entries, not the array.
 */
ulsnn_status_t ulsnn_mlp_set_gradient_events(ulsnn_mlp_t* handle, void* const* events /* host */);

ulsnn_status_t ulsnn_sgd_step(ulsnn_mlp_t* handle, float* const* W, float* const* b,
                              const float* const* dW, const float* const* db, float lr, ulsnn_stream_t stream);
/*
 * Vector operations for the line search and the conjugate-gradient direction of Section 4.2, on flat parameter
 * vectors in device memory.
 * ulsnn_vec_dot: *out (device, one double) = sum_i x[i]*y[i], accumulated in double in an order that depends on n
 *   only (partial sums over blocks of 1024 elements, then a fixed tree), so repeated runs give the same bits.
 *   workspace: device scratch of ulsnn_vec_dot_workspace_bytes(n) bytes, 8-byte aligned.
 * ulsnn_vec_axpby: out[i] = a*x[i] + b*y[i]; out may be x or y.
 */
ulsnn_status_t ulsnn_vec_dot_workspace_bytes(int64_t n, size_t* bytes /* host, out */);
ulsnn_status_t ulsnn_vec_dot(int64_t n, const float* x, const float* y, double* out, void* workspace,
                             size_t workspace_bytes, ulsnn_stream_t stream);
ulsnn_status_t ulsnn_vec_axpby(int64_t n, float a, const float* x, float b, const float* y, float* out,
                               ulsnn_stream_t stream);
/* Synchronises `stream`, then returns ULSNN_OK, ULSNN_ERR_DEVICE_TIMEOUT if any kernel of the library gave up a
 * bounded wait on the current device since the last call of this function there (the status word belongs to the
 * device, not to the handle, which may be NULL; the call clears it), or ULSNN_ERR_CUDA. */
ulsnn_status_t ulsnn_last_device_status(ulsnn_mlp_t* handle, ulsnn_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * Seeded synthetic data, generated in place on the device (no counterpart in the paper, whose data set is
 * not available; used by the benchmarks to fill multi-gigabyte pattern matrices without a host copy).
 * Element i of the tensor gets hash(seed, tensor_id, offset + i) mapped to
 *   mode 0: uniform [0,1) on a 2^-24 grid;  mode 1: uniform [-1,1) on a 2^-23 grid.
 * Labels: (hash >> 11) mod n_classes as int32.  The hash is a two-round splitmix64 finaliser of
 * seed*0x9E3779B97F4A7C15 + tensor_id*0xD1B54A32D192ED03 + index + 1.
 */
ulsnn_status_t ulsnn_fill_uniform(float* dst, int64_t n, uint64_t seed, uint64_t tensor_id, uint64_t offset,
                                  int mode, ulsnn_stream_t stream);
ulsnn_status_t ulsnn_fill_labels(int32_t* dst, int64_t n, uint64_t seed, uint64_t tensor_id, uint64_t offset,
                                 int32_t n_classes, ulsnn_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * Instrumentation (no counterpart in the paper): number of kernel launches the library has enqueued since it
 * was loaded, by kind.  counts (host, out): [0] FFMA GEMM kernels, [1] tcgen05 GEMM kernels, [2] reduction and
 * other small kernels, [3] fill kernels.
 */
void ulsnn_launch_counts(int64_t counts[4]);
/*
 * Per-product device times of a handle (no counterpart in the paper).  With timing switched on, every GEMM launch of
 * ulsnn_mlp_forward_loss / ulsnn_mlp_gradient is bracketed by CUDA events on the call's stream (the events are created
 * when timing is first switched on).  Switching it on also resets the record.  ulsnn_mlp_phase_times waits for the
 * recorded events and returns the device time of each product AVERAGED over the calls made since timing was switched
 * on (at most the 64 most recent; all of them must have been calls of the same kind): n (host, in: capacity of the
 * arrays, out: number of products), ms[i] the mean time of product i, mnk[3*i..3*i+2] its M, N, K.  Products come in
 * launch order: the L forward products, the L-1 delta products (top layer first), the L weight-gradient products
 * (top layer first).
 */
ulsnn_status_t ulsnn_mlp_enable_timing(ulsnn_mlp_t* handle, int on);
ulsnn_status_t ulsnn_mlp_phase_times(ulsnn_mlp_t* handle, int* n, float* ms, int64_t* mnk);
/*
 * Checks of the library's own safety net (no counterpart in the paper).
 * ulsnn_debug_wait_timeout: enqueues one thread block that allocates tensor memory as the product kernels do and then
 *   waits on a barrier nothing ever arrives on, with a limit of limit_cycles SM clock cycles (1 .. 2e9).  The wait runs
 *   out, the block records the time-out in the device status word, frees its tensor memory and returns by itself; the
 *   next ulsnn_last_device_status() on the device returns ULSNN_ERR_DEVICE_TIMEOUT.  Nothing traps or faults, and
 *   the context stays usable.  This is the path every bounded wait of the product kernels takes when it gives up.
 * ulsnn_debug_device_cache_slot: the slot of a device ordinal in the library's per-device host tables (architecture
 *   check, SM count, symbol addresses, kernel attributes, scratch buffers), or -1 when the ordinal is outside them
 *   (such a device is refused).  Host only.
 */
ulsnn_status_t ulsnn_debug_wait_timeout(uint64_t limit_cycles, ulsnn_stream_t stream);
int            ulsnn_debug_device_cache_slot(int device);

#ifdef __cplusplus
}
#endif
#endif /* ULSNN_H */
