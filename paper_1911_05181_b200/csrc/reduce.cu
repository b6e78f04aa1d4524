// Fixed-order reductions and the small memory-bound kernels around the GEMMs.
//
// Every sum here is taken in an order that depends on the shapes only (never on arrival order), in
// double where the number of terms is large, so repeated runs are bitwise identical (Section 4.3:
// error and gradient are additive over patterns; this is the on-device form of that sum).
#include "common.cuh"
#include <math.h>

namespace ulsnn {

namespace {

// out = alpha * sum_s parts[s] + beta*out, one thread per output element, slices in index order, sum in double.
__global__ void splitk_reduce_kernel(const float* __restrict__ parts, int splits, int64_t M, int64_t N, int64_t ldp,
                                     float alpha, float beta, float* __restrict__ out, int64_t ldo,
                                     float* __restrict__ bias_out) {
    const int64_t ncols = N + (bias_out ? 1 : 0);
    const int64_t total = M * ncols;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = e / ncols, j = e - i * ncols;
        double s = 0.0;
        for (int sidx = 0; sidx < splits; ++sidx) s += (double)parts[((int64_t)sidx * M + i) * ldp + j];
        float* dst = (j < N) ? out + i * ldo + j : bias_out + i;
        double v = (double)alpha * s;
        if (beta != 0.f) v += (double)beta * (double)*dst;
        *dst = (float)v;
    }
}

// out[j] = sum_t parts[t*N + j]: a block owns 32 columns; its 32 row lanes each add every 32nd partial row in
// index order (double), then the 32 lane sums are added in lane order.  The order depends on (tiles, N) only.
constexpr int CS_COLS = 32, CS_LANES = 32;
__global__ void __launch_bounds__(CS_COLS * CS_LANES)
colsum_reduce_kernel(const float* __restrict__ parts, int64_t tiles, int64_t N, int accumulate, float* __restrict__ out) {
    __shared__ double red[CS_LANES][CS_COLS + 1];
    const int tx = threadIdx.x % CS_COLS, ty = threadIdx.x / CS_COLS;
    const int64_t j = (int64_t)blockIdx.x * CS_COLS + tx;
    double s = 0.0;
    if (j < N) for (int64_t t = ty; t < tiles; t += CS_LANES) s += (double)parts[t * N + j];
    red[ty][tx] = s;
    __syncthreads();
    if (ty == 0 && j < N) {
        double tot = 0.0;
#pragma unroll
        for (int l = 0; l < CS_LANES; ++l) tot += red[l][tx];
        if (accumulate) tot += (double)out[j];
        out[j] = (float)tot;
    }
}

constexpr int RS_THREADS = 256;

// One warp per pattern (each of a block's 8 warps takes 8 patterns in turn): the lanes combine the per-tile
// (max, sum-exp) pairs -- every lane its tiles in index order, then a fixed shuffle tree -- into the log-sum-exp,
// and turn the pattern's chunk maxima into the factors exp(m - lse).  lse - z_label is then summed over the
// block's 64 patterns in a fixed tree.  Everything a pattern needs from memory is asked for before the first use.
constexpr int RS_ROWS = 64;
__global__ void __launch_bounds__(RS_THREADS)
rowstats_kernel(const float2* __restrict__ stats, int64_t stats_ld, int tiles,
                const float* __restrict__ zlabel, int64_t n, float* __restrict__ lse,
                float* __restrict__ chunk_tab, int64_t chunk_ld, int n_chunks,
                double* __restrict__ block_partials) {
    __shared__ double red[RS_ROWS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll 2
    for (int i = 0; i < RS_ROWS / 8; ++i) {
        const int row = warp * (RS_ROWS / 8) + i;
        const int64_t p = (int64_t)blockIdx.x * RS_ROWS + row;
        double term = 0.0;
        if (p < n) {                                        // uniform over the warp
            const float2* st = stats + p * stats_ld;
            float* q = chunk_tab ? chunk_tab + p * chunk_ld : nullptr;
            const float2 first = lane < tiles ? st[lane] : make_float2(-INFINITY, 0.f);
            float qv[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) { const int t = lane + 32 * k; qv[k] = (q && t < n_chunks) ? q[t] : 0.f; }
            const float zl = zlabel[p];
            float mx = first.x;
            for (int t = lane + 32; t < tiles; t += 32) mx = fmaxf(mx, st[t].x);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            // the tile sums are fp32 sums of fp32 exponentials: rescaling them needs no more than expf
            double s = (double)first.y * (double)expf(first.x - mx);
            for (int t = lane + 32; t < tiles; t += 32) {
                const float2 v = st[t];
                s += (double)v.y * (double)expf(v.x - mx);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            const double l = (double)mx + log(s);
            if (q) {
#pragma unroll
                for (int k = 0; k < 4; ++k) { const int t = lane + 32 * k; if (t < n_chunks) q[t] = expf((float)((double)qv[k] - l)); }
                for (int t = lane + 128; t < n_chunks; t += 32) q[t] = expf((float)((double)q[t] - l));
            }
            if (lane == 0) lse[p] = (float)l;
            term = l - (double)zl;
        }
        if (lane == 0) red[row] = term;
    }
    __syncthreads();
    for (int o = RS_ROWS / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) block_partials[blockIdx.x] = red[0];
}

// squared-error head: one thread per pattern adds its per-tile sums in tile order, then a fixed tree over the block
__global__ void rowsums_kernel(const float2* __restrict__ stats, int64_t stats_ld, int tiles, int64_t n,
                               double* __restrict__ block_partials) {
    __shared__ double red[RS_THREADS];
    const int64_t p = (int64_t)blockIdx.x * RS_THREADS + threadIdx.x;
    double term = 0.0;
    if (p < n) for (int t = 0; t < tiles; ++t) term += (double)stats[p * stats_ld + t].y;
    red[threadIdx.x] = term;
    __syncthreads();
    for (int o = RS_THREADS / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) block_partials[blockIdx.x] = red[0];
}

__global__ void __launch_bounds__(256)
loss_final_kernel(const double* __restrict__ block_partials, int nblocks, int accumulate, double* __restrict__ loss_out) {
    // one block: 256 threads add every 256th partial in index order, then a fixed tree
    __shared__ double red[256];
    double s = 0.0;
    for (int i = threadIdx.x; i < nblocks; i += 256) s += block_partials[i];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss_out = accumulate ? *loss_out + red[0] : red[0];
}

constexpr int DC_ROWS = 1024;   // patterns per partial row of the delta column sum

__global__ void matrix_colsum_kernel(const float* __restrict__ A, const float* __restrict__ A_lo, int64_t lda, int64_t n,
                                     int64_t cols, float* __restrict__ parts) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= cols) return;
    const int64_t p0 = (int64_t)blockIdx.y * DC_ROWS, p1 = min(n, p0 + DC_ROWS);
    float s = 0.f;
    for (int64_t p = p0; p < p1; ++p) s += A[p * lda + j] + (A_lo ? A_lo[p * lda + j] : 0.f);
    parts[(int64_t)blockIdx.y * cols + j] = s;
}

__global__ void delta_colsum_kernel(const float* __restrict__ Z, int64_t ldz, const float* __restrict__ scale, int64_t scale_ld,
                                    const int32_t* __restrict__ labels, int64_t n, int64_t n_classes,
                                    float* __restrict__ parts) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n_classes) return;
    const int64_t p0 = (int64_t)blockIdx.y * DC_ROWS, p1 = min(n, p0 + DC_ROWS);
    float s = 0.f;
    for (int64_t p = p0; p < p1; ++p) s += Z[p * ldz + j] * scale[p * scale_ld + (j >> 5)] - ((int64_t)labels[p] == j ? 1.f : 0.f);
    parts[(int64_t)blockIdx.y * n_classes + j] = s;
}

// In place: Z[p][j] (= exp(z - m) as the LOGITS epilogue left it) -> Z[p][j] * scale[p][j/32] - [label_p == j], zero in
// the row padding.  One thread per four elements (ldz is a multiple of 4), which lie in one 32-class chunk.
__global__ void delta_inplace_kernel(float* __restrict__ Z, int64_t ldz, const float* __restrict__ scale, int64_t scale_ld,
                                     const int32_t* __restrict__ labels, int64_t n, int n_classes) {
    const int64_t groups = ldz >> 2;
    const int64_t total = n * groups;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t pat = e / groups;
        const int j0 = (int)(e - pat * groups) << 2;
        float4* ptr = reinterpret_cast<float4*>(Z + pat * ldz + j0);
        float4 v = *ptr;
        const float f = (j0 < n_classes) ? __ldg(scale + pat * scale_ld + (j0 >> 5)) : 0.f;
        const int lab = __ldg(labels + pat);
        v.x = (j0 + 0 < n_classes) ? fmaf(v.x, f, j0 + 0 == lab ? -1.f : 0.f) : 0.f;
        v.y = (j0 + 1 < n_classes) ? fmaf(v.y, f, j0 + 1 == lab ? -1.f : 0.f) : 0.f;
        v.z = (j0 + 2 < n_classes) ? fmaf(v.z, f, j0 + 2 == lab ? -1.f : 0.f) : 0.f;
        v.w = (j0 + 3 < n_classes) ? fmaf(v.w, f, j0 + 3 == lab ? -1.f : 0.f) : 0.f;
        *ptr = v;
    }
}

__device__ __forceinline__ float round_tf32(float x) {
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u);
}

__global__ void split_hilo_kernel(const float* __restrict__ x, int64_t n, float* __restrict__ hi, float* __restrict__ lo) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const float v = x[i], h = round_tf32(v);
        hi[i] = h;
        lo[i] = round_tf32(v - h);
    }
}

__global__ void axpby_kernel(int64_t n, float a, const float* __restrict__ x, float b, const float* __restrict__ y, float* out) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = fmaf(a, x[i], b * y[i]);
}

constexpr int DOT_BLOCK = 1024;     // elements per partial sum

// partial sums of x*y over blocks of DOT_BLOCK elements: 256 threads take four elements each (index order inside a
// thread), then a fixed tree over the threads; all in double
__global__ void dot_parts_kernel(int64_t n, const float* __restrict__ x, const float* __restrict__ y, double* __restrict__ parts) {
    __shared__ double red[256];
    const int64_t base = (int64_t)blockIdx.x * DOT_BLOCK + (int64_t)threadIdx.x * 4;
    double s = 0.0;
#pragma unroll
    for (int j = 0; j < 4; ++j) if (base + j < n) s += (double)x[base + j] * (double)y[base + j];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) parts[blockIdx.x] = red[0];
}

__global__ void dot_final_kernel(const double* __restrict__ parts, int64_t nparts, double* __restrict__ out) {
    // one block: 256 threads add every 256th partial in index order, then a fixed tree
    __shared__ double red[256];
    double s = 0.0;
    for (int64_t i = threadIdx.x; i < nparts; i += 256) s += parts[i];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = red[0];
}

// the same step for several tensors in one launch: blockIdx.y picks the tensor
__global__ void sgd_multi_kernel(const SgdBatch b, float lr) {
    float* __restrict__ w = b.w[blockIdx.y];
    const float* __restrict__ g = b.g[blockIdx.y];
    const int64_t n = b.n[blockIdx.y];
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        w[i] = fmaf(-lr, g[i], w[i]);
}

template <typename T>
__global__ void zero_kernel(T* __restrict__ p, int64_t n) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) p[i] = T(0);
}

__global__ void scale_rows_kernel(float* __restrict__ C, int64_t M, int64_t N, int64_t ldc, float beta) {
    const int64_t total = M * N;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = e / N, j = e - i * N;
        C[i * ldc + j] = (beta == 0.f) ? 0.f : beta * C[i * ldc + j];
    }
}

__device__ __forceinline__ uint64_t mix64(uint64_t seed, uint64_t tensor_id, uint64_t index) {
    uint64_t z = seed * 0x9E3779B97F4A7C15ull + tensor_id * 0xD1B54A32D192ED03ull + index + 1ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z = z ^ (z >> 31);
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z = z ^ (z >> 31);
    return z;
}

__global__ void fill_uniform_kernel(float* __restrict__ dst, int64_t n, uint64_t seed, uint64_t tid, uint64_t offset, int mode) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const uint64_t h = mix64(seed, tid, offset + (uint64_t)i);
        const float u = (float)(uint32_t)(h >> 40) * 5.9604644775390625e-8f;   // 2^-24, exact
        dst[i] = mode ? 2.f * u - 1.f : u;
    }
}

__global__ void fill_labels_kernel(int32_t* __restrict__ dst, int64_t n, uint64_t seed, uint64_t tid, uint64_t offset, uint32_t n_classes) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const uint64_t h = mix64(seed, tid, offset + (uint64_t)i);
        dst[i] = (int32_t)((h >> 11) % (uint64_t)n_classes);
    }
}

inline unsigned grid_for(int64_t n, int threads) {
    int64_t b = (n + threads - 1) / threads;
    if (b < 1) b = 1;
    if (b > 148 * 16) b = 148 * 16;
    return (unsigned)b;
}

}  // namespace

ulsnn_status_t launch_splitk_reduce(const float* parts, int splits, int64_t M, int64_t N, int64_t ldp,
                                    float alpha, float beta, float* out, int64_t ldo, float* bias_out,
                                    cudaStream_t stream) {
    if (M <= 0 || N <= 0) return ULSNN_OK;
    splitk_reduce_kernel<<<grid_for(M * (N + 1), 256), 256, 0, stream>>>(parts, splits, M, N, ldp, alpha, beta, out, ldo, bias_out);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

ulsnn_status_t launch_colsum_reduce(const float* parts, int64_t tiles, int64_t N, int accumulate, float* out,
                                    cudaStream_t stream) {
    if (N <= 0) return ULSNN_OK;
    colsum_reduce_kernel<<<(unsigned)((N + CS_COLS - 1) / CS_COLS), CS_COLS * CS_LANES, 0, stream>>>(parts, tiles, N, accumulate, out);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

int rowstats_blocks(int64_t n) { return (int)((n + RS_ROWS - 1) / RS_ROWS); }

ulsnn_status_t launch_rowstats(const float2* stats, int64_t stats_ld, int tiles, const float* zlabel, int64_t n,
                               float* lse, float* chunk_tab, int64_t chunk_ld, int n_chunks, double* block_partials,
                               int accumulate, double* loss_out, cudaStream_t stream) {
    const int nb = rowstats_blocks(n);
    if (nb > 0) {
        rowstats_kernel<<<nb, RS_THREADS, 0, stream>>>(stats, stats_ld, tiles, zlabel, n, lse, chunk_tab, chunk_ld, n_chunks, block_partials);
        ulsnn::count_launch(2);
        if (cudaGetLastError() != cudaSuccess) return ULSNN_ERR_CUDA;
    }
    loss_final_kernel<<<1, 256, 0, stream>>>(block_partials, nb, accumulate, loss_out);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

ulsnn_status_t launch_rowsums(const float2* stats, int64_t stats_ld, int tiles, int64_t n, double* block_partials,
                              int accumulate, double* loss_out, cudaStream_t stream) {
    const int nb = (int)((n + RS_THREADS - 1) / RS_THREADS);        // never more than rowstats_blocks(n): the buffer fits
    if (nb > 0) {
        rowsums_kernel<<<nb, RS_THREADS, 0, stream>>>(stats, stats_ld, tiles, n, block_partials);
        ulsnn::count_launch(2);
        if (cudaGetLastError() != cudaSuccess) return ULSNN_ERR_CUDA;
    }
    loss_final_kernel<<<1, 256, 0, stream>>>(block_partials, nb, accumulate, loss_out);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

ulsnn_status_t launch_matrix_colsum(const float* A, const float* A_lo, int64_t lda, int64_t n, int64_t cols, float* parts,
                                    int accumulate, float* out, cudaStream_t stream) {
    const int tiles = (int)((n + DC_ROWS - 1) / DC_ROWS);
    if (tiles > 65535) return ULSNN_ERR_TOO_LARGE;
    if (tiles > 0) {
        dim3 grid((unsigned)((cols + 127) / 128), (unsigned)tiles);
        matrix_colsum_kernel<<<grid, 128, 0, stream>>>(A, A_lo, lda, n, cols, parts);
        ulsnn::count_launch(2);
        if (cudaGetLastError() != cudaSuccess) return ULSNN_ERR_CUDA;
    }
    return launch_colsum_reduce(parts, tiles, cols, accumulate, out, stream);
}

int delta_colsum_tiles(int64_t n) { return (int)((n + DC_ROWS - 1) / DC_ROWS); }

ulsnn_status_t launch_delta_colsum(const float* Z, int64_t ldz, const float* scale, int64_t scale_ld, const int32_t* labels,
                                   int64_t n, int64_t n_classes, float* parts, int accumulate, float* out,
                                   cudaStream_t stream) {
    const int tiles = delta_colsum_tiles(n);
    if (tiles > 65535) return ULSNN_ERR_TOO_LARGE;
    if (tiles > 0) {
        dim3 grid((unsigned)((n_classes + 127) / 128), (unsigned)tiles);
        delta_colsum_kernel<<<grid, 128, 0, stream>>>(Z, ldz, scale, scale_ld, labels, n, n_classes, parts);
        ulsnn::count_launch(2);
        if (cudaGetLastError() != cudaSuccess) return ULSNN_ERR_CUDA;
    }
    return launch_colsum_reduce(parts, tiles, n_classes, accumulate, out, stream);
}

ulsnn_status_t launch_delta_inplace(float* Z, int64_t ldz, const float* scale, int64_t scale_ld, const int32_t* labels,
                                    int64_t n, int64_t n_classes, cudaStream_t stream) {
    if (n <= 0) return ULSNN_OK;
    if ((ldz & 3) != 0 || (((uintptr_t)Z) & 15) != 0) return ULSNN_ERR_INVALID_ARG;
    delta_inplace_kernel<<<grid_for(n * (ldz >> 2), 256), 256, 0, stream>>>(Z, ldz, scale, scale_ld, labels, n, (int)n_classes);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

ulsnn_status_t launch_split_hilo(const float* x, int64_t n, float* hi, float* lo, cudaStream_t stream) {
    if (n <= 0) return ULSNN_OK;
    split_hilo_kernel<<<grid_for(n, 256), 256, 0, stream>>>(x, n, hi, lo);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

ulsnn_status_t launch_axpby(int64_t n, float a, const float* x, float b, const float* y, float* out, cudaStream_t stream) {
    if (n <= 0) return ULSNN_OK;
    axpby_kernel<<<grid_for(n, 256), 256, 0, stream>>>(n, a, x, b, y, out);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

int64_t dot_parts(int64_t n) { return n > 0 ? (n + DOT_BLOCK - 1) / DOT_BLOCK : 0; }

ulsnn_status_t launch_dot(int64_t n, const float* x, const float* y, double* out, double* parts, cudaStream_t stream) {
    const int64_t np = dot_parts(n);
    if (np > 0x7fffffff) return ULSNN_ERR_TOO_LARGE;
    if (np > 0) {
        dot_parts_kernel<<<(unsigned)np, 256, 0, stream>>>(n, x, y, parts);
        ulsnn::count_launch(2);
        if (cudaGetLastError() != cudaSuccess) return ULSNN_ERR_CUDA;
    }
    dot_final_kernel<<<1, 256, 0, stream>>>(parts, np, out);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

ulsnn_status_t launch_sgd_multi(const SgdBatch& b, float lr, cudaStream_t stream) {
    if (b.count <= 0) return ULSNN_OK;
    if (b.count > SgdBatch::MAX) return ULSNN_ERR_INVALID_ARG;
    int64_t nmax = 0;
    for (int i = 0; i < b.count; ++i) if (b.n[i] > nmax) nmax = b.n[i];
    if (nmax <= 0) return ULSNN_OK;
    int64_t bx = (nmax + 4 * 256 - 1) / (4 * 256);          // about four elements per thread of the largest tensor
    if (bx > 148 * 8) bx = 148 * 8;
    sgd_multi_kernel<<<dim3((unsigned)bx, (unsigned)b.count), 256, 0, stream>>>(b, lr);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

ulsnn_status_t launch_zero(float* p, int64_t n, cudaStream_t stream) {
    if (n <= 0) return ULSNN_OK;
    zero_kernel<float><<<grid_for(n, 256), 256, 0, stream>>>(p, n);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

ulsnn_status_t launch_zero_f64(double* p, int64_t n, cudaStream_t stream) {
    if (n <= 0) return ULSNN_OK;
    zero_kernel<double><<<grid_for(n, 256), 256, 0, stream>>>(p, n);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

// Re-buffering of an operand the tensor-core path cannot address (Section 3.3 copies B' into a buffer laid out for
// the kernel; here the reason is TMA's need for 16-byte aligned rows): dst[r][c] = src[r][c] for c < cols, 0 in the
// padding up to ldd (a multiple of 4).  One warp per 128-column piece of a row, rows strided over the grid; the reads
// are 4-byte (the source rows are not aligned), the writes 16-byte.
__global__ void pack_rows_kernel(const float* __restrict__ src, int64_t rows, int64_t cols, int64_t lds,
                                 float* __restrict__ dst, int64_t ldd) {
    const int lane = threadIdx.x & 31;
    const int64_t pieces = (ldd + 127) / 128;
    const int64_t total = rows * pieces;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t w = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); w < total; w += warps) {
        const int64_t r = w / pieces, c0 = (w % pieces) * 128 + 4 * lane;
        if (c0 >= ldd) continue;
        const float* s = src + r * lds + c0;
        float4 v;
        v.x = c0 + 0 < cols ? __ldg(s + 0) : 0.f;
        v.y = c0 + 1 < cols ? __ldg(s + 1) : 0.f;
        v.z = c0 + 2 < cols ? __ldg(s + 2) : 0.f;
        v.w = c0 + 3 < cols ? __ldg(s + 3) : 0.f;
        *reinterpret_cast<float4*>(dst + r * ldd + c0) = v;
    }
}

ulsnn_status_t launch_pack_rows(const float* src, int64_t rows, int64_t cols, int64_t lds, float* dst, int64_t ldd,
                                cudaStream_t stream) {
    if (rows <= 0 || cols <= 0) return ULSNN_OK;
    const int64_t pieces = rows * ((ldd + 127) / 128);
    int64_t blocks = (pieces + 7) / 8;
    if (blocks > 148 * 32) blocks = 148 * 32;
    pack_rows_kernel<<<(unsigned)blocks, 256, 0, stream>>>(src, rows, cols, lds, dst, ldd);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

ulsnn_status_t launch_scale_rows(float* C, int64_t M, int64_t N, int64_t ldc, float beta, cudaStream_t stream) {
    if (M <= 0 || N <= 0) return ULSNN_OK;
    scale_rows_kernel<<<grid_for(M * N, 256), 256, 0, stream>>>(C, M, N, ldc, beta);
    ulsnn::count_launch(2);
    return cuda_ok(cudaGetLastError());
}

}  // namespace ulsnn

extern "C" ulsnn_status_t ulsnn_fill_uniform(float* dst, int64_t n, uint64_t seed, uint64_t tensor_id, uint64_t offset,
                                             int mode, ulsnn_stream_t stream) {
    if (n < 0 || (n > 0 && !dst) || (mode != 0 && mode != 1)) return ULSNN_ERR_INVALID_ARG;
    if (n == 0) return ULSNN_OK;
    ulsnn::fill_uniform_kernel<<<ulsnn::grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(dst, n, seed, tensor_id, offset, mode);
    ulsnn::count_launch(3);
    return ulsnn::cuda_ok(cudaGetLastError());
}

extern "C" ulsnn_status_t ulsnn_fill_labels(int32_t* dst, int64_t n, uint64_t seed, uint64_t tensor_id, uint64_t offset,
                                            int32_t n_classes, ulsnn_stream_t stream) {
    if (n < 0 || (n > 0 && !dst) || n_classes < 1) return ULSNN_ERR_INVALID_ARG;
    if (n == 0) return ULSNN_OK;
    ulsnn::fill_labels_kernel<<<ulsnn::grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(dst, n, seed, tensor_id, offset, (uint32_t)n_classes);
    ulsnn::count_launch(3);
    return ulsnn::cuda_ok(cudaGetLastError());
}
