// FFMA engine: exact-fp32 products on the CUDA cores (ULSNN_MATH_FP32_SIMT).
//
// It is the comparison kernel for the tensor-core engine, the route for operands that TMA cannot
// address, and it carries the same fused epilogues.  128x128x16 tiles, 256 threads, 8x8 outputs per
// thread, register-staged double buffering.  Operands are addressed by two strides each, so all four
// transpose forms of Section 3.1 are the same kernel.
#include "common.cuh"
#include <math.h>

namespace ulsnn {

namespace {

constexpr int BM = 128, BN = 128, BK = 16, NT = 256, LDS = BM + 4;

struct Tile { float a[2][BK][LDS]; float b[2][BK][LDS]; };

template <bool TRANSFORM>
__device__ __forceinline__ float load_a(const GemmDesc& d, int64_t i, int64_t k, int64_t kend) {
    if (i >= d.M || k >= kend) return 0.f;
    float z = __ldg(d.A + i * d.a_sm + k * d.a_sk);
    if (d.A_lo) z += __ldg(d.A_lo + i * d.a_sm + k * d.a_sk);
    if (TRANSFORM) {
        const int64_t p = d.a_pattern_is_m ? i : k;
        const int64_t c = d.a_pattern_is_m ? k : i;
        z = z * __ldg(d.scale + p * d.scale_ld + (c >> 5)) - ((int64_t)__ldg(d.labels + p) == c ? 1.f : 0.f);
    }
    return z;
}

__device__ __forceinline__ float load_b(const GemmDesc& d, int64_t k, int64_t j, int64_t kend) {
    if (j >= d.N || k >= kend) return 0.f;
    float v = __ldg(d.B + k * d.b_sk + j * d.b_sn);
    if (d.B_lo) v += __ldg(d.B_lo + k * d.b_sk + j * d.b_sn);
    return v;
}

template <int EPI, bool TRANSFORM>
__global__ void __launch_bounds__(NT, 2) simt_gemm_kernel(const GemmDesc d) {
    __shared__ Tile sm;
    const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
    const int64_t m0 = (int64_t)blockIdx.x * BM, n0 = (int64_t)blockIdx.y * BN;
    const int64_t kbeg = (int64_t)blockIdx.z * d.k_per_split;
    const int64_t kend = (EPI == EPI_PARTIAL) ? min(d.K, kbeg + d.k_per_split) : d.K;
    const bool a_kc = (d.a_sk == 1), b_nc = (d.b_sn == 1);

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    // Staging of the next k tile in registers.  When an operand tile lies inside the matrix and its rows are 16-byte
    // aligned, each thread fetches two float4 along the contiguous direction; otherwise eight guarded scalars.
    const bool a_vec = !d.A_lo && ((((uintptr_t)d.A) & 15) == 0) &&
                       (a_kc ? ((d.a_sm & 3) == 0) : ((d.a_sk & 3) == 0)) && (m0 + BM <= d.M) &&
                       (!TRANSFORM || a_kc == (d.a_pattern_is_m != 0));      // logits: the class is the contiguous index
    const bool b_vec = !d.B_lo && ((((uintptr_t)d.B) & 15) == 0) &&
                       (b_nc ? ((d.b_sk & 3) == 0) : ((d.b_sn & 3) == 0)) && (n0 + BN <= d.N);
    float ra[8], rb[8];
    bool va = false, vb = false;        // how the staged registers were fetched
    auto fetch = [&](int64_t k0) {
        const bool kfull = k0 + BK <= kend;
        va = a_vec && kfull; vb = b_vec && kfull;
        if (va) {
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int e = t + NT * i;                                   // float4 index in the 128 x 16 tile
                const int am = a_kc ? (e >> 2) : ((e & 31) << 2), ak = a_kc ? ((e & 3) << 2) : (e >> 5);
                const float4 v = __ldg(reinterpret_cast<const float4*>(d.A + (m0 + am) * d.a_sm + (k0 + ak) * d.a_sk));
                ra[4 * i] = v.x; ra[4 * i + 1] = v.y; ra[4 * i + 2] = v.z; ra[4 * i + 3] = v.w;
                if (TRANSFORM) {
                    // the four values run along the contiguous direction, which is the class: one pattern and one
                    // 32-class chunk (cls is a multiple of 4) for all four
                    const int64_t pat = d.a_pattern_is_m ? m0 + am : k0 + ak;
                    const int64_t cls = d.a_pattern_is_m ? k0 + ak : m0 + am;
                    const float sc = __ldg(d.scale + pat * d.scale_ld + (cls >> 5));
                    const int64_t lab = (int64_t)__ldg(d.labels + pat);
#pragma unroll
                    for (int j = 0; j < 4; ++j) ra[4 * i + j] = ra[4 * i + j] * sc - (cls + j == lab ? 1.f : 0.f);
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int e = t + NT * i;
                const int am = a_kc ? (e >> 4) : (e & 127), ak = a_kc ? (e & 15) : (e >> 7);
                ra[i] = load_a<TRANSFORM>(d, m0 + am, k0 + ak, kend);
            }
        }
        if (vb) {
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int e = t + NT * i;
                const int bn = b_nc ? ((e & 31) << 2) : (e >> 2), bk = b_nc ? (e >> 5) : ((e & 3) << 2);
                const float4 v = __ldg(reinterpret_cast<const float4*>(d.B + (k0 + bk) * d.b_sk + (n0 + bn) * d.b_sn));
                rb[4 * i] = v.x; rb[4 * i + 1] = v.y; rb[4 * i + 2] = v.z; rb[4 * i + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int e = t + NT * i;
                const int bn = b_nc ? (e & 127) : (e >> 4), bk = b_nc ? (e >> 7) : (e & 15);
                rb[i] = load_b(d, k0 + bk, n0 + bn, kend);
            }
        }
    };
    auto stash = [&](int buf) {
        if (va) {
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int e = t + NT * i;
                if (a_kc) {         // four consecutive k of one row: a transposing store
                    const int am = e >> 2, ak = (e & 3) << 2;
#pragma unroll
                    for (int j = 0; j < 4; ++j) sm.a[buf][ak + j][am] = ra[4 * i + j];
                } else {            // four consecutive rows of one k
                    const int am = (e & 31) << 2, ak = e >> 5;
                    *reinterpret_cast<float4*>(&sm.a[buf][ak][am]) = make_float4(ra[4 * i], ra[4 * i + 1], ra[4 * i + 2], ra[4 * i + 3]);
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int e = t + NT * i;
                const int am = a_kc ? (e >> 4) : (e & 127), ak = a_kc ? (e & 15) : (e >> 7);
                sm.a[buf][ak][am] = ra[i];
            }
        }
        if (vb) {
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int e = t + NT * i;
                if (b_nc) {
                    const int bn = (e & 31) << 2, bk = e >> 5;
                    *reinterpret_cast<float4*>(&sm.b[buf][bk][bn]) = make_float4(rb[4 * i], rb[4 * i + 1], rb[4 * i + 2], rb[4 * i + 3]);
                } else {
                    const int bn = e >> 2, bk = (e & 3) << 2;
#pragma unroll
                    for (int j = 0; j < 4; ++j) sm.b[buf][bk + j][bn] = rb[4 * i + j];
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int e = t + NT * i;
                const int bn = b_nc ? (e & 127) : (e >> 4), bk = b_nc ? (e >> 7) : (e & 15);
                sm.b[buf][bk][bn] = rb[i];
            }
        }
    };

    const int64_t nk = (kend > kbeg) ? (kend - kbeg + BK - 1) / BK : 0;
    if (nk > 0) { fetch(kbeg); stash(0); }
    __syncthreads();
    for (int64_t kt = 0; kt < nk; ++kt) {
        const int buf = (int)(kt & 1);
        if (kt + 1 < nk) fetch(kbeg + (kt + 1) * BK);
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            const float4 a0 = *reinterpret_cast<const float4*>(&sm.a[buf][kk][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4*>(&sm.a[buf][kk][64 + ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&sm.b[buf][kk][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&sm.b[buf][kk][64 + tx * 4]);
            const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        if (kt + 1 < nk) stash(buf ^ 1);
        __syncthreads();
    }

    // ---------------------------------------------------------------- epilogue
    auto row_of = [&](int i) -> int64_t { return m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4)); };
    auto col_of = [&](int j) -> int64_t { return n0 + (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4)); };

    if (EPI == EPI_SGEMM) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int64_t r = row_of(i);
            if (r >= d.M) continue;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t c = col_of(j);
                if (c >= d.N) continue;
                float* out = d.C + r * d.ldc + c;
                float v = d.alpha * acc[i][j];
                if (d.beta != 0.f) v = fmaf(d.beta, *out, v);
                *out = v;
            }
        }
    } else if (EPI == EPI_PARTIAL) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int64_t r = row_of(i);
            if (r >= d.M) continue;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t c = col_of(j);
                if (c < d.N) d.partials[((int64_t)blockIdx.z * d.M + r) * d.ldp + c] = acc[i][j];
            }
        }
    } else if (EPI == EPI_BIAS_TANH) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int64_t r = row_of(i);
            if (r >= d.M) continue;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t c = col_of(j);
                if (c < d.N) {
                    const float h = tanhf(acc[i][j] + __ldg(d.bias + c));
                    if (d.C_lo) {
                        const float hi = __uint_as_float((__float_as_uint(h) + 0x1000u) & 0xFFFFE000u);
                        d.C[r * d.ldc + c] = hi;
                        d.C_lo[r * d.ldc + c] = __uint_as_float((__float_as_uint(h - hi) + 0x1000u) & 0xFFFFE000u);
                    } else {
                        d.C[r * d.ldc + c] = h;
                    }
                }
            }
            if (d.ones_cols > 0 && tx == 0 && blockIdx.y == gridDim.y - 1) {
                d.C[r * d.ldc + d.N] = 1.f;
                for (int c = 1; c < d.ones_cols; ++c) d.C[r * d.ldc + d.N + c] = 0.f;
                if (d.C_lo) for (int c = 0; c < d.ones_cols; ++c) d.C_lo[r * d.ldc + d.N + c] = 0.f;
            }
        }
    } else if (EPI == EPI_LOGITS) {
        // Threads tx = 0..15 of one ty share a row and sit in one half-warp: xor-shuffles 8,4,2,1 stay inside it.
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int64_t r = row_of(i);
            const bool rv = r < d.M;
            float v[8];
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t c = col_of(j);
                v[j] = (c < d.N) ? acc[i][j] + __ldg(d.bias + c) : -INFINITY;
                mx = fmaxf(mx, v[j]);
            }
#pragma unroll
            for (int o = 8; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            float s = 0.f, e[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) { e[j] = (v[j] == -INFINITY) ? 0.f : expf(v[j] - mx); s += e[j]; }
#pragma unroll
            for (int o = 8; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (rv) {
                if (tx == 0) {
                    d.stats[r * d.stats_ld + blockIdx.y] = make_float2(mx, s);
                    // the stored exponentials of this tile's four 32-column chunks all refer to the tile maximum
                    if (d.chunk_max)
                        for (int q = 0; q < BN / 32; ++q)
                            if (n0 + 32 * q < d.N) d.chunk_max[r * d.chunk_ld + (n0 >> 5) + q] = mx;
                }
                const int64_t lab = (int64_t)__ldg(d.labels + r);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int64_t c = col_of(j);
                    if (c < d.N) {
                        if (d.C) d.C[r * d.ldc + c] = e[j];
                        if (c == lab) d.zlabel[r] = v[j];
                    }
                }
            }
        }
    } else if (EPI == EPI_TANH_SSE) {
        // Threads tx = 0..15 of one ty share a row and sit in one half-warp (as in the logits epilogue).
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int64_t r = row_of(i);
            const bool rv = r < d.M;
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t c = col_of(j);
                if (rv && c < d.N) {
                    const float y = tanhf(acc[i][j] + __ldg(d.bias + c));
                    const float e = y - __ldg(d.T + r * d.ldt + c);
                    s += e * e;
                    if (d.C) {
                        const float g = 2.f * e * (1.f - y * y);
                        if (d.C_lo) {
                            const float hi = __uint_as_float((__float_as_uint(g) + 0x1000u) & 0xFFFFE000u);
                            d.C[r * d.ldc + c] = hi;
                            d.C_lo[r * d.ldc + c] = __uint_as_float((__float_as_uint(g - hi) + 0x1000u) & 0xFFFFE000u);
                        } else {
                            d.C[r * d.ldc + c] = g;
                        }
                    }
                }
            }
#pragma unroll
            for (int o = 8; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (rv && tx == 0) d.stats[r * d.stats_ld + blockIdx.y] = make_float2(0.f, s);
        }
    } else if (EPI == EPI_TANHP) {
        float cs[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) cs[j] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int64_t r = row_of(i);
            if (r >= d.M) continue;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t c = col_of(j);
                if (c >= d.N) continue;
                float h = __ldg(d.Hm + r * d.ldh + c);
                if (d.Hm_lo) h += __ldg(d.Hm_lo + r * d.ldh + c);
                const float o = (1.f - h * h) * acc[i][j];
                d.C[r * d.ldc + c] = o;
                cs[j] += o;
            }
        }
        if (d.colsum_part) {
            // fixed-order column sums of this 128-row tile: 16 row groups, summed in index order
            float* red = &sm.a[0][0][0];          // 16 x 128 floats, the operand tiles are no longer needed
            __syncthreads();
#pragma unroll
            for (int j = 0; j < 8; ++j) red[ty * BN + (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4))] = cs[j];
            __syncthreads();
            if (t < BN && n0 + t < d.N) {
                float s = 0.f;
#pragma unroll
                for (int g = 0; g < 16; ++g) s += red[g * BN + t];
                d.colsum_part[(int64_t)blockIdx.x * d.N + n0 + t] = s;
            }
        }
    }
}

template <int EPI, bool TR>
ulsnn_status_t launch(const GemmDesc& d, cudaStream_t stream) {
    const int64_t tm = (d.M + BM - 1) / BM, tn = (d.N + BN - 1) / BN;
    const int splits = (EPI == EPI_PARTIAL) ? d.splits : 1;
    if (tm <= 0 || tn <= 0 || tm > 0x7fffffff || tn > 65535 || splits < 1 || splits > 65535) return ULSNN_ERR_INVALID_ARG;
    dim3 grid((unsigned)tm, (unsigned)tn, (unsigned)splits);
    simt_gemm_kernel<EPI, TR><<<grid, NT, 0, stream>>>(d);
    count_launch(0);
    return cuda_ok(cudaGetLastError());
}

}  // namespace

int simt_tile_m() { return BM; }
int simt_tile_n() { return BN; }
int simt_slots() { return 148; }
int simt_colsum_groups() { return 1; }

ulsnn_status_t simt_gemm_launch(const GemmDesc& d, cudaStream_t stream) {
    if (d.M <= 0 || d.N <= 0) return ULSNN_OK;
    const bool tr = d.a_transform != 0;
    switch (d.epi) {
        case EPI_SGEMM:     return tr ? ULSNN_ERR_INVALID_ARG : launch<EPI_SGEMM, false>(d, stream);
        case EPI_BIAS_TANH: return tr ? ULSNN_ERR_INVALID_ARG : launch<EPI_BIAS_TANH, false>(d, stream);
        case EPI_LOGITS:    return tr ? ULSNN_ERR_INVALID_ARG : launch<EPI_LOGITS, false>(d, stream);
        case EPI_TANHP:     return tr ? launch<EPI_TANHP, true>(d, stream) : launch<EPI_TANHP, false>(d, stream);
        case EPI_PARTIAL:   return tr ? launch<EPI_PARTIAL, true>(d, stream) : launch<EPI_PARTIAL, false>(d, stream);
        case EPI_TANH_SSE:  return tr ? ULSNN_ERR_INVALID_ARG : launch<EPI_TANH_SSE, false>(d, stream);
    }
    return ULSNN_ERR_INVALID_ARG;
}

}  // namespace ulsnn
