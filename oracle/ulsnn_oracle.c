/*
 * CPU checker ("oracle") for the error-and-gradient evaluation of a fully
 * connected network and for SGEMM.  TEST INFRASTRUCTURE ONLY: the product
 * library never links, loads or calls anything in this file.
 *
 * Everything is the plain definition written out in double precision on the
 * fp32 input bits: a triple-loop matrix product (Section 3.1: C = alpha*A*B +
 * beta*C, 2MNK flops) and explicit per-pattern back-propagation (Section 4.1,
 * Eqs. 1-3; the matrix identities of Section 4.2 are NOT used here, so that
 * this code shares no structure with the GPU path, which is built from them).
 * No blocking, no fusion, no reordering.  Sums over patterns are plain sums
 * with no 1/n factor (Eq. 3).
 *
 * Parity status: every function here is pinned by tests that do not come from
 * this file (brute-force integer products, central finite differences, the
 * all-zero-weights closed form, softmax row sums, additivity over patterns,
 * the matrix identities of Section 4.2).  Nothing is "parity unpinned".
 *
 * Matrices are row-major; a leading dimension is the distance in elements
 * between consecutive rows (Section 3.4 calls it the stride).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* op(A)[i][k] for row-major storage: 'N' -> A[i*lda+k], 'T' -> A[k*lda+i]. */
static inline double opa(const float* A, int64_t lda, int trans, int64_t i, int64_t k) {
    return trans ? (double)A[k * lda + i] : (double)A[i * lda + k];
}

/*
 * Section 3.1: C_out[i][j] = alpha * sum_k op(A)[i][k] * op(B)[k][j] + beta * C_in[i][j].
 * op(A) is M x K, op(B) is K x N.  Inputs fp32, sum and result in double.
 * beta == 0: C_in is never read (may be NULL or hold NaN).  alpha == 0: A, B never read.
 * C_out is dense M x N (leading dimension N).
 */
void oracle_sgemm(int transA, int transB, int64_t M, int64_t N, int64_t K, double alpha,
                  const float* A, int64_t lda, const float* B, int64_t ldb,
                  double beta, const float* C_in, int64_t ldc, double* C_out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double s = 0.0;
            if (alpha != 0.0) {
                for (int64_t k = 0; k < K; ++k) s += opa(A, lda, transA, i, k) * opa(B, ldb, !transB, j, k);
                s *= alpha;
            }
            if (beta != 0.0) s += beta * (double)C_in[i * ldc + j];
            C_out[i * N + j] = s;
        }
    }
}

/* One entry of the product above (for sampled checks of large products). */
double oracle_sgemm_entry(int transA, int transB, int64_t K, double alpha,
                          const float* A, int64_t lda, const float* B, int64_t ldb,
                          double beta, const float* C_in, int64_t ldc, int64_t i, int64_t j) {
    double s = 0.0;
    if (alpha != 0.0) {
        for (int64_t k = 0; k < K; ++k) s += opa(A, lda, transA, i, k) * opa(B, ldb, !transB, j, k);
        s *= alpha;
    }
    if (beta != 0.0) s += beta * (double)C_in[i * ldc + j];
    return s;
}

/*
 * Magnitude sums of the product above: |alpha| * sum_k |op(A)[i][k]| * |op(B)[k][j]| + |beta| * |C_in[i][j]|.
 * This is the quantity a floating-point evaluation's forward error is proportional to (the error of a sum
 * is bounded by a multiple of the unit roundoff times the sum of the magnitudes of its terms); the ratio of
 * its norm to the norm of the product itself is the product's condition number under cancellation.
 */
void oracle_sgemm_abs(int transA, int transB, int64_t M, int64_t N, int64_t K, double alpha,
                      const float* A, int64_t lda, const float* B, int64_t ldb,
                      double beta, const float* C_in, int64_t ldc, double* out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double s = 0.0;
            if (alpha != 0.0) {
                for (int64_t k = 0; k < K; ++k) s += fabs(opa(A, lda, transA, i, k)) * fabs(opa(B, ldb, !transB, j, k));
                s *= fabs(alpha);
            }
            if (beta != 0.0) s += fabs(beta) * fabs((double)C_in[i * ldc + j]);
            out[i * N + j] = s;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Network description: sizes[0..L], W_l is [sizes[l+1] x sizes[l]] row-major  */
/* (w_jk: j = unit of the next layer, k = unit of this one, Eqs. 1-2), all W_l */
/* concatenated in Wflat, all b_l in bflat.                                    */
/* ------------------------------------------------------------------------- */

typedef struct {
    int L;
    const int32_t* sizes;
    int64_t woff[17], boff[17];
    int64_t nw, nb, maxw;
} net_t;

static int net_init(net_t* n, int L, const int32_t* sizes) {
    if (L < 1 || L > 16) return -1;
    n->L = L; n->sizes = sizes; n->nw = 0; n->nb = 0; n->maxw = 0;
    for (int l = 0; l < L; ++l) {
        n->woff[l] = n->nw; n->boff[l] = n->nb;
        n->nw += (int64_t)sizes[l] * sizes[l + 1];
        n->nb += sizes[l + 1];
    }
    for (int l = 0; l <= L; ++l) if (sizes[l] > n->maxw) n->maxw = sizes[l];
    return 0;
}

/*
 * Forward pass of one pattern.  act[0] = x; hidden layers use tanh (Eq. 2);
 * the last layer's pre-activations z are returned in act[L].
 */
static void forward_one(const net_t* n, const float* Wflat, const float* bflat,
                        const float* x, double** act) {
    for (int k = 0; k < n->sizes[0]; ++k) act[0][k] = (double)x[k];
    for (int l = 0; l < n->L; ++l) {
        const int nin = n->sizes[l], nout = n->sizes[l + 1];
        const float* W = Wflat + n->woff[l];
        const float* b = bflat + n->boff[l];
        for (int j = 0; j < nout; ++j) {
            double s = (double)b[j];
            for (int k = 0; k < nin; ++k) s += (double)W[(int64_t)j * nin + k] * act[l][k];
            act[l + 1][j] = (l + 1 < n->L) ? tanh(s) : s;
        }
    }
}

/* Softmax + cross-entropy head: returns lse - z_label, writes delta = softmax(z) - onehot. */
static double head_softmax_ce(const double* z, int no, int label, double* delta) {
    double m = z[0];
    for (int j = 1; j < no; ++j) if (z[j] > m) m = z[j];
    double s = 0.0;
    for (int j = 0; j < no; ++j) s += exp(z[j] - m);
    const double lse = m + log(s);
    if (delta) {
        for (int j = 0; j < no; ++j) delta[j] = exp(z[j] - lse);
        delta[label] -= 1.0;
    }
    return lse - z[label];
}

/*
 * Paper's head (Eqs. 1 and 3): y = tanh(z), E = sum_j (y_j - t_j)^2.
 * delta = dE/dz = 2 (y - t)(1 - y^2).  (Section 4.2's Y_Delta = (1-Y*Y)*(T-Y) is -1/2 of this.)
 */
static double head_tanh_sse(const double* z, int no, const float* t, double* delta) {
    double e = 0.0;
    for (int j = 0; j < no; ++j) {
        const double y = tanh(z[j]);
        const double d = y - (double)t[j];
        e += d * d;
        if (delta) delta[j] = 2.0 * d * (1.0 - y * y);
    }
    return e;
}

/* Back-propagate delta[L] down to layer 1 and add this pattern's outer products. */
static void backward_one(const net_t* n, const float* Wflat, double** act, double** delta,
                         double* dW, double* db) {
    for (int l = n->L - 1; l >= 0; --l) {
        const int nin = n->sizes[l], nout = n->sizes[l + 1];
        double* dWl = dW + n->woff[l];
        double* dbl = db + n->boff[l];
        const double* d = delta[l + 1];
        for (int j = 0; j < nout; ++j) {
            const double dj = d[j];
            dbl[j] += dj;
            double* row = dWl + (int64_t)j * nin;
            for (int k = 0; k < nin; ++k) row[k] += dj * act[l][k];
        }
        if (l > 0) {   /* delta of hidden layer l: (1 - h^2) * (W_{l+1}^T delta_{l+1}) */
            const float* W = Wflat + n->woff[l];
            for (int k = 0; k < nin; ++k) {
                double s = 0.0;
                for (int j = 0; j < nout; ++j) s += (double)W[(int64_t)j * nin + k] * d[j];
                const double h = act[l][k];
                delta[l][k] = (1.0 - h * h) * s;
            }
        }
    }
}

/*
 * The same back-propagation with every term of every sum taken in absolute value: mag[L] holds the magnitudes
 * of the output deltas' terms, mag[l][k] = (1 - h^2) * sum_j |w_jk| mag[l+1][j], and the pattern adds
 * mag[l+1][j] * |act[l][k]| to aW and mag[l+1][j] to ab.  The results bound what rounding errors anywhere in
 * the evaluation can do to the summed gradient (they are what the errors are proportional to); they are never
 * smaller than the magnitudes of the gradient's own entries.
 */
static void backward_one_abs(const net_t* n, const float* Wflat, double** act, double** mag,
                             double* aW, double* ab) {
    for (int l = n->L - 1; l >= 0; --l) {
        const int nin = n->sizes[l], nout = n->sizes[l + 1];
        double* aWl = aW + n->woff[l];
        double* abl = ab + n->boff[l];
        const double* d = mag[l + 1];
        for (int j = 0; j < nout; ++j) {
            const double dj = d[j];
            abl[j] += dj;
            double* row = aWl + (int64_t)j * nin;
            for (int k = 0; k < nin; ++k) row[k] += dj * fabs(act[l][k]);
        }
        if (l > 0) {
            const float* W = Wflat + n->woff[l];
            for (int k = 0; k < nin; ++k) {
                double s = 0.0;
                for (int j = 0; j < nout; ++j) s += fabs((double)W[(int64_t)j * nin + k]) * d[j];
                const double h = act[l][k];
                mag[l][k] = (1.0 - h * h) * s;
            }
        }
    }
}

static double** alloc_layers(const net_t* n) {
    double** a = (double**)malloc(sizeof(double*) * (n->L + 1));
    for (int l = 0; l <= n->L; ++l) a[l] = (double*)malloc(sizeof(double) * n->sizes[l]);
    return a;
}
static void free_layers(const net_t* n, double** a) {
    for (int l = 0; l <= n->L; ++l) free(a[l]);
    free(a);
}

/*
 * Summed loss (and, if want_grad, summed dW/db) over n_patterns patterns.
 * head == 0: softmax + cross-entropy with int32 labels; head == 1: tanh + summed
 * squared error with a dense fp32 target matrix T [n_patterns x sizes[L]] (ldt).
 * OpenMP over patterns; one private double gradient per thread, combined in
 * thread-index order.  Returns 0, or -1 on a bad description.
 */
static int run(int L, const int32_t* sizes, const float* Wflat, const float* bflat,
               const float* X, int64_t ldx, const int32_t* labels, const float* T, int64_t ldt,
               int64_t n_patterns, int head, int want_grad,
               double* dW, double* db, double* loss_out) {
    net_t n;
    if (net_init(&n, L, sizes)) return -1;
    int nthreads = oracle_num_threads();
    if (nthreads > n_patterns) nthreads = n_patterns > 0 ? (int)n_patterns : 1;
    double* gW = NULL; double* gb = NULL;
    double* losses = (double*)calloc(nthreads, sizeof(double));
    if (want_grad) {
        gW = (double*)calloc((size_t)nthreads * n.nw, sizeof(double));
        gb = (double*)calloc((size_t)nthreads * n.nb, sizeof(double));
    }
#pragma omp parallel num_threads(nthreads)
    {
#ifdef _OPENMP
        const int t = omp_get_thread_num();
#else
        const int t = 0;
#endif
        double** act = alloc_layers(&n);
        double** delta = alloc_layers(&n);
        const int64_t p0 = n_patterns * t / nthreads, p1 = n_patterns * (t + 1) / nthreads;
        double loss = 0.0;
        for (int64_t p = p0; p < p1; ++p) {
            forward_one(&n, Wflat, bflat, X + p * ldx, act);
            double* dl = want_grad ? delta[L] : NULL;
            if (head == 0) loss += head_softmax_ce(act[L], sizes[L], labels[p], dl);
            else           loss += head_tanh_sse(act[L], sizes[L], T + p * ldt, dl);
            if (want_grad) backward_one(&n, Wflat, act, delta, gW + (size_t)t * n.nw, gb + (size_t)t * n.nb);
        }
        losses[t] = loss;
        free_layers(&n, act);
        free_layers(&n, delta);
    }
    double loss = 0.0;
    for (int t = 0; t < nthreads; ++t) loss += losses[t];
    *loss_out = loss;
    if (want_grad) {
        for (int64_t i = 0; i < n.nw; ++i) { double s = 0.0; for (int t = 0; t < nthreads; ++t) s += gW[(size_t)t * n.nw + i]; dW[i] = s; }
        for (int64_t i = 0; i < n.nb; ++i) { double s = 0.0; for (int t = 0; t < nthreads; ++t) s += gb[(size_t)t * n.nb + i]; db[i] = s; }
        free(gW); free(gb);
    }
    free(losses);
    return 0;
}

int oracle_mlp_forward_loss(int L, const int32_t* sizes, const float* Wflat, const float* bflat,
                            const float* X, int64_t ldx, const int32_t* labels, int64_t n_patterns,
                            double* loss_out) {
    return run(L, sizes, Wflat, bflat, X, ldx, labels, NULL, 0, n_patterns, 0, 0, NULL, NULL, loss_out);
}

int oracle_mlp_gradient(int L, const int32_t* sizes, const float* Wflat, const float* bflat,
                        const float* X, int64_t ldx, const int32_t* labels, int64_t n_patterns,
                        double* dW, double* db, double* loss_out) {
    return run(L, sizes, Wflat, bflat, X, ldx, labels, NULL, 0, n_patterns, 0, 1, dW, db, loss_out);
}

/* The paper's own network: tanh output units and summed squared error (Eqs. 1 and 3). */
int oracle_mlp_sse_gradient(int L, const int32_t* sizes, const float* Wflat, const float* bflat,
                            const float* X, int64_t ldx, const float* T, int64_t ldt, int64_t n_patterns,
                            int want_grad, double* dW, double* db, double* loss_out) {
    return run(L, sizes, Wflat, bflat, X, ldx, NULL, T, ldt, n_patterns, 1, want_grad, dW, db, loss_out);
}

/*
 * Per-pattern quantities of the softmax head, for invariants and for sampled
 * checks: probs[p][j] = softmax(z_p)_j (dense, n_patterns x sizes[L]) and the
 * last hidden activations hid[p][k] (n_patterns x sizes[L-1]); either may be NULL.
 */
int oracle_mlp_probe(int L, const int32_t* sizes, const float* Wflat, const float* bflat,
                     const float* X, int64_t ldx, int64_t n_patterns, double* probs, double* hid) {
    net_t n;
    if (net_init(&n, L, sizes)) return -1;
#pragma omp parallel
    {
        double** act = alloc_layers(&n);
        double* d = (double*)malloc(sizeof(double) * sizes[L]);
#pragma omp for schedule(static)
        for (int64_t p = 0; p < n_patterns; ++p) {
            forward_one(&n, Wflat, bflat, X + p * ldx, act);
            if (probs) {
                head_softmax_ce(act[L], sizes[L], 0, d);
                d[0] += 1.0;
                memcpy(probs + p * sizes[L], d, sizeof(double) * sizes[L]);
            }
            if (hid) memcpy(hid + p * sizes[L - 1], act[L - 1], sizeof(double) * sizes[L - 1]);
        }
        free(d);
        free_layers(&n, act);
    }
    return 0;
}

/*
 * Magnitude sums of the summed gradient (see backward_one_abs).  head == 0: the output deltas softmax(z) - onehot
 * enter as softmax(z) + onehot (the subtraction at the label is a cancellation too); head == 1: as |dE/dz|.
 * aW, ab have the layout of dW, db.
 */
int oracle_mlp_gradient_abs(int L, const int32_t* sizes, const float* Wflat, const float* bflat,
                            const float* X, int64_t ldx, const int32_t* labels, const float* T, int64_t ldt,
                            int64_t n_patterns, int head, double* aW, double* ab) {
    net_t n;
    if (net_init(&n, L, sizes)) return -1;
    int nthreads = oracle_num_threads();
    if (nthreads > n_patterns) nthreads = n_patterns > 0 ? (int)n_patterns : 1;
    double* gW = (double*)calloc((size_t)nthreads * n.nw, sizeof(double));
    double* gb = (double*)calloc((size_t)nthreads * n.nb, sizeof(double));
#pragma omp parallel num_threads(nthreads)
    {
#ifdef _OPENMP
        const int t = omp_get_thread_num();
#else
        const int t = 0;
#endif
        double** act = alloc_layers(&n);
        double** mag = alloc_layers(&n);
        const int64_t p0 = n_patterns * t / nthreads, p1 = n_patterns * (t + 1) / nthreads;
        for (int64_t p = p0; p < p1; ++p) {
            forward_one(&n, Wflat, bflat, X + p * ldx, act);
            if (head == 0) {
                head_softmax_ce(act[L], sizes[L], labels[p], mag[L]);
                mag[L][labels[p]] += 2.0;                   /* (softmax - 1) + 2 = softmax + 1 */
            } else {
                head_tanh_sse(act[L], sizes[L], T + p * ldt, mag[L]);
                for (int j = 0; j < sizes[L]; ++j) mag[L][j] = fabs(mag[L][j]);
            }
            backward_one_abs(&n, Wflat, act, mag, gW + (size_t)t * n.nw, gb + (size_t)t * n.nb);
        }
        free_layers(&n, act);
        free_layers(&n, mag);
    }
    for (int64_t i = 0; i < n.nw; ++i) { double s = 0.0; for (int t = 0; t < nthreads; ++t) s += gW[(size_t)t * n.nw + i]; aW[i] = s; }
    for (int64_t i = 0; i < n.nb; ++i) { double s = 0.0; for (int t = 0; t < nthreads; ++t) s += gb[(size_t)t * n.nb + i]; ab[i] = s; }
    free(gW); free(gb);
    return 0;
}

/* Section 4.2's plain step W := W - alpha * grad: in double, rounded once to fp32. */
void oracle_sgd_step(int64_t n, const float* w, const float* g, double lr, float* w_out) {
    for (int64_t i = 0; i < n; ++i) w_out[i] = (float)((double)w[i] - lr * (double)g[i]);
}
