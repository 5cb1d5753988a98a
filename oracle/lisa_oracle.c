/*
 * LiSA shared-layer attention forward -- CPU oracle (test infrastructure only).
 *
 * A plain, slow, fp64 statement of what the layer computes, written from the
 * paper's equations.  Everything is materialised; there is no tiling, no online
 * softmax and no code shared with the CUDA library.  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may call it; the product path
 * never does.
 *
 * Notation follows the paper: l (here N) positions, h (here Hq) query heads,
 * d_k (here d) head width, r low-rank width per head, A the pre-softmax score
 * matrix of a layer, A_Delta the low-rank difference, P the attention weights.
 *
 * Passages followed:
 *   Eq. 1-2  (Sec. 2.1)  P_i = Softmax(Q_i K_i^T / sqrt(d_k)), out_i = P_i V_i
 *   Sec. 5.1 "Learn to share attention weights": the aligner is an FFN over
 *            the head axis of A^T in R^{l x l x h}, applied per position (i,j)
 *   Eq. 3    A_Delta = Q_LR K_LR^T / sqrt(r)
 *   Eq. 4    A = Integrate(A_align, A_Delta): addition, or (Sec. 5.1 "An
 *            overview") concatenation [A_{n-1}; A_Delta] on the head axis
 *            before the FFN
 *   Sec. 5.2 decode stage: the previous layer's score row (h x l) is kept and
 *            K_LR replaces K in the cache
 *   Eq. 1, 3 the projections H W^V_i, H W^Q_LR, H W^K_LR and the product with W^O
 *            (oracle_project: a plain matrix product)
 *
 * Readings taken where the paper is silent (each is listed in the design
 * document as well): the aligner acts on pre-softmax scores that already carry
 * the 1/sqrt(d_k) factor; r is per head; the causal mask is applied after the
 * whole chain of shared layers, directly before Softmax; with grouped-query
 * attention query head h reads key/value head h / (Hq/Hkv); a one-layer FFN
 * has no activation.
 *
 * Parity status: every function below is pinned by tests/test_oracle_pins.py
 * against closed forms, library routines on special cases, and an independent
 * brute-force script.  Agreement with the authors' own code or trained
 * checkpoints is "parity unpinned" (neither is available).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_ACT_NONE = 0, ORACLE_ACT_RELU = 1, ORACLE_ACT_SILU = 2 };
enum { ORACLE_INTEGRATE_ADD = 0, ORACLE_INTEGRATE_CONCAT = 1, ORACLE_INTEGRATE_PLUS = 2 };

/* One shared layer of a chain: its low-rank Q'/K' and its aligner FFN.
 * qp [B,N,Hq,r], kp [B,N,Hkv,r]; w1 [h_in,m] with h_in = Hq (ADD) or 2*Hq
 * (CONCAT, rows 0..Hq-1 multiply A_{n-1}, rows Hq..2Hq-1 multiply A_Delta);
 * b1 [m] or NULL; w2 [m,Hq] and b2 [Hq] (NULL allowed) for a two-layer FFN;
 * ffn_layers == 1 means y = W1^T x + b1 with m == Hq and no activation. */
typedef struct {
    const double* qp;
    const double* kp;
    const double* w1;
    const double* b1;
    const double* w2;
    const double* b2;
    int32_t r;
    int32_t m;
    int32_t act;
    int32_t integrate;
    int32_t ffn_layers;
} oracle_link;

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static double act_apply(double x, int act) {
    if (act == ORACLE_ACT_RELU) return x > 0.0 ? x : 0.0;
    if (act == ORACLE_ACT_SILU) return x / (1.0 + exp(-x));
    return x;
}

/* Sec. 5.1: one position (i,j).  a = A_{n-1}[:,i,j], delta = A_Delta[:,i,j],
 * both of length h; writes A_n[:,i,j] to out.  hid is scratch of length m. */
static void align_integrate(const double* a, const double* delta, int h, const oracle_link* lk,
                            double* hid, double* out) {
    if (lk->integrate == ORACLE_INTEGRATE_PLUS) {
        for (int g = 0; g < h; ++g) out[g] = a[g] + delta[g];
        return;
    }
    const int m = lk->m;
    for (int u = 0; u < m; ++u) {
        double s = lk->b1 ? lk->b1[u] : 0.0;
        for (int x = 0; x < h; ++x) s += a[x] * lk->w1[(size_t)x * m + u];
        if (lk->integrate == ORACLE_INTEGRATE_CONCAT)
            for (int x = 0; x < h; ++x) s += delta[x] * lk->w1[(size_t)(h + x) * m + u];
        hid[u] = s;
    }
    if (lk->ffn_layers == 1) {
        for (int g = 0; g < h; ++g) out[g] = hid[g];
    } else {
        for (int u = 0; u < m; ++u) hid[u] = act_apply(hid[u], lk->act);
        for (int g = 0; g < h; ++g) {
            double s = lk->b2 ? lk->b2[g] : 0.0;
            for (int u = 0; u < m; ++u) s += hid[u] * lk->w2[(size_t)u * h + g];
            out[g] = s;
        }
    }
    if (lk->integrate == ORACLE_INTEGRATE_ADD)
        for (int g = 0; g < h; ++g) out[g] += delta[g];
}

/* Eq. 2, the bracket labelled A: A[b,h,i,j] = Q[b,i,h,:].K[b,j,g(h),:]/sqrt(d)
 * for ALL i,j (no mask).  Q [B,N,Hq,d], K [B,N,Hkv,d], A [B,Hq,N,N]. */
void oracle_scores(const double* Q, const double* K, int B, int N, int Hq, int Hkv, int d, double* A) {
    const int G = Hq / Hkv;
    const double scale = 1.0 / sqrt((double)d);
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < N; ++i)
            for (int h = 0; h < Hq; ++h)
                for (int j = 0; j < N; ++j) {
                    const double* q = Q + (((size_t)b * N + i) * Hq + h) * d;
                    const double* k = K + (((size_t)b * N + j) * Hkv + h / G) * d;
                    double s = 0.0;
                    for (int x = 0; x < d; ++x) s += q[x] * k[x];
                    A[(((size_t)b * Hq + h) * N + i) * N + j] = s * scale;
                }
}

/* One shared layer on materialised scores: A_out = Integrate(Align(A_in), A_Delta)
 * (Eq. 3-4), for all positions.  A_in, A_out [B,Hq,N,N]; may not alias. */
void oracle_link_apply(const double* A_in, const oracle_link* lk, int B, int N, int Hq, int Hkv, double* A_out) {
    const size_t plane = (size_t)N * N;
    double* D = (double*)malloc(sizeof(double) * (size_t)B * Hq * plane);
    oracle_scores(lk->qp, lk->kp, B, N, Hq, Hkv, lk->r, D); /* Eq. 3 with width r */
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < N; ++i) {
            double* a = (double*)malloc(sizeof(double) * (3 * (size_t)Hq + (size_t)lk->m + 1));
            double* dl = a + Hq;
            double* out = dl + Hq;
            double* hid = out + Hq;
            for (int j = 0; j < N; ++j) {
                for (int h = 0; h < Hq; ++h) {
                    const size_t at = ((size_t)b * Hq + h) * plane + (size_t)i * N + j;
                    a[h] = A_in[at];
                    dl[h] = D[at];
                }
                align_integrate(a, dl, Hq, lk, hid, out);
                for (int h = 0; h < Hq; ++h) A_out[((size_t)b * Hq + h) * plane + (size_t)i * N + j] = out[h];
            }
            free(a);
        }
    free(D);
}

/* Causal Softmax over j <= i (Eq. 2); entries j > i are exactly 0.  [B,Hq,N,N]. */
void oracle_causal_softmax(const double* A, int B, int N, int Hq, double* P) {
#pragma omp parallel for schedule(static)
    for (long row = 0; row < (long)B * Hq * N; ++row) {
        const int i = (int)(row % N);
        const double* a = A + (size_t)row * N;
        double* p = P + (size_t)row * N;
        double mx = a[0];
        for (int j = 1; j <= i; ++j) mx = a[j] > mx ? a[j] : mx;
        double sum = 0.0;
        for (int j = 0; j <= i; ++j) {
            p[j] = exp(a[j] - mx);
            sum += p[j];
        }
        for (int j = 0; j <= i; ++j) p[j] /= sum;
        for (int j = i + 1; j < N; ++j) p[j] = 0.0;
    }
}

/* Eq. 1, one head: O[b,i,h,:] = sum_j P[b,h,i,j] V[b,j,g(h),:].  V [B,N,Hkv,d], O [B,N,Hq,d]. */
void oracle_pv(const double* P, const double* V, int B, int N, int Hq, int Hkv, int d, double* O) {
    const int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < N; ++i)
            for (int h = 0; h < Hq; ++h) {
                double* o = O + (((size_t)b * N + i) * Hq + h) * d;
                for (int x = 0; x < d; ++x) o[x] = 0.0;
                const double* p = P + (((size_t)b * Hq + h) * N + i) * N;
                for (int j = 0; j < N; ++j) {
                    const double* v = V + (((size_t)b * N + j) * Hkv + h / G) * d;
                    for (int x = 0; x < d; ++x) o[x] += p[j] * v[x];
                }
            }
}

/* The whole layer, everything materialised, in the paper's order: anchor
 * scores A_0, then for k = 1..c the link's A_Delta and aligner, then mask,
 * Softmax and the product with this layer's V.  c == 0 is standard attention.
 * A_out and P_out ([B,Hq,N,N]) are optional (NULL to skip). */
int oracle_prefill_full(const double* Q0, const double* K0, const double* V, const oracle_link* links, int c,
                        int B, int N, int Hq, int Hkv, int d, double* O, double* A_out, double* P_out) {
    const size_t total = (size_t)B * Hq * N * N;
    double* A = (double*)malloc(sizeof(double) * total);
    double* T = (double*)malloc(sizeof(double) * total);
    if (!A || !T) { free(A); free(T); return 1; }
    oracle_scores(Q0, K0, B, N, Hq, Hkv, d, A);
    for (int k = 0; k < c; ++k) {
        oracle_link_apply(A, &links[k], B, N, Hq, Hkv, T);
        double* sw = A; A = T; T = sw;
    }
    if (A_out) memcpy(A_out, A, sizeof(double) * total);
    oracle_causal_softmax(A, B, N, Hq, T);
    if (P_out) memcpy(P_out, T, sizeof(double) * total);
    oracle_pv(T, V, B, N, Hq, Hkv, d, O);
    free(A);
    free(T);
    return 0;
}

/* Row-sampled form of the same definition: query row i depends only on keys
 * j <= i, so the layer can be evaluated for a list of (b,i) pairs alone.
 * rows_b/rows_i [n_rows]; O [n_rows,Hq,d]; A_out (optional) [n_rows,Hq,N] holds
 * the final scores for j <= i and 0 beyond. */
int oracle_prefill_rows(const double* Q0, const double* K0, const double* V, const oracle_link* links, int c,
                        int B, int N, int Hq, int Hkv, int d, const int32_t* rows_b, const int32_t* rows_i,
                        int n_rows, double* O, double* A_out) {
    const int G = Hq / Hkv;
    int mmax = 1;
    for (int k = 0; k < c; ++k) mmax = links[k].m > mmax ? links[k].m : mmax;
    (void)B;
#pragma omp parallel for schedule(dynamic, 1)
    for (int t = 0; t < n_rows; ++t) {
        const int b = rows_b[t], i = rows_i[t];
        const int n = i + 1;
        double* A = (double*)malloc(sizeof(double) * (size_t)Hq * n * 2);
        double* p = A + (size_t)Hq * n;
        double* tmp = (double*)malloc(sizeof(double) * (4 * (size_t)Hq + mmax));
        double *a = tmp, *dl = tmp + Hq, *out = tmp + 2 * Hq, *hid = tmp + 3 * Hq;
        for (int h = 0; h < Hq; ++h)
            for (int j = 0; j < n; ++j) {
                const double* q = Q0 + (((size_t)b * N + i) * Hq + h) * d;
                const double* kk = K0 + (((size_t)b * N + j) * Hkv + h / G) * d;
                double s = 0.0;
                for (int x = 0; x < d; ++x) s += q[x] * kk[x];
                A[(size_t)h * n + j] = s * (1.0 / sqrt((double)d));
            }
        for (int k = 0; k < c; ++k) {
            const oracle_link* lk = &links[k];
            const int r = lk->r;
            for (int j = 0; j < n; ++j) {
                for (int h = 0; h < Hq; ++h) {
                    const double* q = lk->qp + (((size_t)b * N + i) * Hq + h) * r;
                    const double* kk = lk->kp + (((size_t)b * N + j) * Hkv + h / G) * r;
                    double s = 0.0;
                    for (int x = 0; x < r; ++x) s += q[x] * kk[x];
                    dl[h] = s * (1.0 / sqrt((double)r));
                    a[h] = A[(size_t)h * n + j];
                }
                align_integrate(a, dl, Hq, lk, hid, out);
                for (int h = 0; h < Hq; ++h) A[(size_t)h * n + j] = out[h];
            }
        }
        for (int h = 0; h < Hq; ++h) {
            const double* ar = A + (size_t)h * n;
            double* pr = p + (size_t)h * n;
            double mx = ar[0];
            for (int j = 1; j < n; ++j) mx = ar[j] > mx ? ar[j] : mx;
            double sum = 0.0;
            for (int j = 0; j < n; ++j) { pr[j] = exp(ar[j] - mx); sum += pr[j]; }
            for (int j = 0; j < n; ++j) pr[j] /= sum;
            double* o = O + ((size_t)t * Hq + h) * d;
            for (int x = 0; x < d; ++x) o[x] = 0.0;
            for (int j = 0; j < n; ++j) {
                const double* v = V + (((size_t)b * N + j) * Hkv + h / G) * d;
                for (int x = 0; x < d; ++x) o[x] += pr[j] * v[x];
            }
            if (A_out) {
                double* ao = A_out + ((size_t)t * Hq + h) * N;
                for (int j = 0; j < N; ++j) ao[j] = j < n ? ar[j] : 0.0;
            }
        }
        free(tmp);
        free(A);
    }
    return 0;
}

/* Decode step of a shared layer (Sec. 5.2, decoding stage): the single query
 * row at the end of a context of lens[b] cached positions.  The previous
 * layer's score row is GIVEN (prev [B,Hq,Lmax]); kp [B,Lmax,Hkv,r] and
 * v [B,Lmax,Hkv,d] are the cached K_LR and V in position-major order;
 * qp [B,Hq,r] is the new token's Q_LR.  Only lk->w1..ffn_layers, r, m are read
 * from the link (its qp/kp fields are ignored).  Returns O [B,Hq,d] and the
 * layer's own score row row_out [B,Hq,Lmax] (entries beyond lens[b] are 0). */
int oracle_decode_shared(const double* prev, const double* qp, const double* kp, const double* v,
                         const oracle_link* lk, const int32_t* lens, int B, int Lmax, int Hq, int Hkv, int d,
                         double* O, double* row_out) {
    const int G = Hq / Hkv;
    const int r = lk->r;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const int L = lens[b];
        double* A = (double*)malloc(sizeof(double) * (size_t)Hq * L * 2);
        double* p = A + (size_t)Hq * L;
        double* tmp = (double*)malloc(sizeof(double) * (4 * (size_t)Hq + lk->m + 1));
        double *a = tmp, *dl = tmp + Hq, *out = tmp + 2 * Hq, *hid = tmp + 3 * Hq;
        for (int j = 0; j < L; ++j) {
            for (int h = 0; h < Hq; ++h) {
                const double* q = qp + ((size_t)b * Hq + h) * r;
                const double* kk = kp + (((size_t)b * Lmax + j) * Hkv + h / G) * r;
                double s = 0.0;
                for (int x = 0; x < r; ++x) s += q[x] * kk[x];
                dl[h] = s * (1.0 / sqrt((double)r));
                a[h] = prev[((size_t)b * Hq + h) * Lmax + j];
            }
            align_integrate(a, dl, Hq, lk, hid, out);
            for (int h = 0; h < Hq; ++h) A[(size_t)h * L + j] = out[h];
        }
        for (int h = 0; h < Hq; ++h) {
            const double* ar = A + (size_t)h * L;
            double* pr = p + (size_t)h * L;
            double mx = ar[0];
            for (int j = 1; j < L; ++j) mx = ar[j] > mx ? ar[j] : mx;
            double sum = 0.0;
            for (int j = 0; j < L; ++j) { pr[j] = exp(ar[j] - mx); sum += pr[j]; }
            for (int j = 0; j < L; ++j) pr[j] /= sum;
            double* o = O + ((size_t)b * Hq + h) * d;
            for (int x = 0; x < d; ++x) o[x] = 0.0;
            for (int j = 0; j < L; ++j) {
                const double* vv = v + (((size_t)b * Lmax + j) * Hkv + h / G) * d;
                for (int x = 0; x < d; ++x) o[x] += pr[j] * vv[x];
            }
            if (row_out) {
                double* ro = row_out + ((size_t)b * Hq + h) * Lmax;
                for (int j = 0; j < Lmax; ++j) ro[j] = j < L ? ar[j] : 0.0;
            }
        }
        free(tmp);
        free(A);
    }
    return 0;
}

/* Decode step of a standard layer (Eq. 1-2 for the last row of the context):
 * q [B,Hq,d], k and v [B,Lmax,Hkv,d].  Returns O [B,Hq,d] and the pre-softmax
 * score row row_out [B,Hq,Lmax] that a following shared layer consumes. */
int oracle_decode_anchor(const double* q, const double* k, const double* v, const int32_t* lens, int B, int Lmax,
                         int Hq, int Hkv, int d, double* O, double* row_out) {
    const int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const int L = lens[b];
        double* ar = (double*)malloc(sizeof(double) * (size_t)L * 2);
        double* pr = ar + L;
        for (int h = 0; h < Hq; ++h) {
            const double* qq = q + ((size_t)b * Hq + h) * d;
            for (int j = 0; j < L; ++j) {
                const double* kk = k + (((size_t)b * Lmax + j) * Hkv + h / G) * d;
                double s = 0.0;
                for (int x = 0; x < d; ++x) s += qq[x] * kk[x];
                ar[j] = s * (1.0 / sqrt((double)d));
            }
            double mx = ar[0];
            for (int j = 1; j < L; ++j) mx = ar[j] > mx ? ar[j] : mx;
            double sum = 0.0;
            for (int j = 0; j < L; ++j) { pr[j] = exp(ar[j] - mx); sum += pr[j]; }
            for (int j = 0; j < L; ++j) pr[j] /= sum;
            double* o = O + ((size_t)b * Hq + h) * d;
            for (int x = 0; x < d; ++x) o[x] = 0.0;
            for (int j = 0; j < L; ++j) {
                const double* vv = v + (((size_t)b * Lmax + j) * Hkv + h / G) * d;
                for (int x = 0; x < d; ++x) o[x] += pr[j] * vv[x];
            }
            if (row_out) {
                double* ro = row_out + ((size_t)b * Hq + h) * Lmax;
                for (int j = 0; j < Lmax; ++j) ro[j] = j < L ? ar[j] : 0.0;
            }
        }
        free(ar);
    }
    return 0;
}

/* Sec. 5.2 memory model, in bytes, for n_shared layers using LiSA at sequence
 * length l with h heads (2-byte elements as in the paper):
 *   K-cache bytes saved          n_shared * h * l * (d_k - r) * 2
 *   prefill score matrix         h * l * l * 2
 *   decode score row             h * l * 2
 * out[0] = net saving in prefill, out[1] = net saving in decode. */
void oracle_memory_saving(long n_shared, long h, long l, long d_k, long r, long* out) {
    const long k_saved = n_shared * h * l * (d_k - r) * 2;
    out[0] = k_saved - h * l * l * 2;
    out[1] = k_saved - h * l * 2;
}

/* Projection either side of the attention: C[row, col] = sum_k X[row, k] * W[k, col], X [rows, d_in], W [d_in, n_out]
 * row-major (row = input unit, as the paper writes H W).  Eq. 1: the per-head H W^V_i are column blocks of one such
 * product and W^O multiplies the concatenated heads; Eq. 3: H W^Q_LR and H W^K_LR.  Plain triple loop, fp64. */
void oracle_project(const double* X, const double* W, long rows, long d_in, long n_out, double* C) {
#pragma omp parallel for schedule(static)
    for (long i = 0; i < rows; ++i)
        for (long j = 0; j < n_out; ++j) {
            double acc = 0.0;
            for (long k = 0; k < d_in; ++k) acc += X[i * d_in + k] * W[k * n_out + j];
            C[i * n_out + j] = acc;
        }
}
