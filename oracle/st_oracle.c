/*
 * CPU oracle for structured tensor contractions -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64 loop nests over the FULL dense iteration space (no use of
 * symmetry, sparsity or packed layouts in the arithmetic).  The method of the
 * paper is lossless (Section 6, Eq. "R_T o P_T (T) = T" and the soundness
 * corollary): structured execution must reach exactly the dense result, so the
 * oracle is the dense definition written out.
 *
 * This file shares nothing with the CUDA library: no header, no index
 * formula, no table.  The packed layouts are reproduced here only by walking
 * the unique set T_U in lexicographic order with a running counter (Section 4,
 * "Compressed Tensor": T_C = T * T_U; Section 5.5: loop nests over the ranges
 * given by T_U), never by a closed form.
 *
 * Only tests, the smoke check and the CPU-baseline leg of the benchmark may
 * call into this file.
 *
 * Every float input is widened exactly to double before use; each function
 * also returns S = sum of |terms|, the normaliser of the error metric.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <math.h>
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

void oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ---------------------------------------------------------------------------
 * Second moment (Section 3, Sigma(x) = x (x) x, summed over the samples:
 * "creation and addition" of covariance matrices, Section 7.2).
 * T[i,j] = sum_n X[n,i] X[n,j] for ALL (i,j) in [0,d)^2.
 * ------------------------------------------------------------------------- */
void oracle_moment2(const float *X, int64_t N, int64_t d, int64_t ldx,
                    double *T, double *S)
{
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < d; ++i) {
        for (int64_t j = 0; j < d; ++j) {
            double t = 0.0, s = 0.0;
            for (int64_t n = 0; n < N; ++n) {
                double term = (double)X[n * ldx + i] * (double)X[n * ldx + j];
                t += term;
                s += fabs(term);
            }
            T[i * d + j] = t;
            S[i * d + j] = s;
        }
    }
}

/* Same definition, for a list of sampled (i,j) entries only (used where the
 * full d x d x N nest would take too long).  Every entry is still the full
 * sum over n, taken in increasing n. */
void oracle_moment2_at(const float *X, int64_t N, int64_t d, int64_t ldx,
                       const int64_t *ii, const int64_t *jj, int64_t m,
                       double *T, double *S)
{
    (void)d;
    #pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < m; ++e) {
        double t = 0.0, s = 0.0;
        const int64_t i = ii[e], j = jj[e];
        for (int64_t n = 0; n < N; ++n) {
            double term = (double)X[n * ldx + i] * (double)X[n * ldx + j];
            t += term;
            s += fabs(term);
        }
        T[e] = t;
        S[e] = s;
    }
}

/* ---------------------------------------------------------------------------
 * Third moment (Section 3, term M2 = f (x) vec(f (x) f), summed over samples).
 * T[i,j,k] = sum_n X[n,i] X[n,j] X[n,k] for ALL (i,j,k) in [0,d)^3.
 * ------------------------------------------------------------------------- */
void oracle_moment3(const float *X, int64_t N, int64_t d, int64_t ldx,
                    double *T, double *S)
{
    #pragma omp parallel for collapse(2) schedule(static)
    for (int64_t i = 0; i < d; ++i) {
        for (int64_t j = 0; j < d; ++j) {
            for (int64_t k = 0; k < d; ++k) {
                double t = 0.0, s = 0.0;
                for (int64_t n = 0; n < N; ++n) {
                    const float *x = X + n * ldx;
                    double term = (double)x[i] * (double)x[j] * (double)x[k];
                    t += term;
                    s += fabs(term);
                }
                T[(i * d + j) * d + k] = t;
                S[(i * d + j) * d + k] = s;
            }
        }
    }
}

/* Same definition, for a list of sampled (i,j,k) entries only. */
void oracle_moment3_at(const float *X, int64_t N, int64_t d, int64_t ldx,
                       const int64_t *ii, const int64_t *jj, const int64_t *kk, int64_t m,
                       double *T, double *S)
{
    (void)d;
    #pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < m; ++e) {
        double t = 0.0, s = 0.0;
        const int64_t i = ii[e], j = jj[e], k = kk[e];
        for (int64_t n = 0; n < N; ++n) {
            const float *x = X + n * ldx;
            double term = (double)x[i] * (double)x[j] * (double)x[k];
            t += term;
            s += fabs(term);
        }
        T[e] = t;
        S[e] = s;
    }
}

/* Fourth moment (Section 3, term M3 = vec(f (x) f) (x) vec(f (x) f)). */
void oracle_moment4(const float *X, int64_t N, int64_t d, int64_t ldx,
                    double *T, double *S)
{
    #pragma omp parallel for collapse(2) schedule(static)
    for (int64_t i = 0; i < d; ++i) {
        for (int64_t j = 0; j < d; ++j) {
            for (int64_t k = 0; k < d; ++k) {
                for (int64_t l = 0; l < d; ++l) {
                    double t = 0.0, s = 0.0;
                    for (int64_t n = 0; n < N; ++n) {
                        const float *x = X + n * ldx;
                        double term = (double)x[i] * (double)x[j] *
                                      (double)x[k] * (double)x[l];
                        t += term;
                        s += fabs(term);
                    }
                    T[((i * d + j) * d + k) * d + l] = t;
                    S[((i * d + j) * d + k) * d + l] = s;
                }
            }
        }
    }
}

/* Same definition, for a list of sampled (i,j,k,l) entries only. */
void oracle_moment4_at(const float *X, int64_t N, int64_t d, int64_t ldx,
                       const int64_t *ii, const int64_t *jj, const int64_t *kk, const int64_t *ll,
                       int64_t m, double *T, double *S)
{
    (void)d;
    #pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < m; ++e) {
        double t = 0.0, s = 0.0;
        const int64_t i = ii[e], j = jj[e], k = kk[e], l = ll[e];
        for (int64_t n = 0; n < N; ++n) {
            const float *x = X + n * ldx;
            double term = (double)x[i] * (double)x[j] * (double)x[k] * (double)x[l];
            t += term;
            s += fabs(term);
        }
        T[e] = t;
        S[e] = s;
    }
}

/* ---------------------------------------------------------------------------
 * MTTKRP (Table 1): A(i,r) = sum_j sum_k B(i,j,k) C(j,r) D(k,r) over the FULL
 * J x K range of a dense B (zeros wherever the structure says so).  Rows
 * i in [i0, i1) only, so that sampled rows can be checked at full size.
 * A and S are [i1-i0, R].
 * ------------------------------------------------------------------------- */
void oracle_mttkrp(const float *B, int64_t I, int64_t J, int64_t K,
                   const float *C, const float *D, int64_t R,
                   int64_t i0, int64_t i1, double *A, double *S)
{
    (void)I;
    #pragma omp parallel for collapse(2) schedule(static)
    for (int64_t i = i0; i < i1; ++i) {
        for (int64_t r = 0; r < R; ++r) {
            double t = 0.0, s = 0.0;
            for (int64_t j = 0; j < J; ++j) {
                for (int64_t k = 0; k < K; ++k) {
                    double term = (double)B[(i * J + j) * K + k] *
                                  (double)C[j * R + r] * (double)D[k * R + r];
                    t += term;
                    s += fabs(term);
                }
            }
            A[(i - i0) * R + r] = t;
            S[(i - i0) * R + r] = s;
        }
    }
}

/* ---------------------------------------------------------------------------
 * TTM (Table 1): A(i,j,r) = sum_k B(i,j,k) U(k,r).  B is given as `rows`
 * mode-3 fibres [rows, K] (rows = I*J for a whole dense tensor, or any list
 * of sampled fibres).  A and S are [rows, R].
 * ------------------------------------------------------------------------- */
void oracle_ttm(const float *B, int64_t rows, int64_t K,
                const float *U, int64_t R, double *A, double *S)
{
    #pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < rows; ++m) {
        for (int64_t r = 0; r < R; ++r) {
            double t = 0.0, s = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double term = (double)B[m * K + k] * (double)U[k * R + r];
                t += term;
                s += fabs(term);
            }
            A[m * R + r] = t;
            S[m * R + r] = s;
        }
    }
}

/* ---------------------------------------------------------------------------
 * Pack / unpack by walking the unique set with a running counter.
 *
 * kind: 0 upper-triangular matrix      T_U(i,j)   = 0<=i<=j<d     (Section 4)
 *       1 tetrahedral order-3 tensor   T_U(i,j,k) = 0<=i<=j<=k<d  (Section 2)
 *       2 band matrix                  T_U(i,j)   = i-kl<=j<=i+ku
 *       3 block-diagonal matrix = direct sum of nb blocks of bs x bs
 *                                      (Figure "operations in STUR", e1 (+) e2)
 *       4 one row of a matrix          T_U(i,j) = (i = r)          (R_r of Figure "matrix structures";
 *       5 one column of a matrix       T_U(i,j) = (j = c)           C_c of the same figure; Table 1's
 *                                      "fixed i" / "fixed j" structures on the first two modes; the
 *                                      fixed index is passed in kl)
 *       6 order-4 tensor               T_U(i,j,k,l) = 0<=i<=j<=k<=l<d  (Section 3, the unique 4-tuples
 *                                      of M3; dense counterpart d x d x d x d)
 * Each position carries `inner` contiguous elements of `es` bytes (a trailing
 * dense mode).  fill: 0 = zeros outside T_U, 1 = redundancy map of the
 * symmetric structure (Figure "structures in STUR": T_R(i,j,i',j') =
 * (0<=j<i<n)*(i'=j)*(j'=i); order 3: the representative of (i,j,k) is its
 * sorted index triple).
 *
 * The band layout has fixed width kl+ku+1 per row; slots that fall outside
 * the matrix are written as zero bytes by pack and skipped by unpack.
 * Returns the number of packed positions, or -1 for an unsupported request.
 * ------------------------------------------------------------------------- */
static void sort3(int64_t *a, int64_t *b, int64_t *c)
{
    int64_t t;
    if (*a > *b) { t = *a; *a = *b; *b = t; }
    if (*b > *c) { t = *b; *b = *c; *c = t; }
    if (*a > *b) { t = *a; *a = *b; *b = t; }
}

/* Kinds 4, 5, 6 are written as a walk over the WHOLE dense index space in
 * lexicographic order with a membership test of T_U (no loop bounds derived
 * from the structure). */
static int in_unique_set(int kind, int64_t fixed, int64_t i, int64_t j, int64_t k, int64_t l)
{
    if (kind == 4) return i == fixed;
    if (kind == 5) return j == fixed;
    return i <= j && j <= k && k <= l;
}

int64_t oracle_pack(int kind, int64_t d, int64_t inner, int64_t kl, int64_t ku,
                    int64_t nb, int64_t bs, int64_t es,
                    const unsigned char *dense, unsigned char *packed)
{
    const size_t w = (size_t)(inner * es);
    int64_t p = 0;
    if (kind == 0) {
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = i; j < d; ++j) {
                if (packed) memcpy(packed + (size_t)p * w, dense + (size_t)(i * d + j) * w, w);
                ++p;
            }
    } else if (kind == 1) {
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = i; j < d; ++j)
                for (int64_t k = j; k < d; ++k) {
                    if (packed) memcpy(packed + (size_t)p * w,
                                       dense + (size_t)((i * d + j) * d + k) * w, w);
                    ++p;
                }
    } else if (kind == 2) {
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = i - kl; j <= i + ku; ++j) {
                if (packed) {
                    if (j >= 0 && j < d)
                        memcpy(packed + (size_t)p * w, dense + (size_t)(i * d + j) * w, w);
                    else
                        memset(packed + (size_t)p * w, 0, w);
                }
                ++p;
            }
    } else if (kind == 3) {
        if (d != nb * bs) return -1;
        for (int64_t b = 0; b < nb; ++b)
            for (int64_t i = b * bs; i < (b + 1) * bs; ++i)
                for (int64_t j = b * bs; j < (b + 1) * bs; ++j) {
                    if (packed) memcpy(packed + (size_t)p * w, dense + (size_t)(i * d + j) * w, w);
                    ++p;
                }
    } else if (kind == 4 || kind == 5) {
        if (kl < 0 || kl >= d) return -1;
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = 0; j < d; ++j)
                if (in_unique_set(kind, kl, i, j, 0, 0)) {
                    if (packed) memcpy(packed + (size_t)p * w, dense + (size_t)(i * d + j) * w, w);
                    ++p;
                }
    } else if (kind == 6) {
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = 0; j < d; ++j)
                for (int64_t k = 0; k < d; ++k)
                    for (int64_t l = 0; l < d; ++l)
                        if (in_unique_set(kind, 0, i, j, k, l)) {
                            if (packed) memcpy(packed + (size_t)p * w,
                                               dense + (size_t)(((i * d + j) * d + k) * d + l) * w, w);
                            ++p;
                        }
    } else {
        return -1;
    }
    return p;
}

int64_t oracle_unpack(int kind, int64_t d, int64_t inner, int64_t kl, int64_t ku,
                      int64_t nb, int64_t bs, int64_t es, int fill,
                      const unsigned char *packed, unsigned char *dense)
{
    const size_t w = (size_t)(inner * es);
    int64_t p = 0;
    if (fill != 0 && fill != 1) return -1;
    if (fill == 1 && kind != 0 && kind != 1 && kind != 6) return -1;
    if (kind == 0) {
        memset(dense, 0, (size_t)(d * d) * w);
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = i; j < d; ++j) {
                memcpy(dense + (size_t)(i * d + j) * w, packed + (size_t)p * w, w);
                ++p;
            }
        if (fill == 1)   /* T = T_C + T_R * T_C  (Section 6, Property 5) */
            for (int64_t i = 0; i < d; ++i)
                for (int64_t j = 0; j < i; ++j)
                    memcpy(dense + (size_t)(i * d + j) * w, dense + (size_t)(j * d + i) * w, w);
    } else if (kind == 1) {
        memset(dense, 0, (size_t)(d * d * d) * w);
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = i; j < d; ++j)
                for (int64_t k = j; k < d; ++k) {
                    memcpy(dense + (size_t)((i * d + j) * d + k) * w, packed + (size_t)p * w, w);
                    ++p;
                }
        if (fill == 1)
            for (int64_t i = 0; i < d; ++i)
                for (int64_t j = 0; j < d; ++j)
                    for (int64_t k = 0; k < d; ++k) {
                        int64_t a = i, b = j, c = k;
                        sort3(&a, &b, &c);
                        if (a == i && b == j && c == k) continue;
                        memcpy(dense + (size_t)((i * d + j) * d + k) * w,
                               dense + (size_t)((a * d + b) * d + c) * w, w);
                    }
    } else if (kind == 2) {
        memset(dense, 0, (size_t)(d * d) * w);
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = i - kl; j <= i + ku; ++j) {
                if (j >= 0 && j < d)
                    memcpy(dense + (size_t)(i * d + j) * w, packed + (size_t)p * w, w);
                ++p;
            }
    } else if (kind == 3) {
        if (d != nb * bs) return -1;
        memset(dense, 0, (size_t)(d * d) * w);
        for (int64_t b = 0; b < nb; ++b)
            for (int64_t i = b * bs; i < (b + 1) * bs; ++i)
                for (int64_t j = b * bs; j < (b + 1) * bs; ++j) {
                    memcpy(dense + (size_t)(i * d + j) * w, packed + (size_t)p * w, w);
                    ++p;
                }
    } else if (kind == 4 || kind == 5) {
        if (kl < 0 || kl >= d) return -1;
        memset(dense, 0, (size_t)(d * d) * w);
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = 0; j < d; ++j)
                if (in_unique_set(kind, kl, i, j, 0, 0)) {
                    memcpy(dense + (size_t)(i * d + j) * w, packed + (size_t)p * w, w);
                    ++p;
                }
    } else if (kind == 6) {
        memset(dense, 0, (size_t)(d * d * d * d) * w);
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = 0; j < d; ++j)
                for (int64_t k = 0; k < d; ++k)
                    for (int64_t l = 0; l < d; ++l)
                        if (in_unique_set(kind, 0, i, j, k, l)) {
                            memcpy(dense + (size_t)(((i * d + j) * d + k) * d + l) * w, packed + (size_t)p * w, w);
                            ++p;
                        }
        if (fill == 1)   /* the representative of (i,j,k,l) is its sorted index tuple */
            for (int64_t i = 0; i < d; ++i)
                for (int64_t j = 0; j < d; ++j)
                    for (int64_t k = 0; k < d; ++k)
                        for (int64_t l = 0; l < d; ++l) {
                            int64_t v[4] = {i, j, k, l};
                            for (int a = 1; a < 4; ++a)          /* insertion sort */
                                for (int b = a; b > 0 && v[b - 1] > v[b]; --b) {
                                    int64_t t = v[b]; v[b] = v[b - 1]; v[b - 1] = t;
                                }
                            if (v[0] == i && v[1] == j && v[2] == k && v[3] == l) continue;
                            memcpy(dense + (size_t)(((i * d + j) * d + k) * d + l) * w,
                                   dense + (size_t)(((v[0] * d + v[1]) * d + v[2]) * d + v[3]) * w, w);
                        }
    } else {
        return -1;
    }
    return p;
}

/* Position of one index tuple in the packed order, found by walking the unique
 * set from the start (slow on purpose).  c (and e) are ignored for matrix kinds.
 * Returns -1 when the tuple is not in T_U. */
int64_t oracle_locate(int kind, int64_t d, int64_t kl, int64_t ku,
                      int64_t nb, int64_t bs, int64_t a, int64_t b, int64_t c, int64_t e)
{
    int64_t p = 0;
    if (kind == 0) {
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = i; j < d; ++j) { if (i == a && j == b) return p; ++p; }
    } else if (kind == 1) {
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = i; j < d; ++j)
                for (int64_t k = j; k < d; ++k) { if (i == a && j == b && k == c) return p; ++p; }
    } else if (kind == 2) {
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = i - kl; j <= i + ku; ++j) {
                if (i == a && j == b && j >= 0 && j < d) return p;
                ++p;
            }
    } else if (kind == 3) {
        for (int64_t q = 0; q < nb; ++q)
            for (int64_t i = q * bs; i < (q + 1) * bs; ++i)
                for (int64_t j = q * bs; j < (q + 1) * bs; ++j) { if (i == a && j == b) return p; ++p; }
    } else if (kind == 4 || kind == 5) {
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = 0; j < d; ++j)
                if (in_unique_set(kind, kl, i, j, 0, 0)) { if (i == a && j == b) return p; ++p; }
    } else if (kind == 6) {
        for (int64_t i = 0; i < d; ++i)
            for (int64_t j = 0; j < d; ++j)
                for (int64_t k = 0; k < d; ++k)
                    for (int64_t l = 0; l < d; ++l)
                        if (in_unique_set(kind, 0, i, j, k, l)) {
                            if (i == a && j == b && k == c && l == e) return p;
                            ++p;
                        }
    }
    return -1;
}
