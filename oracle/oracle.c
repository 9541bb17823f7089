/*
 * CPU oracle for the sparse contraction chains.  TEST INFRASTRUCTURE ONLY: it is used by
 * the tests, by the smoke check and by the benchmark's CPU-baseline leg; the product path
 * never calls it and shares no code with it.
 *
 * Every function evaluates the chain's plain, unfused Einsum definition (the
 * "Description" column of the paper's Table of kernels, Section 6) as one perfectly
 * nested loop over the stored nonzeros of B in COORDINATE (COO) form, in the order they
 * are given, with fp64 products and fp64 accumulation.  The paper's argument that every
 * linear loop order and every branched (fissioned/fused) nest computes the same output
 * (Sections 4.1 and 4.3) makes this definition the reference for every schedule.
 *
 * Besides A each function can return S, the sum of the absolute values of the same terms
 * per output element; tolerances are stated relative to S.
 *
 * The only reorganisation: nonzeros are first bucketed by their output slice/row i with a
 * stable counting sort, so that disjoint output slices can be evaluated by different
 * threads.  Within one output element the terms are still added in input order, so the
 * result is bit-identical to the single serial loop.
 *
 * `sel` (optional) lists the slices/rows i to evaluate; the outputs then hold n_sel
 * slices in that order (every output slice depends only on the nonzeros with that i).
 *
 * Pins (tests/test_oracle_pins.py): dense brute-force Einsum on tiny inputs, closed forms
 * for all-ones operands, identity-factor special cases that reduce to densification / SpMM /
 * GEMM, linearity, and invariance under permutation of the COO order.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int64_t n_out;      /* number of output slices */
    int64_t *start;     /* [n_out + 1] */
    int64_t *order;     /* nonzero indices grouped by output slice, input order inside */
    int64_t *out_of_i;  /* [I] output index of slice i or -1 */
} buckets_t;

static int make_buckets(buckets_t *b, int64_t nnz, const int32_t *coords, int order_,
                        int64_t I, int64_t n_sel, const int64_t *sel)
{
    memset(b, 0, sizeof(*b));
    b->out_of_i = (int64_t *)malloc(sizeof(int64_t) * (size_t)(I > 0 ? I : 1));
    if (!b->out_of_i) return -1;
    if (sel) {
        for (int64_t i = 0; i < I; ++i) b->out_of_i[i] = -1;
        for (int64_t s = 0; s < n_sel; ++s) {
            if (sel[s] < 0 || sel[s] >= I) return -2;
            b->out_of_i[sel[s]] = s;
        }
        b->n_out = n_sel;
    } else {
        for (int64_t i = 0; i < I; ++i) b->out_of_i[i] = i;
        b->n_out = I;
    }
    b->start = (int64_t *)calloc((size_t)b->n_out + 2, sizeof(int64_t));
    b->order = (int64_t *)malloc(sizeof(int64_t) * (size_t)(nnz > 0 ? nnz : 1));
    if (!b->start || !b->order) return -1;
    for (int64_t p = 0; p < nnz; ++p) {
        int64_t i = coords[p * order_];
        if (i < 0 || i >= I) return -2;
        int64_t o = b->out_of_i[i];
        if (o >= 0) b->start[o + 2]++;
    }
    for (int64_t o = 0; o < b->n_out; ++o) b->start[o + 2] += b->start[o + 1];
    /* start[o+1] is now the fill cursor of slice o */
    for (int64_t p = 0; p < nnz; ++p) {
        int64_t o = b->out_of_i[coords[p * order_]];
        if (o >= 0) b->order[b->start[o + 1]++] = p;
    }
    return 0;
}

static void free_buckets(buckets_t *b)
{
    free(b->start); free(b->order); free(b->out_of_i);
}

static void set_threads(int threads)
{
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Kernel 6 <SpTTM,TTM>:  A(i,l,m) = sum_{j,k} B(i,j,k) * C(j,l) * D(k,m). */
int oracle_spttm_ttm3(int64_t nnz, const int32_t *coords, const float *vals,
                      int64_t I, int64_t J, int64_t K, int64_t L, int64_t M,
                      const float *C, const float *D,
                      int64_t n_sel, const int64_t *sel, double *A, double *S, int threads)
{
    buckets_t b;
    int rc = make_buckets(&b, nnz, coords, 3, I, n_sel, sel);
    if (rc) { free_buckets(&b); return rc; }
    for (int64_t p = 0; p < nnz; ++p)
        if (coords[3 * p + 1] < 0 || coords[3 * p + 1] >= J || coords[3 * p + 2] < 0 || coords[3 * p + 2] >= K) {
            free_buckets(&b); return -2;
        }
    set_threads(threads);
    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t o = 0; o < b.n_out; ++o) {
        double *Ao = A + o * L * M;
        double *So = S ? S + o * L * M : NULL;
        for (int64_t x = 0; x < L * M; ++x) Ao[x] = 0.0;
        if (So) for (int64_t x = 0; x < L * M; ++x) So[x] = 0.0;
        for (int64_t q = b.start[o]; q < b.start[o + 1]; ++q) {
            int64_t p = b.order[q];
            int64_t j = coords[3 * p + 1], k = coords[3 * p + 2];
            double v = (double)vals[p];
            for (int64_t l = 0; l < L; ++l)
                for (int64_t m = 0; m < M; ++m) {
                    double term = v * (double)C[j * L + l] * (double)D[k * M + m];
                    Ao[l * M + m] += term;
                    if (So) So[l * M + m] += fabs(term);
                }
        }
    }
    free_buckets(&b);
    return 0;
}

/* Order-4 generalisation:  A(i,l,m,n) = sum_{j,k,o} B(i,j,k,o) * C(j,l) * D(k,m) * E(o,n). */
int oracle_spttm_ttm4(int64_t nnz, const int32_t *coords, const float *vals,
                      int64_t I, int64_t J, int64_t K, int64_t O,
                      int64_t L, int64_t M, int64_t N,
                      const float *C, const float *D, const float *E,
                      int64_t n_sel, const int64_t *sel, double *A, double *S, int threads)
{
    buckets_t b;
    int rc = make_buckets(&b, nnz, coords, 4, I, n_sel, sel);
    if (rc) { free_buckets(&b); return rc; }
    for (int64_t p = 0; p < nnz; ++p)
        if (coords[4 * p + 1] < 0 || coords[4 * p + 1] >= J || coords[4 * p + 2] < 0 ||
            coords[4 * p + 2] >= K || coords[4 * p + 3] < 0 || coords[4 * p + 3] >= O) {
            free_buckets(&b); return -2;
        }
    set_threads(threads);
    const int64_t T = L * M * N;
    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t o = 0; o < b.n_out; ++o) {
        double *Ao = A + o * T;
        double *So = S ? S + o * T : NULL;
        for (int64_t x = 0; x < T; ++x) Ao[x] = 0.0;
        if (So) for (int64_t x = 0; x < T; ++x) So[x] = 0.0;
        for (int64_t q = b.start[o]; q < b.start[o + 1]; ++q) {
            int64_t p = b.order[q];
            int64_t j = coords[4 * p + 1], k = coords[4 * p + 2], oo = coords[4 * p + 3];
            double v = (double)vals[p];
            for (int64_t l = 0; l < L; ++l)
                for (int64_t m = 0; m < M; ++m)
                    for (int64_t n = 0; n < N; ++n) {
                        double term = v * (double)C[j * L + l] * (double)D[k * M + m] * (double)E[oo * N + n];
                        Ao[(l * M + m) * N + n] += term;
                        if (So) So[(l * M + m) * N + n] += fabs(term);
                    }
        }
    }
    free_buckets(&b);
    return 0;
}

/* Kernel 1 <SDDMM,SpMM>:  A(i,l) = sum_{j,k} B(i,j) * C(i,k) * D(j,k) * E(j,l).
 * P (optional, [nnz], input order) receives the sampled values
 * P(p) = B(i,j) * sum_k C(i,k) * D(j,k) of the SDDMM stage, which exist exactly on the
 * stored coordinates of B; entries of unselected rows are left untouched. */
int oracle_sddmm_spmm(int64_t nnz, const int32_t *coords, const float *vals,
                      int64_t I, int64_t J, int64_t K, int64_t L,
                      const float *C, const float *D, const float *E,
                      int64_t n_sel, const int64_t *sel, double *A, double *S, double *P, int threads)
{
    buckets_t b;
    int rc = make_buckets(&b, nnz, coords, 2, I, n_sel, sel);
    if (rc) { free_buckets(&b); return rc; }
    for (int64_t p = 0; p < nnz; ++p)
        if (coords[2 * p + 1] < 0 || coords[2 * p + 1] >= J) { free_buckets(&b); return -2; }
    set_threads(threads);
    #pragma omp parallel for schedule(dynamic, 16)
    for (int64_t o = 0; o < b.n_out; ++o) {
        double *Ao = A + o * L;
        double *So = S ? S + o * L : NULL;
        for (int64_t x = 0; x < L; ++x) Ao[x] = 0.0;
        if (So) for (int64_t x = 0; x < L; ++x) So[x] = 0.0;
        for (int64_t q = b.start[o]; q < b.start[o + 1]; ++q) {
            int64_t p = b.order[q];
            int64_t i = coords[2 * p], j = coords[2 * p + 1];
            double v = (double)vals[p];
            double samp = 0.0;
            for (int64_t k = 0; k < K; ++k)
                for (int64_t l = 0; l < L; ++l) {
                    double term = v * (double)C[i * K + k] * (double)D[j * K + k] * (double)E[j * L + l];
                    Ao[l] += term;
                    if (So) So[l] += fabs(term);
                }
            if (P) {
                for (int64_t k = 0; k < K; ++k) samp += (double)C[i * K + k] * (double)D[j * K + k];
                P[p] = v * samp;
            }
        }
    }
    free_buckets(&b);
    return 0;
}

/* Kernel 4 <SpMM,GEMM>:  A(i,m) = sum_{j,l} B(i,j) * C(j,l) * D(l,m). */
int oracle_spmm_gemm(int64_t nnz, const int32_t *coords, const float *vals,
                     int64_t I, int64_t J, int64_t L, int64_t M,
                     const float *C, const float *D,
                     int64_t n_sel, const int64_t *sel, double *A, double *S, int threads)
{
    buckets_t b;
    int rc = make_buckets(&b, nnz, coords, 2, I, n_sel, sel);
    if (rc) { free_buckets(&b); return rc; }
    for (int64_t p = 0; p < nnz; ++p)
        if (coords[2 * p + 1] < 0 || coords[2 * p + 1] >= J) { free_buckets(&b); return -2; }
    set_threads(threads);
    #pragma omp parallel for schedule(dynamic, 16)
    for (int64_t o = 0; o < b.n_out; ++o) {
        double *Ao = A + o * M;
        double *So = S ? S + o * M : NULL;
        for (int64_t x = 0; x < M; ++x) Ao[x] = 0.0;
        if (So) for (int64_t x = 0; x < M; ++x) So[x] = 0.0;
        for (int64_t q = b.start[o]; q < b.start[o + 1]; ++q) {
            int64_t p = b.order[q];
            int64_t j = coords[2 * p + 1];
            double v = (double)vals[p];
            for (int64_t l = 0; l < L; ++l)
                for (int64_t m = 0; m < M; ++m) {
                    double term = v * (double)C[j * L + l] * (double)D[l * M + m];
                    Ao[m] += term;
                    if (So) So[m] += fabs(term);
                }
        }
    }
    free_buckets(&b);
    return 0;
}

/* Kernel 3 <SpMMH,GEMM>:  A(i,m) = sum_{j,l} B(i,j) * C(j,l) * D(j,l) * E(l,m)  (Table of kernels,
 * Description column: SpMM with the Hadamard product of two dense matrices, then a GEMM; the paper's
 * letters are A_il = sum_jk B_ij C_jk D_jk E_kl). */
int oracle_spmmh_gemm(int64_t nnz, const int32_t *coords, const float *vals,
                      int64_t I, int64_t J, int64_t L, int64_t M,
                      const float *C, const float *D, const float *E,
                      int64_t n_sel, const int64_t *sel, double *A, double *S, int threads)
{
    buckets_t b;
    int rc = make_buckets(&b, nnz, coords, 2, I, n_sel, sel);
    if (rc) { free_buckets(&b); return rc; }
    for (int64_t p = 0; p < nnz; ++p)
        if (coords[2 * p + 1] < 0 || coords[2 * p + 1] >= J) { free_buckets(&b); return -2; }
    set_threads(threads);
    #pragma omp parallel for schedule(dynamic, 16)
    for (int64_t o = 0; o < b.n_out; ++o) {
        double *Ao = A + o * M;
        double *So = S ? S + o * M : NULL;
        for (int64_t x = 0; x < M; ++x) Ao[x] = 0.0;
        if (So) for (int64_t x = 0; x < M; ++x) So[x] = 0.0;
        for (int64_t q = b.start[o]; q < b.start[o + 1]; ++q) {
            int64_t p = b.order[q];
            int64_t j = coords[2 * p + 1];
            double v = (double)vals[p];
            for (int64_t l = 0; l < L; ++l)
                for (int64_t m = 0; m < M; ++m) {
                    double term = v * (double)C[j * L + l] * (double)D[j * L + l] * (double)E[l * M + m];
                    Ao[m] += term;
                    if (So) So[m] += fabs(term);
                }
        }
    }
    free_buckets(&b);
    return 0;
}

/* Kernel 8 <MTTKRP,GEMM>:  A(i,m) = sum_{j,k,r} B(i,j,k) * C(j,r) * D(k,r) * E(r,m)  (Table of kernels,
 * Description column with every index that is not an output index summed; the paper's letters are
 * A_im = sum B_ikl C_lj D_kj E_jm). */
int oracle_mttkrp_gemm(int64_t nnz, const int32_t *coords, const float *vals,
                       int64_t I, int64_t J, int64_t K, int64_t R, int64_t M,
                       const float *C, const float *D, const float *E,
                       int64_t n_sel, const int64_t *sel, double *A, double *S, int threads)
{
    buckets_t b;
    int rc = make_buckets(&b, nnz, coords, 3, I, n_sel, sel);
    if (rc) { free_buckets(&b); return rc; }
    for (int64_t p = 0; p < nnz; ++p)
        if (coords[3 * p + 1] < 0 || coords[3 * p + 1] >= J || coords[3 * p + 2] < 0 || coords[3 * p + 2] >= K) {
            free_buckets(&b);
            return -2;
        }
    set_threads(threads);
    #pragma omp parallel for schedule(dynamic, 16)
    for (int64_t o = 0; o < b.n_out; ++o) {
        double *Ao = A + o * M;
        double *So = S ? S + o * M : NULL;
        for (int64_t x = 0; x < M; ++x) Ao[x] = 0.0;
        if (So) for (int64_t x = 0; x < M; ++x) So[x] = 0.0;
        for (int64_t q = b.start[o]; q < b.start[o + 1]; ++q) {
            int64_t p = b.order[q];
            int64_t j = coords[3 * p + 1], k = coords[3 * p + 2];
            double v = (double)vals[p];
            for (int64_t r = 0; r < R; ++r)
                for (int64_t m = 0; m < M; ++m) {
                    double term = v * (double)C[j * R + r] * (double)D[k * R + r] * (double)E[r * M + m];
                    Ao[m] += term;
                    if (So) So[m] += fabs(term);
                }
        }
    }
    free_buckets(&b);
    return 0;
}

/* Kernel 5 <3D TTMC>:  A(l,m,n) = sum_{i,j,k} B(i,j,k) * C(i,l) * D(j,m) * E(k,n)  (all three
 * modes contracted; the running example of Sections 1, 3 and 4).  Every nonzero contributes to
 * every output element, so the loop nest is the linear one of the paper's first schedule with the
 * nonzero loop innermost per output element; threads split the output elements, the order of the
 * terms of one element is the input order.
 * n_sel > 0: only the output elements listed in sel (flat indices (l*M + m)*N + n) are computed,
 * A and S then hold n_sel values. */
int oracle_ttmc3(int64_t nnz, const int32_t *coords, const float *vals,
                 int64_t I, int64_t J, int64_t K, int64_t L, int64_t M, int64_t N,
                 const float *C, const float *D, const float *E,
                 int64_t n_sel, const int64_t *sel, double *A, double *S, int threads)
{
    for (int64_t p = 0; p < nnz; ++p)
        if (coords[3 * p] < 0 || coords[3 * p] >= I || coords[3 * p + 1] < 0 || coords[3 * p + 1] >= J ||
            coords[3 * p + 2] < 0 || coords[3 * p + 2] >= K)
            return -2;
    const int64_t n_out = sel ? n_sel : L * M * N;
    for (int64_t x = 0; x < n_out; ++x)
        if (sel && (sel[x] < 0 || sel[x] >= L * M * N)) return -2;
    set_threads(threads);
    #pragma omp parallel for schedule(static)
    for (int64_t x = 0; x < n_out; ++x) {
        const int64_t e = sel ? sel[x] : x;
        const int64_t l = e / (M * N), m = (e / N) % M, n = e % N;
        double a = 0.0, s = 0.0;
        for (int64_t p = 0; p < nnz; ++p) {
            const int64_t i = coords[3 * p], j = coords[3 * p + 1], k = coords[3 * p + 2];
            const double term = (double)vals[p] * (double)C[i * L + l] * (double)D[j * M + m] * (double)E[k * N + n];
            a += term;
            s += fabs(term);
        }
        A[x] = a;
        if (S) S[x] = s;
    }
    return 0;
}

/* Kernel 2 <SDDMM,SpMM,GEMM>:  A(i,m) = sum_{j,k,l} B(i,j) * C(i,k) * D(j,k) * E(j,l) * F(l,m). */
int oracle_sddmm_spmm_gemm(int64_t nnz, const int32_t *coords, const float *vals,
                           int64_t I, int64_t J, int64_t K, int64_t L, int64_t M,
                           const float *C, const float *D, const float *E, const float *F,
                           int64_t n_sel, const int64_t *sel, double *A, double *S, int threads)
{
    buckets_t b;
    int rc = make_buckets(&b, nnz, coords, 2, I, n_sel, sel);
    if (rc) { free_buckets(&b); return rc; }
    for (int64_t p = 0; p < nnz; ++p)
        if (coords[2 * p + 1] < 0 || coords[2 * p + 1] >= J) { free_buckets(&b); return -2; }
    set_threads(threads);
    #pragma omp parallel for schedule(dynamic, 4)
    for (int64_t o = 0; o < b.n_out; ++o) {
        double *Ao = A + o * M;
        double *So = S ? S + o * M : NULL;
        for (int64_t x = 0; x < M; ++x) Ao[x] = 0.0;
        if (So) for (int64_t x = 0; x < M; ++x) So[x] = 0.0;
        for (int64_t q = b.start[o]; q < b.start[o + 1]; ++q) {
            int64_t p = b.order[q];
            int64_t i = coords[2 * p], j = coords[2 * p + 1];
            double v = (double)vals[p];
            for (int64_t k = 0; k < K; ++k)
                for (int64_t l = 0; l < L; ++l)
                    for (int64_t m = 0; m < M; ++m) {
                        double term = v * (double)C[i * K + k] * (double)D[j * K + k] * (double)E[j * L + l] * (double)F[l * M + m];
                        Ao[m] += term;
                        if (So) So[m] += fabs(term);
                    }
        }
    }
    free_buckets(&b);
    return 0;
}
