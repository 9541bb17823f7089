/* TEST INFRASTRUCTURE ONLY: the paper's scheduled loop nests on the CPU.
 *
 * oracle.c evaluates every chain as its unfused definition (one perfectly nested loop per stored nonzero).  This
 * file evaluates the same chains the way the paper schedules them: the branched nests of the Table of kernels
 * (Section 6), with their temporaries, over CSR / CSF storage (pos / crd arrays per level, Section 2.1), in the
 * paper's loop order and letters.  It serves two purposes and no product code uses it:
 *   - a second, structurally different evaluation that must agree with the definition (Section 4: every
 *     fissioned and fused schedule computes the unfused Einsum), which pins the oracle and the schedules at once;
 *   - a CPU time for the schedule the GPU path runs, next to the time of the unfused definition.
 * Inputs are fp32 (as stored), temporaries and outputs fp64.  The outer loop over i runs in parallel (OpenMP,
 * dynamic), every iteration owning its own output rows; kernel 5 reduces per-thread copies of its output.
 *
 * Storage.  CSR: pos1[I + 1], crd1[nnz] (columns j), vals.  CSF order 3: slice_i[S] (the non-empty slices),
 * pos1[S + 1] over fibers, crd1[F] (j), pos2[F + 1] over nonzeros, crd2[nnz] (k), vals.  Order 4 has one level more.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static void set_threads(int threads)
{
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
}

/* Kernel 6 <SpTTM,TTM>, nest  i, j' < t(m) ; k': t(m) += B(i,j,k) D(k,m) , l,m: A(i,l,m) += t(m) C(j,l) >.
 * A (I x L x M) must be zero on entry. */
int nest_spttm_ttm3(int64_t S, const int32_t *slice_i, const int64_t *pos1, const int32_t *crd1, const int64_t *pos2,
                    const int32_t *crd2, const float *vals, int64_t L, int64_t M, const float *C, const float *D,
                    double *A, int threads)
{
    set_threads(threads);
    int bad = 0;
    #pragma omp parallel
    {
        double *t = (double *)malloc(sizeof(double) * (size_t)M);
        if (!t) {
            #pragma omp atomic write
            bad = 1;
        }
        #pragma omp barrier
        if (!bad) {
            #pragma omp for schedule(dynamic, 4)
            for (int64_t s = 0; s < S; ++s) {
                double *Ai = A + (int64_t)slice_i[s] * L * M;
                for (int64_t f = pos1[s]; f < pos1[s + 1]; ++f) {             /* j' */
                    const int64_t j = crd1[f];
                    for (int64_t m = 0; m < M; ++m) t[m] = 0.0;
                    for (int64_t p = pos2[f]; p < pos2[f + 1]; ++p) {          /* k' */
                        const double b = (double)vals[p];
                        const float *Dk = D + (int64_t)crd2[p] * M;
                        for (int64_t m = 0; m < M; ++m) t[m] += b * (double)Dk[m];
                    }
                    for (int64_t l = 0; l < L; ++l) {
                        const double c = (double)C[j * L + l];
                        for (int64_t m = 0; m < M; ++m) Ai[l * M + m] += t[m] * c;
                    }
                }
            }
        }
        free(t);
    }
    return bad ? -1 : 0;
}

/* Order-4 chain with the two-level nesting of kernel 5's second schedule:
 *   i, j' < T2(m,n) ; k' < t(n) ; o': t(n) += B(i,j,k,o) E(o,n) , m,n: T2(m,n) += t(n) D(k,m) > ,
 *                     l,m,n: A(i,l,m,n) += T2(m,n) C(j,l) >.
 * A (I x L x M x N) must be zero on entry. */
int nest_spttm_ttm4(int64_t S, const int32_t *slice_i, const int64_t *pos1, const int32_t *crd1, const int64_t *pos2,
                    const int32_t *crd2, const int64_t *pos3, const int32_t *crd3, const float *vals, int64_t L, int64_t M,
                    int64_t N, const float *C, const float *D, const float *E, double *A, int threads)
{
    set_threads(threads);
    int bad = 0;
    #pragma omp parallel
    {
        double *t = (double *)malloc(sizeof(double) * (size_t)(N + M * N));
        double *T2 = t ? t + N : NULL;
        if (!t) {
            #pragma omp atomic write
            bad = 1;
        }
        #pragma omp barrier
        if (!bad) {
            #pragma omp for schedule(dynamic, 1)
            for (int64_t s = 0; s < S; ++s) {
                double *Ai = A + (int64_t)slice_i[s] * L * M * N;
                for (int64_t f = pos1[s]; f < pos1[s + 1]; ++f) {                 /* j' */
                    const int64_t j = crd1[f];
                    for (int64_t x = 0; x < M * N; ++x) T2[x] = 0.0;
                    for (int64_t g = pos2[f]; g < pos2[f + 1]; ++g) {              /* k' */
                        const float *Dk = D + (int64_t)crd2[g] * M;
                        for (int64_t n = 0; n < N; ++n) t[n] = 0.0;
                        for (int64_t p = pos3[g]; p < pos3[g + 1]; ++p) {          /* o' */
                            const double b = (double)vals[p];
                            const float *Eo = E + (int64_t)crd3[p] * N;
                            for (int64_t n = 0; n < N; ++n) t[n] += b * (double)Eo[n];
                        }
                        for (int64_t m = 0; m < M; ++m) {
                            const double d = (double)Dk[m];
                            for (int64_t n = 0; n < N; ++n) T2[m * N + n] += t[n] * d;
                        }
                    }
                    for (int64_t l = 0; l < L; ++l) {
                        const double c = (double)C[j * L + l];
                        for (int64_t x = 0; x < M * N; ++x) Ai[l * M * N + x] += T2[x] * c;
                    }
                }
            }
        }
        free(t);
    }
    return bad ? -1 : 0;
}

/* Kernel 1 <SDDMM,SpMM>, nest  i, j' < t ; k: t += B(i,j) C(i,k) D(j,k) , l: A(i,l) += t E(j,l) >.
 * A (I x L) must be zero on entry. */
int nest_sddmm_spmm(int64_t I, const int64_t *pos1, const int32_t *crd1, const float *vals, int64_t K, int64_t L,
                    const float *C, const float *D, const float *E, double *A, int threads)
{
    set_threads(threads);
    #pragma omp parallel for schedule(dynamic, 64)
    for (int64_t i = 0; i < I; ++i) {
        const float *Ci = C + i * K;
        double *Ai = A + i * L;
        for (int64_t p = pos1[i]; p < pos1[i + 1]; ++p) {                          /* j' */
            const int64_t j = crd1[p];
            const double b = (double)vals[p];
            const float *Dj = D + j * K, *Ej = E + j * L;
            double t = 0.0;
            for (int64_t k = 0; k < K; ++k) t += b * (double)Ci[k] * (double)Dj[k];
            for (int64_t l = 0; l < L; ++l) Ai[l] += t * (double)Ej[l];
        }
    }
    return 0;
}

/* Kernel 4 <SpMM,GEMM> as the Table of kernels schedules it, nest
 *   i < T(l) ; j',l: T(l) += B(i,j) C(j,l) , l,m: A(i,m) += T(l) D(l,m) >.   A (I x M) must be zero on entry. */
int nest_spmm_gemm_left(int64_t I, const int64_t *pos1, const int32_t *crd1, const float *vals, int64_t L, int64_t M,
                        const float *C, const float *D, double *A, int threads)
{
    set_threads(threads);
    int bad = 0;
    #pragma omp parallel
    {
        double *T = (double *)malloc(sizeof(double) * (size_t)L);
        if (!T) {
            #pragma omp atomic write
            bad = 1;
        }
        #pragma omp barrier
        if (!bad) {
            #pragma omp for schedule(dynamic, 64)
            for (int64_t i = 0; i < I; ++i) {
                for (int64_t l = 0; l < L; ++l) T[l] = 0.0;
                for (int64_t p = pos1[i]; p < pos1[i + 1]; ++p) {                  /* j' */
                    const double b = (double)vals[p];
                    const float *Cj = C + (int64_t)crd1[p] * L;
                    for (int64_t l = 0; l < L; ++l) T[l] += b * (double)Cj[l];
                }
                double *Ai = A + i * M;
                for (int64_t l = 0; l < L; ++l) {
                    const double tl = T[l];
                    const float *Dl = D + l * M;
                    for (int64_t m = 0; m < M; ++m) Ai[m] += tl * (double)Dl[m];
                }
            }
        }
        free(T);
    }
    return bad ? -1 : 0;
}

/* The other association order of kernel 4, with the J x M temporary that Stage 1 of the scheduler admits
 * (Section 5.2): j,l,m: E(j,m) += C(j,l) D(l,m) ; i, j', m: A(i,m) += B(i,j) E(j,m).
 * Etmp (J x M) is caller-provided scratch; A (I x M) must be zero on entry. */
int nest_spmm_gemm_right(int64_t I, int64_t J, const int64_t *pos1, const int32_t *crd1, const float *vals, int64_t L, int64_t M,
                         const float *C, const float *D, double *Etmp, double *A, int threads)
{
    set_threads(threads);
    #pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < J; ++j) {
        double *Ej = Etmp + j * M;
        for (int64_t m = 0; m < M; ++m) Ej[m] = 0.0;
        for (int64_t l = 0; l < L; ++l) {
            const double c = (double)C[j * L + l];
            const float *Dl = D + l * M;
            for (int64_t m = 0; m < M; ++m) Ej[m] += c * (double)Dl[m];
        }
    }
    #pragma omp parallel for schedule(dynamic, 64)
    for (int64_t i = 0; i < I; ++i) {
        double *Ai = A + i * M;
        for (int64_t p = pos1[i]; p < pos1[i + 1]; ++p) {                          /* j' */
            const double b = (double)vals[p];
            const double *Ej = Etmp + (int64_t)crd1[p] * M;
            for (int64_t m = 0; m < M; ++m) Ai[m] += b * Ej[m];
        }
    }
    return 0;
}

/* Kernel 5 <3D TTMC>, second schedule of the Table of kernels:
 *   i < T(m,n) ; j' < t(n) ; k': t(n) += B(i,j,k) E(k,n) , m,n: T(m,n) += t(n) D(j,m) > , l,m,n: A(l,m,n) += T(m,n) C(i,l) >.
 * Every thread adds into its own copy of A (L x M x N); the copies are summed in thread order.  A is overwritten. */
int nest_ttmc3(int64_t S, const int32_t *slice_i, const int64_t *pos1, const int32_t *crd1, const int64_t *pos2,
               const int32_t *crd2, const float *vals, int64_t L, int64_t M, int64_t N, const float *C, const float *D,
               const float *E, double *A, int threads)
{
    set_threads(threads);
    int nt = 1;
#ifdef _OPENMP
    nt = omp_get_max_threads();
#endif
    const int64_t LMN = L * M * N;
    double *copies = (double *)calloc((size_t)nt * (size_t)LMN, sizeof(double));
    if (!copies) return -1;
    int bad = 0;
    #pragma omp parallel num_threads(nt)
    {
        int me = 0;
#ifdef _OPENMP
        me = omp_get_thread_num();
#endif
        double *Ame = copies + (int64_t)me * LMN;
        double *t = (double *)malloc(sizeof(double) * (size_t)(N + M * N));
        double *T = t ? t + N : NULL;
        if (!t) {
            #pragma omp atomic write
            bad = 1;
        }
        #pragma omp barrier
        if (!bad) {
            #pragma omp for schedule(dynamic, 4)
            for (int64_t s = 0; s < S; ++s) {
                const int64_t i = slice_i[s];
                for (int64_t x = 0; x < M * N; ++x) T[x] = 0.0;
                for (int64_t f = pos1[s]; f < pos1[s + 1]; ++f) {                  /* j' */
                    const float *Dj = D + (int64_t)crd1[f] * M;
                    for (int64_t n = 0; n < N; ++n) t[n] = 0.0;
                    for (int64_t p = pos2[f]; p < pos2[f + 1]; ++p) {              /* k' */
                        const double b = (double)vals[p];
                        const float *Ek = E + (int64_t)crd2[p] * N;
                        for (int64_t n = 0; n < N; ++n) t[n] += b * (double)Ek[n];
                    }
                    for (int64_t m = 0; m < M; ++m) {
                        const double d = (double)Dj[m];
                        for (int64_t n = 0; n < N; ++n) T[m * N + n] += t[n] * d;
                    }
                }
                for (int64_t l = 0; l < L; ++l) {
                    const double c = (double)C[i * L + l];
                    for (int64_t x = 0; x < M * N; ++x) Ame[l * M * N + x] += T[x] * c;
                }
            }
        }
        free(t);
    }
    for (int64_t x = 0; x < LMN; ++x) {
        double sum = 0.0;
        for (int w = 0; w < nt; ++w) sum += copies[(int64_t)w * LMN + x];
        A[x] = sum;
    }
    free(copies);
    return bad ? -1 : 0;
}

/* Kernel 2 <SDDMM,SpMM,GEMM>, two-level nest of the Table of kernels:
 *   i < T(l) ; j' < t ; k: t += B(i,j) C(i,k) D(j,k) , l: T(l) += t E(j,l) > , l,m: A(i,m) += T(l) F(l,m) >.
 * A (I x M) must be zero on entry. */
int nest_sddmm_spmm_gemm(int64_t I, const int64_t *pos1, const int32_t *crd1, const float *vals, int64_t K, int64_t L, int64_t M,
                         const float *C, const float *D, const float *E, const float *F, double *A, int threads)
{
    set_threads(threads);
    int bad = 0;
    #pragma omp parallel
    {
        double *T = (double *)malloc(sizeof(double) * (size_t)L);
        if (!T) {
            #pragma omp atomic write
            bad = 1;
        }
        #pragma omp barrier
        if (!bad) {
            #pragma omp for schedule(dynamic, 64)
            for (int64_t i = 0; i < I; ++i) {
                const float *Ci = C + i * K;
                for (int64_t l = 0; l < L; ++l) T[l] = 0.0;
                for (int64_t p = pos1[i]; p < pos1[i + 1]; ++p) {                  /* j' */
                    const int64_t j = crd1[p];
                    const double b = (double)vals[p];
                    const float *Dj = D + j * K, *Ej = E + j * L;
                    double t = 0.0;
                    for (int64_t k = 0; k < K; ++k) t += b * (double)Ci[k] * (double)Dj[k];
                    for (int64_t l = 0; l < L; ++l) T[l] += t * (double)Ej[l];
                }
                double *Ai = A + i * M;
                for (int64_t l = 0; l < L; ++l) {
                    const double tl = T[l];
                    const float *Fl = F + l * M;
                    for (int64_t m = 0; m < M; ++m) Ai[m] += tl * (double)Fl[m];
                }
            }
        }
        free(T);
    }
    return bad ? -1 : 0;
}

/* Kernel 3 <SpMMH,GEMM>, nest  i < T(l) ; j',l: T(l) += B(i,j) C(j,l) D(j,l) , l,m: A(i,m) += T(l) E(l,m) >.
 * A (I x M) must be zero on entry. */
int nest_spmmh_gemm(int64_t I, const int64_t *pos1, const int32_t *crd1, const float *vals, int64_t L, int64_t M,
                    const float *C, const float *D, const float *E, double *A, int threads)
{
    set_threads(threads);
    int bad = 0;
    #pragma omp parallel
    {
        double *T = (double *)malloc(sizeof(double) * (size_t)L);
        if (!T) {
            #pragma omp atomic write
            bad = 1;
        }
        #pragma omp barrier
        if (!bad) {
            #pragma omp for schedule(dynamic, 64)
            for (int64_t i = 0; i < I; ++i) {
                for (int64_t l = 0; l < L; ++l) T[l] = 0.0;
                for (int64_t p = pos1[i]; p < pos1[i + 1]; ++p) {                  /* j' */
                    const int64_t j = crd1[p];
                    const double b = (double)vals[p];
                    const float *Cj = C + j * L, *Dj = D + j * L;
                    for (int64_t l = 0; l < L; ++l) T[l] += b * (double)Cj[l] * (double)Dj[l];
                }
                double *Ai = A + i * M;
                for (int64_t l = 0; l < L; ++l) {
                    const double tl = T[l];
                    const float *El = E + l * M;
                    for (int64_t m = 0; m < M; ++m) Ai[m] += tl * (double)El[m];
                }
            }
        }
        free(T);
    }
    return bad ? -1 : 0;
}

/* Kernel 8 <MTTKRP,GEMM>, nest
 *   i < T(r) ; j' < t(r) ; k',r: t(r) += B(i,j,k) D(k,r) , r: T(r) += t(r) C(j,r) > , r,m: A(i,m) += T(r) E(r,m) >.
 * A (I x M) must be zero on entry. */
int nest_mttkrp_gemm(int64_t S, const int32_t *slice_i, const int64_t *pos1, const int32_t *crd1, const int64_t *pos2,
                     const int32_t *crd2, const float *vals, int64_t R, int64_t M, const float *C, const float *D,
                     const float *E, double *A, int threads)
{
    set_threads(threads);
    int bad = 0;
    #pragma omp parallel
    {
        double *t = (double *)malloc(sizeof(double) * (size_t)(2 * R));
        double *T = t ? t + R : NULL;
        if (!t) {
            #pragma omp atomic write
            bad = 1;
        }
        #pragma omp barrier
        if (!bad) {
            #pragma omp for schedule(dynamic, 4)
            for (int64_t s = 0; s < S; ++s) {
                for (int64_t r = 0; r < R; ++r) T[r] = 0.0;
                for (int64_t f = pos1[s]; f < pos1[s + 1]; ++f) {                  /* j' */
                    const float *Cj = C + (int64_t)crd1[f] * R;
                    for (int64_t r = 0; r < R; ++r) t[r] = 0.0;
                    for (int64_t p = pos2[f]; p < pos2[f + 1]; ++p) {              /* k' */
                        const double b = (double)vals[p];
                        const float *Dk = D + (int64_t)crd2[p] * R;
                        for (int64_t r = 0; r < R; ++r) t[r] += b * (double)Dk[r];
                    }
                    for (int64_t r = 0; r < R; ++r) T[r] += t[r] * (double)Cj[r];
                }
                double *Ai = A + (int64_t)slice_i[s] * M;
                for (int64_t r = 0; r < R; ++r) {
                    const double tr = T[r];
                    const float *Er = E + r * M;
                    for (int64_t m = 0; m < M; ++m) Ai[m] += tr * (double)Er[m];
                }
            }
        }
        free(t);
    }
    return bad ? -1 : 0;
}

/* Kernel 7 <SpTTM,SpTTM>, nest  i, j' < T(l) ; k',l: T(l) += B(i,j,k) C(k,l) , l,m: A(f,m) += T(l) D(l,m) >  with one
 * output row per level-1 fiber f = (i,j), in storage order (the output keeps B's (i,j) pattern).
 * A (F x M) must be zero on entry. */
int nest_spttm_spttm(int64_t F, const int64_t *pos2, const int32_t *crd2, const float *vals, int64_t L, int64_t M,
                     const float *C, const float *D, double *A, int threads)
{
    set_threads(threads);
    int bad = 0;
    #pragma omp parallel
    {
        double *T = (double *)malloc(sizeof(double) * (size_t)L);
        if (!T) {
            #pragma omp atomic write
            bad = 1;
        }
        #pragma omp barrier
        if (!bad) {
            #pragma omp for schedule(dynamic, 64)
            for (int64_t f = 0; f < F; ++f) {                                      /* i, j' */
                for (int64_t l = 0; l < L; ++l) T[l] = 0.0;
                for (int64_t p = pos2[f]; p < pos2[f + 1]; ++p) {                  /* k' */
                    const double b = (double)vals[p];
                    const float *Ck = C + (int64_t)crd2[p] * L;
                    for (int64_t l = 0; l < L; ++l) T[l] += b * (double)Ck[l];
                }
                double *Af = A + f * M;
                for (int64_t l = 0; l < L; ++l) {
                    const double tl = T[l];
                    const float *Dl = D + l * M;
                    for (int64_t m = 0; m < M; ++m) Af[m] += tl * (double)Dl[m];
                }
            }
        }
        free(T);
    }
    return bad ? -1 : 0;
}
