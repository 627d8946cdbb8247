/*
 * CPU oracle, second form: the CSB matrix-vector product as the plain loop nest of the paper's
 * CSB-Engine (Section 4.3.1) -- for every block read the kept inputs through ColIdx, multiply by
 * the kernel matrix, accumulate into the outputs through RowIdx, block-rows accumulated
 * horizontally -- on the five arrays of Section 3.1.1 (n{}, m{}, RowIdx{}, ColIdx{}, Val{}).
 *
 * TEST INFRASTRUCTURE ONLY: no code is shared with the CUDA library, and no product path may call
 * this.  It exists so that the reported CPU baseline does the method's compressed work rather than
 * the dense work the method avoids.  Double accumulation, no blocking or vectorisation tricks.
 * Pinned by tests/test_oracle_csb.py against the float64 masked-dense product.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC -o libcsb_loops.so csb_loops.c
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <time.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int64_t rows, cols, nbr, nbc, nnz;
    int br, bc;
    int32_t *m, *n;          /* kept rows / columns per block            */
    int64_t *val_off;        /* prefix sums of m*n                       */
    int64_t *ridx_off, *cidx_off;
    int32_t *row_idx, *col_idx;
    double *val;             /* kernel matrices, row-major inside a block */
} csb_loops_t;

/* Encode: `stored` holds the values as stored (already rounded to the storage type by the caller). */
csb_loops_t* csb_loops_encode(const float* stored, int64_t rows, int64_t cols, int br, int bc,
                              const uint8_t* row_keep, const uint8_t* col_keep) {
    csb_loops_t* A = (csb_loops_t*)calloc(1, sizeof *A);
    A->rows = rows; A->cols = cols; A->br = br; A->bc = bc;
    A->nbr = (rows + br - 1) / br; A->nbc = (cols + bc - 1) / bc;
    const int64_t nblk = A->nbr * A->nbc;
    A->m = calloc(nblk, sizeof(int32_t)); A->n = calloc(nblk, sizeof(int32_t));
    A->val_off = calloc(nblk + 1, sizeof(int64_t));
    A->ridx_off = calloc(nblk + 1, sizeof(int64_t)); A->cidx_off = calloc(nblk + 1, sizeof(int64_t));
    for (int64_t b = 0; b < nblk; ++b) {
        const int64_t bi = b / A->nbc, bj = b % A->nbc;
        int m = 0, n = 0;
        for (int i = 0; i < br && bi * br + i < rows; ++i) m += row_keep[b * br + i] != 0;
        for (int j = 0; j < bc && bj * bc + j < cols; ++j) n += col_keep[b * bc + j] != 0;
        A->m[b] = m; A->n[b] = n;
        A->val_off[b + 1] = A->val_off[b] + (int64_t)m * n;
        A->ridx_off[b + 1] = A->ridx_off[b] + m; A->cidx_off[b + 1] = A->cidx_off[b] + n;
    }
    A->nnz = A->val_off[nblk];
    A->row_idx = calloc(A->ridx_off[nblk] + 1, sizeof(int32_t));
    A->col_idx = calloc(A->cidx_off[nblk] + 1, sizeof(int32_t));
    A->val = calloc(A->nnz + 1, sizeof(double));
    for (int64_t b = 0; b < nblk; ++b) {
        const int64_t bi = b / A->nbc, bj = b % A->nbc;
        int32_t* ri = A->row_idx + A->ridx_off[b]; int32_t* ci = A->col_idx + A->cidx_off[b];
        int m = 0, n = 0;
        for (int i = 0; i < br && bi * br + i < rows; ++i) if (row_keep[b * br + i]) ri[m++] = i;
        for (int j = 0; j < bc && bj * bc + j < cols; ++j) if (col_keep[b * bc + j]) ci[n++] = j;
        double* v = A->val + A->val_off[b];
        for (int r = 0; r < m; ++r)
            for (int k = 0; k < n; ++k) *v++ = (double)stored[(bi * br + ri[r]) * cols + bj * bc + ci[k]];
    }
    return A;
}

int64_t csb_loops_nnz(const csb_loops_t* A) { return A->nnz; }

void csb_loops_free(csb_loops_t* A) {
    if (!A) return;
    free(A->m); free(A->n); free(A->val_off); free(A->ridx_off); free(A->cidx_off);
    free(A->row_idx); free(A->col_idx); free(A->val); free(A);
}

/* y = A . x ; block-rows are independent, so threads take whole block-rows. */
void csb_loops_spmv(const csb_loops_t* A, const double* x, double* y, int threads) {
    memset(y, 0, (size_t)A->rows * sizeof(double));
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads > 0 ? threads : 1)
#endif
    for (int64_t bi = 0; bi < A->nbr; ++bi)
        for (int64_t bj = 0; bj < A->nbc; ++bj) {
            const int64_t b = bi * A->nbc + bj;
            const int32_t* ri = A->row_idx + A->ridx_off[b]; const int32_t* ci = A->col_idx + A->cidx_off[b];
            const double* v = A->val + A->val_off[b];
            const int m = A->m[b], n = A->n[b];
            for (int r = 0; r < m; ++r) {
                double acc = 0.0;
                for (int k = 0; k < n; ++k) acc += v[(int64_t)r * n + k] * x[bj * A->bc + ci[k]];
                y[bi * A->br + ri[r]] += acc;
            }
        }
}

/* Seconds per product over `reps` products (wall clock). */
double csb_loops_time_spmv(const csb_loops_t* A, const double* x, double* y, int threads, int reps) {
    struct timespec t0, t1;
    clock_gettime(CLOCK_MONOTONIC, &t0);
    for (int i = 0; i < reps; ++i) csb_loops_spmv(A, x, y, threads);
    clock_gettime(CLOCK_MONOTONIC, &t1);
    return ((t1.tv_sec - t0.tv_sec) + 1e-9 * (t1.tv_nsec - t0.tv_nsec)) / (reps > 0 ? reps : 1);
}
