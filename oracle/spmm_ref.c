/*
 * TEST INFRASTRUCTURE ONLY -- never part of the product path.
 *
 * Plain, single-threaded, fp64 reference for sparse x dense matrix
 * multiplication C = A x B (paper Sec. 2.3, "Sparse Formats": A is m x k and
 * sparse, B is k x n and dense).  A is read straight from CSR; none of the
 * paper's formats, tiles or schedules appear here, and no code is shared
 * with the CUDA library.
 *
 * Every input value (bf16 / fp16 / fp32 in storage) is widened to double by
 * the caller before this routine runs; the product of two such values is
 * exact in double, so C_ref is the real-number result up to ~1e-16 relative
 * accumulation error.  The routine also returns S[i][j] = sum_p |a_ip b_pj|,
 * which the parity tests use as the scale of the allowed error.
 *
 * Pins (tests/test_oracle_spmm.py): brute-force dense triple loop, identity
 * and permutation matrices, all-ones closed form, exact integer linearity,
 * empty rows, column independence.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

/*
 * C[i][j] = sum_{p = row_ptr[i]}^{row_ptr[i+1]-1} vals[p] * B[col_idx[p]][j]
 * S[i][j] = sum of |vals[p] * B[col_idx[p]][j]| over the same p
 *
 * rows i in [row_begin, row_end) only (lets a caller time or check a slice;
 * every row is independent).  B is row-major with leading dimension ldb,
 * C and S are row-major with leading dimension ldc and are fully
 * overwritten for the requested rows.  S may be NULL.
 */
void spmm_csr_ref(int64_t row_begin, int64_t row_end, int64_t n,
                  const int64_t *row_ptr, const int32_t *col_idx,
                  const double *vals, const double *B, int64_t ldb,
                  double *C, double *S, int64_t ldc)
{
    for (int64_t i = row_begin; i < row_end; ++i) {
        double *c = C + (size_t)i * (size_t)ldc;
        double *s = S ? S + (size_t)i * (size_t)ldc : NULL;
        for (int64_t j = 0; j < n; ++j) {
            c[j] = 0.0;
            if (s) s[j] = 0.0;
        }
        for (int64_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
            const double a = vals[p];
            const double *b = B + (size_t)col_idx[p] * (size_t)ldb;
            for (int64_t j = 0; j < n; ++j) {
                const double t = a * b[j];
                c[j] += t;
                if (s) s[j] += fabs(t);
            }
        }
    }
}
