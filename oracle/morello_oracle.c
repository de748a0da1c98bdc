/*
 * CPU oracle for MatmulAccum  --  TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * Only the tests, the smoke check and the benchmark's cpu_baseline / reference
 * leg may call this file.  It shares no code with the CUDA library and is
 * never a fallback for it.
 *
 * What it computes (paper Section 2, "Tiling": dimensions are ordered
 * batch, m, k, n and the output is batch x m x n; Section 2.2: the
 * accumulating primitive MatmulAccum adds into the existing contents of its
 * output, and the operand types are bf16, bf16 -> f32; Section 2.2 item 3 on
 * Move: a bf16 -> f32 move is an upcast copy, i.e. the inputs are widened
 * exactly before they are multiplied):
 *
 *     C[b,i,j]  <-  C[b,i,j] + sum_{p=0}^{k-1} A[b,i,p] * B[b,p,j]
 *
 * Layout: dense row-major A[b][m][k], B[b][k][n] (bf16 bit patterns in
 * uint16_t), C[b][m][n] (float).
 *
 * Precision: the paper fixes no summation order (Section 2: the iteration
 * order of a tile loop is undefined; Section 2.2 says only that MatmulAccum
 * accumulates into its output), so the oracle is the plain definition: add the
 * exact products (a bf16 x bf16 product has at most 16 significant bits, exact
 * in double) for p = 0..k-1 in increasing order in double, starting from zero,
 * then add (double)C, and round ONCE to float (round-to-nearest-even, the C
 * default).  C comes last because a double has 53 bits: a sum that starts
 * from C loses low bits of C as soon as a partial sum exceeds 2^29 |C|, and
 * does not get them back when the products cancel (exact rational arithmetic
 * finds such elements in long sums of small integers); with C last the sum of
 * integer-valued products is exact and C enters with one rounding.
 *
 * Pins (tests/test_oracle_pins.py): exact rational brute force on tiny
 * shapes, closed forms, identity / zero / one-hot operands, the accumulate
 * invariant, integer exactness against integer matrix products, power-of-two
 * scaling, and agreement with a float64 library contraction.
 * NaN / Inf / subnormal inputs follow IEEE 754 through the C arithmetic below;
 * a pin with hand-written expectations (subnormal inputs and sums, infinities
 * of both signs, NaN operands, Inf x 0, Inf - Inf) fixes that for every variant.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

/* bf16 is the upper 16 bits of an IEEE binary32: widening is a 16-bit shift. */
static inline double bf16_to_double(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/*
 * The definition, written as the literal triple loop (b, i, j, p).
 * Serial; meant for small shapes.
 */
void oracle_matmul_accum_naive(int64_t b, int64_t m, int64_t k, int64_t n,
                               const uint16_t *A, const uint16_t *B, float *C)
{
    for (int64_t bb = 0; bb < b; ++bb)
        for (int64_t i = 0; i < m; ++i)
            for (int64_t j = 0; j < n; ++j) {
                double s = 0.0;
                for (int64_t p = 0; p < k; ++p)
                    s += bf16_to_double(A[(bb * m + i) * k + p]) *
                         bf16_to_double(B[(bb * k + p) * n + j]);
                C[(bb * m + i) * n + j] = (float)((double)C[(bb * m + i) * n + j] + s);
            }
}

/* Columns are handed out in blocks of this many, so that a problem with few
 * rows (the vector-matrix multiply has one) still uses every host thread. */
#define ORACLE_COL_BLOCK 1024

/*
 * Columns [j0, j1) of one output row (bb, i): the same arithmetic per element
 * in the same p order as the triple loop, with the j loop innermost so that B
 * is walked along its rows.  `s` is a caller-provided buffer of j1 - j0
 * doubles.  If T_row is not NULL it receives sum_p |A[b,i,p] * B[b,p,j]| (the
 * scale of the floating-point tolerance) for those columns.
 */
static void oracle_row(int64_t bb, int64_t i, int64_t m, int64_t k, int64_t n,
                       int64_t j0, int64_t j1,
                       const uint16_t *A, const uint16_t *B,
                       const float *Cin_row, float *Cout_row, double *T_row,
                       double *s)
{
    for (int64_t j = j0; j < j1; ++j) s[j - j0] = 0.0;
    if (T_row) for (int64_t j = j0; j < j1; ++j) T_row[j] = 0.0;
    for (int64_t p = 0; p < k; ++p) {
        const double a = bf16_to_double(A[(bb * m + i) * k + p]);
        const uint16_t *Brow = B + (bb * k + p) * n;
        for (int64_t j = j0; j < j1; ++j) s[j - j0] += a * bf16_to_double(Brow[j]);
        if (T_row)
            for (int64_t j = j0; j < j1; ++j)
                T_row[j] += fabs(a * bf16_to_double(Brow[j]));
    }
    for (int64_t j = j0; j < j1; ++j) Cout_row[j] = (float)((double)Cin_row[j] + s[j - j0]);
}

/*
 * Whole problem, in place on C.  Output elements are independent, so (row,
 * column block) tasks are handed to host threads (OpenMP) when the library is
 * built with -fopenmp; the arithmetic of every element is unchanged by the
 * threading.  Returns 0, or -1 if the scratch buffer could not be allocated.
 */
int oracle_matmul_accum(int64_t b, int64_t m, int64_t k, int64_t n,
                        const uint16_t *A, const uint16_t *B, float *C)
{
    if (b <= 0 || m <= 0 || n <= 0) return 0;
    const int64_t nblk = (n + ORACLE_COL_BLOCK - 1) / ORACLE_COL_BLOCK;
    int failed = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc(ORACLE_COL_BLOCK * sizeof(double));
        if (!s) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int64_t t = 0; t < b * m * nblk; ++t) {
                const int64_t r = t / nblk, j0 = (t % nblk) * ORACLE_COL_BLOCK;
                const int64_t j1 = j0 + ORACLE_COL_BLOCK < n ? j0 + ORACLE_COL_BLOCK : n;
                float *row = C + r * n;
                oracle_row(r / m, r % m, m, k, n, j0, j1, A, B, row, row, NULL, s);
            }
        }
        free(s);
    }
    return failed ? -1 : 0;
}

/*
 * Selected rows only (for checking samples of a large problem and for timing
 * a bounded sample): rows[t] = bb * m + i.  C_in is the full input C and is
 * not modified; out[t][0..n) receives the result row; T (nrows x n doubles,
 * may be NULL) receives sum_p |A*B| for those rows.
 */
int oracle_matmul_accum_rows(int64_t b, int64_t m, int64_t k, int64_t n,
                             const uint16_t *A, const uint16_t *B,
                             const float *C_in, int64_t nrows,
                             const int64_t *rows, float *out, double *T)
{
    if (n <= 0 || nrows <= 0) return 0;
    const int64_t nblk = (n + ORACLE_COL_BLOCK - 1) / ORACLE_COL_BLOCK;
    int failed = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc(ORACLE_COL_BLOCK * sizeof(double));
        if (!s) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int64_t t = 0; t < nrows * nblk; ++t) {
                const int64_t q = t / nblk, j0 = (t % nblk) * ORACLE_COL_BLOCK;
                const int64_t j1 = j0 + ORACLE_COL_BLOCK < n ? j0 + ORACLE_COL_BLOCK : n;
                const int64_t r = rows[q];
                if (r < 0 || r >= b * m) continue;
                oracle_row(r / m, r % m, m, k, n, j0, j1, A, B, C_in + r * n,
                           out + q * n, T ? T + q * n : NULL, s);
            }
        }
        free(s);
    }
    return failed ? -1 : 0;
}

/*
 * T[b,i,j] = sum_p |A[b,i,p] * B[b,p,j]| in double: the magnitude the
 * floating-point acceptance rule scales with
 * (|gpu - oracle| <= 1e-5 * T + 1e-6).
 */
void oracle_abs_dot(int64_t b, int64_t m, int64_t k, int64_t n,
                    const uint16_t *A, const uint16_t *B, double *T)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < b * m; ++r) {
        const int64_t bb = r / m, i = r % m;
        double *Trow = T + r * n;
        for (int64_t j = 0; j < n; ++j) Trow[j] = 0.0;
        for (int64_t p = 0; p < k; ++p) {
            const double a = bf16_to_double(A[(bb * m + i) * k + p]);
            const uint16_t *Brow = B + (bb * k + p) * n;
            for (int64_t j = 0; j < n; ++j)
                Trow[j] += fabs(a * bf16_to_double(Brow[j]));
        }
    }
}

#ifdef _OPENMP
#include <omp.h>
int oracle_num_threads(void) { return omp_get_max_threads(); }
void oracle_set_num_threads(int t) { if (t > 0) omp_set_num_threads(t); }
#else
int oracle_num_threads(void) { return 1; }
void oracle_set_num_threads(int t) { (void)t; }
#endif

/*
 * The same operation on float32 inputs (the paper's other benchmark, Section 7: a
 * float32, 2048-square matrix multiplication):
 *
 *     C[b,i,j]  <-  C[b,i,j] + sum_{p=0}^{k-1} A[b,i,p] * B[b,p,j],   A, B, C float
 *
 * A product of two floats has at most 48 significant bits and is exact in double; the
 * sum starts from zero, runs over p in increasing order in double, (double)C is added
 * last and the result is rounded once to float.  T (may be NULL) receives sum_p |A*B|.  Rows are independent and are
 * handed to host threads.  Returns 0, or -1 if a row buffer could not be allocated.
 */
int oracle_matmul_accum_f32(int64_t b, int64_t m, int64_t k, int64_t n,
                            const float *A, const float *B, float *C, double *T)
{
    if (b <= 0 || m <= 0 || n <= 0) return 0;
    int failed = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc((size_t)n * sizeof(double));
        if (!s) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int64_t r = 0; r < b * m; ++r) {
                const int64_t bb = r / m;
                float *Crow = C + r * n;
                double *Trow = T ? T + r * n : NULL;
                for (int64_t j = 0; j < n; ++j) s[j] = 0.0;
                if (Trow) for (int64_t j = 0; j < n; ++j) Trow[j] = 0.0;
                for (int64_t p = 0; p < k; ++p) {
                    const double a = (double)A[r * k + p];
                    const float *Brow = B + (bb * k + p) * n;
                    for (int64_t j = 0; j < n; ++j) s[j] += a * (double)Brow[j];
                    if (Trow) for (int64_t j = 0; j < n; ++j) Trow[j] += fabs(a * (double)Brow[j]);
                }
                for (int64_t j = 0; j < n; ++j) Crow[j] = (float)((double)Crow[j] + s[j]);
            }
        }
        free(s);
    }
    return failed ? -1 : 0;
}

/*
 * The bf16 operation with the right-hand side stored column-major (the paper's Spec
 * carries a layout per operand; its Section 2.2 example has a col_major rhs):
 *
 *     C[b,i,j]  <-  C[b,i,j] + sum_{p=0}^{k-1} A[b,i,p] * Bt[b,j,p],   Bt[b][n][k]
 *
 * Same arithmetic as above (double accumulation of exact products in increasing p, C added
 * last, one rounding); only the indexing of the right-hand side differs.
 */
void oracle_matmul_accum_bt(int64_t b, int64_t m, int64_t k, int64_t n,
                            const uint16_t *A, const uint16_t *Bt, float *C)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < b * m; ++r) {
        const int64_t bb = r / m;
        for (int64_t j = 0; j < n; ++j) {
            double s = 0.0;
            const uint16_t *col = Bt + (bb * n + j) * k;
            for (int64_t p = 0; p < k; ++p)
                s += bf16_to_double(A[r * k + p]) * bf16_to_double(col[p]);
            C[r * n + j] = (float)((double)C[r * n + j] + s);
        }
    }
}

/*
 * The bf16 operation with the right-hand side in a packed layout (paper Section 2.4.2: a
 * layout may carry a strip dimension of size s on one logical dimension; Goto-style packing).
 * Here the strips run over the column index j: strip j / s holds columns [s (j / s), s (j / s) + s)
 * of every row, row-major inside the strip, and the strips follow one another,
 *
 *     offset(p, j) = (j / s) * k * s  +  p * s  +  (j mod s),      Bp[b][ceil(n / s)][k][s]
 *
 * (the last strip is padded to s columns; the padding is never read).
 *
 *     C[b,i,j]  <-  C[b,i,j] + sum_{p=0}^{k-1} A[b,i,p] * Bp[b][j / s][p][j mod s]
 *
 * Same arithmetic as everywhere above (double accumulation of exact products in increasing p,
 * C added last, one rounding); only the indexing of the right-hand side differs.
 */
void oracle_matmul_accum_packed_b(int64_t s, int64_t b, int64_t m, int64_t k, int64_t n,
                                  const uint16_t *A, const uint16_t *Bp, float *C)
{
    const int64_t strips = (n + s - 1) / s;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < b * m; ++r) {
        const int64_t bb = r / m;
        for (int64_t j = 0; j < n; ++j) {
            double sum = 0.0;
            const uint16_t *col = Bp + ((bb * strips + j / s) * k) * s + (j % s);
            for (int64_t p = 0; p < k; ++p)
                sum += bf16_to_double(A[r * k + p]) * bf16_to_double(col[p * s]);
            C[r * n + j] = (float)((double)C[r * n + j] + sum);
        }
    }
}
