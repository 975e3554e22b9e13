/*
 * Adasum fp64 CPU oracle — TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, literal statement of what the paper's N-way Adasum combine computes.
 * Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may call it.
 * It shares no code, header, table or helper with the CUDA library.
 *
 * What it follows (arXiv 2006.02924):
 *   - the pair operator, Section 3 (the displayed Adasum equation) and the
 *     "Apply Adasum" step of Algorithm 1:
 *         Adasum(a,b) = (1 - a.b / (2 |a|^2)) a + (1 - a.b / (2 |b|^2)) b
 *     with v = [a.b, a.a, b.b] the three scalars of Algorithm 1's "partial dot products" step;
 *   - the N-way form, Section 3.4 (recursive halves) realised bottom-up as Algorithm 1 does:
 *     neighbours at distance 1 first (workers 2i and 2i+1), then blocks of 2, 4, ...;
 *   - per-layer application, Section 3.6 / Section 4.4.3: every tensor of the fused buffer
 *     is reduced on its own, with its own dot products and norms;
 *   - wide accumulation, Section 4.4.1: dot products and norms are accumulated in double.
 *
 * Readings where the paper is silent:
 *   - |g|^2 is the squared L2 norm (Algorithm 1 uses a.a and b.b);
 *   - an operand whose squared norm is exactly zero gets coefficient 1 (it contributes
 *     nothing, and the other operand passes through unchanged); no epsilon anywhere;
 *   - when the number of operands at a level is odd (the paper requires a power of two),
 *     the unpaired last operand is carried to the next level unchanged;
 *   - N = 1 returns the input.
 *
 * Everything is fp64: inputs are converted exactly from their stored bits, every
 * intermediate vector stays fp64, sums run left to right.
 *
 * Pins (tests that do not go through this file's own formula): orthogonal pair -> a+b,
 * parallel pair -> (1+c)/2 g, swap symmetry, two-order average, explicit matrix form,
 * N-way orthogonal / identical extremes of the orthogonality measure, top-down brute
 * force in numpy, zero-norm rules, homogeneity, norm identity and bound, the 0.9428
 * lemma value.  Full-size benchmark configurations have no printed expected values in
 * the paper: beyond those pins they are parity unpinned except through this oracle.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_F16 = 1, ORACLE_BF16 = 2, ORACLE_F64 = 3 };

/* Exact conversion of one stored element to double. */
static double element_as_double(const void *buf, int dtype, int64_t i)
{
    switch (dtype) {
    case ORACLE_F64:
        return ((const double *)buf)[i];
    case ORACLE_F32:
        return (double)((const float *)buf)[i];
    case ORACLE_BF16: {
        uint32_t bits = ((uint32_t)((const uint16_t *)buf)[i]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    case ORACLE_F16: {
        uint16_t h = ((const uint16_t *)buf)[i];
        int sign = (h >> 15) & 1;
        int expo = (h >> 10) & 0x1f;
        int mant = h & 0x3ff;
        double v;
        if (expo == 0)
            v = ldexp((double)mant, -24);              /* zero and subnormals */
        else if (expo == 31)
            v = mant ? NAN : INFINITY;
        else
            v = ldexp(1.0 + (double)mant / 1024.0, expo - 15);
        return sign ? -v : v;
    }
    default:
        return NAN;
    }
}

/* Algorithm 1, "Apply Adasum": the two scale factors from v = [a.b, a.a, b.b].
 * Zero-norm reading: a zero operand keeps coefficient 1. */
void adasum_oracle_coefficients(double dot, double norm_a, double norm_b,
                                double *coef_a, double *coef_b)
{
    *coef_a = (norm_a == 0.0) ? 1.0 : 1.0 - dot / (2.0 * norm_a);
    *coef_b = (norm_b == 0.0) ? 1.0 : 1.0 - dot / (2.0 * norm_b);
}

/* One application of the operator on two fp64 vectors of length n; result into dst
 * (dst may be a). */
static void adasum_two(const double *a, const double *b, int64_t n, double *dst)
{
    double dot = 0.0, norm_a = 0.0, norm_b = 0.0;
    for (int64_t e = 0; e < n; ++e) {
        dot += a[e] * b[e];
        norm_a += a[e] * a[e];
        norm_b += b[e] * b[e];
    }
    double ca, cb;
    adasum_oracle_coefficients(dot, norm_a, norm_b, &ca, &cb);
    for (int64_t e = 0; e < n; ++e)
        dst[e] = ca * a[e] + cb * b[e];
}

/* Binary tree over the N operands of ONE tensor (Section 3.4; Algorithm 1's bottom-up
 * order: pairs (2i, 2i+1) at every level).  x[w] are fp64 working vectors that are
 * overwritten.  The result ends in x[0]. */
static void adasum_tree(double **x, int n_operands, int64_t n)
{
    int m = n_operands;
    while (m > 1) {
        int pairs = m / 2;
        for (int i = 0; i < pairs; ++i) {
            double *a = x[2 * i], *b = x[2 * i + 1];
            adasum_two(a, b, n, a);
            double *tmp = x[i];           /* keep every buffer reachable for free() */
            x[i] = a;
            x[2 * i] = tmp;
        }
        if (m & 1) {                      /* odd count: carry the last operand */
            double *tmp = x[pairs];
            x[pairs] = x[m - 1];
            x[m - 1] = tmp;
        }
        m = (m + 1) / 2;
    }
}

/* The recursion of Section 3.4 taken top-down, Adasum(g[lo, hi)) = Adasum(Adasum(left half),
 * Adasum(right half)), the left half holding floor(count / 2) operands.  For a power-of-two count
 * this is the same tree as adasum_tree; otherwise the shapes differ.  Result in x[lo]. */
static void adasum_halves(double **x, int lo, int hi, int64_t n)
{
    if (hi - lo < 2)
        return;
    int mid = lo + (hi - lo) / 2;
    adasum_halves(x, lo, mid, n);
    adasum_halves(x, mid, hi, n);
    adasum_two(x[lo], x[mid], n, x[lo]);
}

/* Linear order of Section 3.4: Adasum(g[0..n+1]) = Adasum(Adasum(g[0..n]), g[n+1]). */
static void adasum_chain(double **x, int n_operands, int64_t n)
{
    for (int w = 1; w < n_operands; ++w)
        adasum_two(x[0], x[w], n, x[0]);
}

static int reduce_tensor(const void *const *grads, int dtype, int64_t begin, int64_t end,
                         int n_workers, int linear_order, double *out, double *sum_leaf_norms)
{
    int64_t n = end - begin;
    double **x = (double **)calloc((size_t)n_workers, sizeof(double *));
    if (!x)
        return 1;
    int rc = 0;
    double leaf_norms = 0.0;
    for (int w = 0; w < n_workers && !rc; ++w) {
        x[w] = (double *)malloc((size_t)(n > 0 ? n : 1) * sizeof(double));
        if (!x[w]) {
            rc = 1;
            break;
        }
        for (int64_t e = 0; e < n; ++e) {
            x[w][e] = element_as_double(grads[w], dtype, begin + e);
            leaf_norms += x[w][e] * x[w][e];
        }
    }
    if (!rc) {
        if (linear_order == 1)
            adasum_chain(x, n_workers, n);
        else if (linear_order == 2)
            adasum_halves(x, 0, n_workers, n);
        else
            adasum_tree(x, n_workers, n);
        memcpy(out + begin, x[0], (size_t)n * sizeof(double));
        if (sum_leaf_norms)
            *sum_leaf_norms = leaf_norms;
    }
    for (int w = 0; w < n_workers; ++w)
        free(x[w]);
    free(x);
    return rc;
}

/*
 * N-way Adasum of N fused gradient buffers, tensor by tensor.
 *   grads          N host pointers, each a buffer of offsets[num_tensors] elements of `dtype`
 *   offsets        num_tensors+1 element offsets, offsets[0] = 0, non-decreasing
 *   linear_order   0: binary tree, bottom-up pairs (the form used in practice); 1: the sequential
 *                  recursion; 2: the binary tree taken top-down by halves
 *   out            offsets[num_tensors] doubles
 *   orthogonality  optional, num_tensors doubles: |Adasum(g_1..g_N)|^2 / sum_i |g_i|^2
 *                  (Section 3.6); NaN for a tensor whose leaves are all zero
 *   threads        tensors are independent, so they may be reduced on several threads;
 *                  the arithmetic inside one tensor is never split.  <= 0: library default
 * Returns 0, or 1 on allocation failure / bad arguments.
 */
int adasum_oracle_reduce(const void *const *grads, int dtype, const int64_t *offsets,
                         int num_tensors, int n_workers, int linear_order, double *out,
                         double *orthogonality, int threads)
{
    if (!grads || !offsets || !out || num_tensors < 0 || n_workers < 1 || dtype < 0 || dtype > 3)
        return 1;
    int failed = 0;
#ifdef _OPENMP
    if (threads > 0)
        omp_set_num_threads(threads);
#else
    (void)threads;
#endif
#pragma omp parallel for schedule(dynamic, 1) reduction(| : failed)
    for (int t = 0; t < num_tensors; ++t) {
        double leaf_norms = 0.0;
        int rc = reduce_tensor(grads, dtype, offsets[t], offsets[t + 1], n_workers, linear_order,
                               out, &leaf_norms);
        failed |= rc;
        if (!rc && orthogonality) {
            double norm_out = 0.0;
            for (int64_t e = offsets[t]; e < offsets[t + 1]; ++e)
                norm_out += out[e] * out[e];
            orthogonality[t] = (leaf_norms == 0.0) ? NAN : norm_out / leaf_norms;
        }
    }
    return failed;
}

/* Number of threads the reduce call will actually use for `threads`. */
int adasum_oracle_threads(int threads)
{
#ifdef _OPENMP
    return threads > 0 ? threads : omp_get_max_threads();
#else
    (void)threads;
    return 1;
#endif
}
