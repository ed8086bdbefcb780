/*
 * CPU oracle for densifying IndexedSlices gradients.  TEST INFRASTRUCTURE ONLY:
 * nothing on the product path may call, link or import this file.  It shares
 * no code with the CUDA library.
 *
 * What it computes is the plain definition of the operation the paper
 * introduces in Section 4 ("Densifying Assumed-sparse Tensors", Listing 1):
 * an IndexedSlices gradient -- row indices plus [n_rows, d] value rows, as
 * described in Section 3 -- is converted to a dense [vocab, d] tensor, and the
 * dense tensors are then accumulated by reduction (Algorithm 1, the "reduce"
 * branch).  The R-way input is the concatenation of slices that Algorithm 1's
 * "gather" branch (and the cross-rank gather of Section 3) would have built.
 *
 *   out[v, c] = dense_in[v, c] (or 0)  +  sum over slices r, rows i with
 *                                          indices_r[i] == v of values_r[i, c]
 *
 * Written out as that double loop, one thread, no sorting, no blocking.  All
 * accumulation is in fp64 so the result does not depend on summation order at
 * the precision the tests look at.  Next to the sum it returns
 *   mag[v, c]  = |dense_in[v, c]| + sum |values_r[i, c]|     (the "sum of |terms|")
 *   cnt[v]     = number of valid input rows that name row v
 *   n_bad      = number of input rows whose index is outside [0, vocab)
 * Rows with an out-of-range index contribute nothing (the paper is silent on
 * them; this is the reading the library documents).
 *
 * Parity pins (tests marked "not gpu"): brute-force per-element sums, the
 * column-sum invariant, exact small-integer inputs, all-unique / all-same
 * closed forms, linearity, empty-slice idempotence, library scatter-add.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    const void* indices; /* int32 or int64, n_rows entries */
    const void* values;  /* float or bf16 bits (uint16), n_rows * d entries, row-major */
    int64_t n_rows;
} oracle_slice_t;

/* bfloat16 is the top half of an IEEE binary32: widening is exact. */
static double bf16_bits_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* One correctly rounded (nearest, ties to even) conversion fp64 -> bf16,
 * without passing through fp32 (which would round twice). */
static uint16_t double_to_bf16_bits(double x) {
    uint32_t u;
    float f;
    if (isnan(x)) return 0x7FC0u;
    if (x == 0.0 || isinf(x)) {
        f = (float)x;
    } else {
        int e = ilogb(x);
        if (e < -126) e = -126;          /* subnormal range: fixed spacing */
        double ulp = ldexp(1.0, e - 7);  /* bf16 keeps 8 significant bits */
        double q = rint(x / ulp);        /* default rounding mode: ties to even */
        double r = q * ulp;
        if (fabs(r) >= ldexp(1.0, 128)) r = (x > 0) ? INFINITY : -INFINITY;
        f = (float)r;                    /* exact: r is a bf16 number */
    }
    memcpy(&u, &f, sizeof u);
    return (uint16_t)(u >> 16);
}

/*
 * index_is_i64 : 1 = int64 indices, 0 = int32
 * value_is_bf16: 1 = values are bf16 bit patterns, 0 = float
 * out_is_bf16  : dtype of dense_in (if given) and of out_rounded
 * acc, mag     : [vocab*d] doubles (caller-allocated); acc is the unrounded result
 * out_rounded  : [vocab*d] in the output dtype, may be NULL
 * cnt          : [vocab] int64, may be NULL
 * returns 0, or -1 on a bad argument.
 */
int dst_oracle_densify(const oracle_slice_t* slices, int32_t R, int index_is_i64, int value_is_bf16,
                       int out_is_bf16, int64_t d, int64_t vocab, const void* dense_in,
                       double* acc, double* mag, void* out_rounded, int64_t* cnt, int64_t* n_bad) {
    if (R < 0 || d < 0 || vocab < 0 || (R > 0 && !slices) || !acc || !mag) return -1;
    const int64_t total = vocab * d;
    int64_t bad = 0;

    /* Start from the dense partner: the projection-matrix gradient that shares
     * the weight with the embedding (Section 3). */
    for (int64_t k = 0; k < total; ++k) {
        double x = 0.0;
        if (dense_in) {
            x = out_is_bf16 ? bf16_bits_to_double(((const uint16_t*)dense_in)[k])
                            : (double)((const float*)dense_in)[k];
        }
        acc[k] = x;
        mag[k] = fabs(x);
    }
    if (cnt) memset(cnt, 0, (size_t)vocab * sizeof(int64_t));

    /* Scatter-sum every row of every slice, in the order given. */
    for (int32_t r = 0; r < R; ++r) {
        const oracle_slice_t* s = &slices[r];
        if (s->n_rows < 0) return -1;
        for (int64_t i = 0; i < s->n_rows; ++i) {
            int64_t v = index_is_i64 ? ((const int64_t*)s->indices)[i]
                                     : (int64_t)((const int32_t*)s->indices)[i];
            if (v < 0 || v >= vocab) { ++bad; continue; }
            if (cnt) cnt[v] += 1;
            double* a = acc + v * d;
            double* m = mag + v * d;
            if (value_is_bf16) {
                const uint16_t* row = (const uint16_t*)s->values + i * d;
                for (int64_t c = 0; c < d; ++c) {
                    double x = bf16_bits_to_double(row[c]);
                    a[c] += x;
                    m[c] += fabs(x);
                }
            } else {
                const float* row = (const float*)s->values + i * d;
                for (int64_t c = 0; c < d; ++c) {
                    double x = (double)row[c];
                    a[c] += x;
                    m[c] += fabs(x);
                }
            }
        }
    }

    /* Round once to the output dtype. */
    if (out_rounded) {
        if (out_is_bf16) {
            uint16_t* o = (uint16_t*)out_rounded;
            for (int64_t k = 0; k < total; ++k) o[k] = double_to_bf16_bits(acc[k]);
        } else {
            float* o = (float*)out_rounded;
            for (int64_t k = 0; k < total; ++k) o[k] = (float)acc[k];
        }
    }
    if (n_bad) *n_bad = bad;
    return 0;
}

/* Exposed so a test can pin the rounding helper against an independent rounding. */
uint16_t dst_oracle_round_bf16(double x) { return double_to_bf16_bits(x); }
double dst_oracle_widen_bf16(uint16_t b) { return bf16_bits_to_double(b); }
