/*
 * CPU oracle for segmented scan / segmented sum / CSR SpMV.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, sequential, obviously
 * correct statement of what the GPU library must compute.  It shares no code
 * with the CUDA path and must never be called from it: only the test-suite,
 * the smoke check and the "cpu_baseline"/"reference" legs of the benchmark may
 * load it.
 *
 * Every function is the *definition* written out (the method reaches the plain
 * result exactly for integers and up to rounding for floats), so there is no
 * blocking, no speculation and no tile structure here.
 *
 *   - Segmented scan:  Problem 2.1 / Eq. (1) of the paper:
 *         z(i) = x(i)            if i == 0 or f(i) != 0
 *         z(i) = z(i-1) + x(i)   otherwise
 *   - Segmented sum:   Section 2 (text after Problem 2.1): the last element of
 *         each segment of the segmented-scanned array, in segment order.
 *   - CSR form:        Section 4.3 (remark after Algorithm 4.4): the segment
 *         description may be an integer vector of segment start indices; here
 *         the usual CSR row-pointer array off[0..S] (start of segment r is
 *         off[r], one past its end is off[r+1]); an empty segment sums to 0
 *         (Appendix, Algorithm A.4 and A.6 handle empty rows that way).
 *   - CSR SpMV:        Algorithm 4.4 / Algorithm A.5:  z(k) = val(k) * x(col(k)),
 *         then the segmented sum of z over the rows.
 *
 * Arithmetic: integer paths accumulate in int64 and return the low 32 bits
 * (two's-complement wrap); floating-point paths decode fp16 exactly to double
 * and accumulate sequentially in double.  Next to every fp result the oracle
 * returns a(i) = sum of |x| over the same range, which the error bound
 * |gpu - z| <= 2e-3 * a + 1e-6 needs.
 *
 * Readings of the paper taken here (each is also listed in the design notes):
 *   - f(0) is never consulted: index 0 always opens a segment.
 *   - any non-zero flag byte marks a segment start.
 *   - the scan is inclusive.
 *
 * Parity pins: every function below is pinned by the CPU test-suite against
 * the paper's worked example, closed forms, brute force and library routines;
 * none is "parity unpinned".
 */
#include <stdint.h>
#include <stddef.h>
#include <math.h>

/* Exact decode of an IEEE-754 binary16 bit pattern to double. */
static double half_bits_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int m = h & 0x3ff;
    double v;
    if (e == 0) {
        v = ldexp((double)m, -24);              /* zero and subnormals: m * 2^-24 */
    } else if (e == 31) {
        v = m ? NAN : INFINITY;
    } else {
        v = ldexp((double)(m + 1024), e - 25);  /* (1 + m/1024) * 2^(e-15) */
    }
    return sign ? -v : v;
}

double mmv_oracle_half_to_double(uint16_t h) { return half_bits_to_double(h); }

/* ------------------------------------------------------------------------ */
/* Segmented inclusive scan, Eq. (1).                                        */
/* ------------------------------------------------------------------------ */

/*
 * fp16 values (bit patterns), uint8 flags.  z[i] is the scan in double, a[i]
 * the running sum of |x| inside the segment.  state[0..1] = (z, a) of the
 * element just before x[0] when this call continues an earlier chunk
 * (has_prev != 0); on return state holds (z, a) of the last element, so a
 * long array can be streamed chunk by chunk.  With has_prev == 0 this is
 * exactly Eq. (1).
 */
void mmv_oracle_seg_scan_f16(const uint16_t *x, const uint8_t *f, int64_t n,
                             double *z, double *a, int has_prev, double *state)
{
    double zp = 0.0, ap = 0.0;
    int open = 0;                       /* is there a z(i-1) to continue from? */
    if (has_prev && state) { zp = state[0]; ap = state[1]; open = 1; }
    for (int64_t i = 0; i < n; ++i) {
        double xi = half_bits_to_double(x[i]);
        if (!open || f[i] != 0) { zp = xi; ap = fabs(xi); }
        else                    { zp = zp + xi; ap = ap + fabs(xi); }
        open = 1;
        z[i] = zp;
        if (a) a[i] = ap;
    }
    if (state) { state[0] = zp; state[1] = ap; }
}

/* int8 values, int32 result with two's-complement wrap (int64 accumulate). */
void mmv_oracle_seg_scan_i8(const int8_t *x, const uint8_t *f, int64_t n,
                            int32_t *z, int has_prev, int64_t *state)
{
    int64_t zp = 0;
    int open = 0;
    if (has_prev && state) { zp = state[0]; open = 1; }
    for (int64_t i = 0; i < n; ++i) {
        if (!open || f[i] != 0) zp = (int64_t)x[i];
        else                    zp = zp + (int64_t)x[i];
        open = 1;
        z[i] = (int32_t)(uint32_t)(uint64_t)zp;     /* low 32 bits */
    }
    if (state) state[0] = zp;
}

/* int8 values, int64 result: Eq. (1) without any wrap (|z| <= 128 n). */
void mmv_oracle_seg_scan_i8_wide(const int8_t *x, const uint8_t *f, int64_t n, int64_t *z)
{
    int64_t zp = 0;
    for (int64_t i = 0; i < n; ++i) {
        if (i == 0 || f[i] != 0) zp = (int64_t)x[i];
        else                     zp = zp + (int64_t)x[i];
        z[i] = zp;
    }
}

/*
 * Segmented EXCLUSIVE scan: e(i) = 0 if i = 0 or f(i) != 0, else z(i-1) with z the
 * scan of Eq. (1); that is, the sum of the elements of i's segment in front of
 * i.  a[i] is the sum of |x| over the same elements.  (The paper states the
 * inclusive problem only; this is the usual companion definition.)
 */
void mmv_oracle_seg_scan_excl_f16(const uint16_t *x, const uint8_t *f, int64_t n, double *e, double *a)
{
    double run = 0.0, arun = 0.0;       /* sum of the open segment so far */
    for (int64_t i = 0; i < n; ++i) {
        double xi = half_bits_to_double(x[i]);
        if (i == 0 || f[i] != 0) { run = 0.0; arun = 0.0; }
        e[i] = run;
        if (a) a[i] = arun;
        run = run + xi;
        arun = arun + fabs(xi);
    }
}

void mmv_oracle_seg_scan_excl_i8(const int8_t *x, const uint8_t *f, int64_t n, int32_t *e)
{
    int64_t run = 0;
    for (int64_t i = 0; i < n; ++i) {
        if (i == 0 || f[i] != 0) run = 0;
        e[i] = (int32_t)(uint32_t)(uint64_t)run;     /* low 32 bits */
        run = run + (int64_t)x[i];
    }
}

/*
 * Start flags from CSR offsets: f(i) = 1 iff i is the start index off[r] of a
 * non-empty segment r.  Returns 0, or -1 if the offsets are not a
 * non-decreasing sequence from 0 to n.
 */
int mmv_oracle_flags_from_offsets(const int32_t *off, int64_t nseg, int64_t n, uint8_t *f)
{
    for (int64_t i = 0; i < n; ++i) f[i] = 0;
    if (nseg < 0) return -1;
    if (nseg == 0) return n == 0 ? 0 : -1;
    if (off[0] != 0 || off[nseg] != n) return -1;
    for (int64_t r = 0; r < nseg; ++r) {
        if (off[r] > off[r + 1]) return -1;
        if (off[r] < off[r + 1]) f[off[r]] = 1;
    }
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Segmented sum.                                                            */
/* ------------------------------------------------------------------------ */

/*
 * Flag form: out[k] = z(e_k), e_k the last index of the k-th segment, where z
 * is the segmented scan.  Returns the number of segments K
 * (1 + #{i >= 1 : f(i) != 0}, or 0 when n == 0).  out/a need capacity K <= n.
 */
int64_t mmv_oracle_seg_sum_flags_f16(const uint16_t *x, const uint8_t *f, int64_t n,
                                     double *out, double *a)
{
    int64_t k = 0;
    double zp = 0.0, ap = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double xi = half_bits_to_double(x[i]);
        if (i == 0 || f[i] != 0) { zp = xi; ap = fabs(xi); }
        else                     { zp += xi; ap += fabs(xi); }
        if (i == n - 1 || f[i + 1] != 0) {      /* i closes its segment */
            out[k] = zp;
            if (a) a[k] = ap;
            ++k;
        }
    }
    return k;
}

int64_t mmv_oracle_seg_sum_flags_i8(const int8_t *x, const uint8_t *f, int64_t n, int32_t *out)
{
    int64_t k = 0, zp = 0;
    for (int64_t i = 0; i < n; ++i) {
        if (i == 0 || f[i] != 0) zp = (int64_t)x[i];
        else                     zp += (int64_t)x[i];
        if (i == n - 1 || f[i + 1] != 0) out[k++] = (int32_t)(uint32_t)(uint64_t)zp;
    }
    return k;
}

/*
 * CSR form: out[r] = sum of x over [off[r], off[r+1]), 0 for an empty range.
 * Elements outside [off[0], off[nseg]) belong to no segment.
 */
void mmv_oracle_seg_sum_csr_f16(const uint16_t *x, const int32_t *off, int64_t nseg,
                                double *out, double *a)
{
    for (int64_t r = 0; r < nseg; ++r) {
        double s = 0.0, sa = 0.0;
        for (int64_t i = off[r]; i < off[r + 1]; ++i) {
            double xi = half_bits_to_double(x[i]);
            s += xi;
            sa += fabs(xi);
        }
        out[r] = s;
        if (a) a[r] = sa;
    }
}

void mmv_oracle_seg_sum_csr_i8(const int8_t *x, const int32_t *off, int64_t nseg, int32_t *out)
{
    for (int64_t r = 0; r < nseg; ++r) {
        int64_t s = 0;
        for (int64_t i = off[r]; i < off[r + 1]; ++i) s += (int64_t)x[i];
        out[r] = (int32_t)(uint32_t)(uint64_t)s;
    }
}

/* ------------------------------------------------------------------------ */
/* Segmented running maximum / minimum: Eq. (1) with max or min in place of   */
/* the addition (an operator without an inverse: Section 2 notes that the     */
/* speculate-and-revert method needs a group, so this is the plain recurrence).*/
/* want_min = 0: maximum, 1: minimum.                                         */
/* ------------------------------------------------------------------------ */
void mmv_oracle_seg_scan_minmax_f16(const uint16_t *x, const uint8_t *f, int64_t n, int want_min, double *z)
{
    double zp = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double xi = half_bits_to_double(x[i]);
        if (i == 0 || f[i] != 0) zp = xi;
        else if (want_min ? (xi < zp) : (xi > zp)) zp = xi;
        z[i] = zp;
    }
}

/* The same on values given as doubles (bfloat16 inputs are decoded first). */
void mmv_oracle_seg_scan_minmax_f64(const double *x, const uint8_t *f, int64_t n, int want_min, double *z)
{
    double zp = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        if (i == 0 || f[i] != 0) zp = x[i];
        else if (want_min ? (x[i] < zp) : (x[i] > zp)) zp = x[i];
        z[i] = zp;
    }
}

void mmv_oracle_seg_scan_minmax_i8(const int8_t *x, const uint8_t *f, int64_t n, int want_min, int32_t *z)
{
    int32_t zp = 0;
    for (int64_t i = 0; i < n; ++i) {
        int32_t xi = (int32_t)x[i];
        if (i == 0 || f[i] != 0) zp = xi;
        else if (want_min ? (xi < zp) : (xi > zp)) zp = xi;
        z[i] = zp;
    }
}

/* ------------------------------------------------------------------------ */
/* COMPRESS (Section 2): keep x(i) where f(i) != 0, in order.  Elements are   */
/* copied as they are (elem_bytes each); returns the number kept.             */
/* ------------------------------------------------------------------------ */
int64_t mmv_oracle_compress(const uint8_t *x, const uint8_t *f, int64_t n, int elem_bytes, uint8_t *out)
{
    int64_t k = 0;
    for (int64_t i = 0; i < n; ++i) {
        if (f[i] != 0) {
            for (int b = 0; b < elem_bytes; ++b) out[k * elem_bytes + b] = x[i * elem_bytes + b];
            ++k;
        }
    }
    return k;
}

/* ------------------------------------------------------------------------ */
/* bfloat16 values: decoded exactly to double, then the same definitions on   */
/* double inputs (Eq. (1), its exclusive companion, the two segmented sums).  */
/* ------------------------------------------------------------------------ */

/* Exact decode of a bfloat16 bit pattern (1 sign, 8 exponent, 7 mantissa bits). */
double mmv_oracle_bf16_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 7) & 0xff;
    int m = h & 0x7f;
    double v;
    if (e == 0) {
        v = ldexp((double)m, -133);             /* zero and subnormals: m * 2^-7 * 2^-126 */
    } else if (e == 255) {
        v = m ? NAN : INFINITY;
    } else {
        v = ldexp((double)(m + 128), e - 134);  /* (1 + m/128) * 2^(e-127) */
    }
    return sign ? -v : v;
}

void mmv_oracle_decode_bf16(const uint16_t *h, int64_t n, double *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = mmv_oracle_bf16_to_double(h[i]);
}

void mmv_oracle_seg_scan_f64(const double *x, const uint8_t *f, int64_t n, double *z, double *a)
{
    double zp = 0.0, ap = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        if (i == 0 || f[i] != 0) { zp = x[i]; ap = fabs(x[i]); }
        else                     { zp = zp + x[i]; ap = ap + fabs(x[i]); }
        z[i] = zp;
        if (a) a[i] = ap;
    }
}

void mmv_oracle_seg_scan_excl_f64(const double *x, const uint8_t *f, int64_t n, double *e, double *a)
{
    double run = 0.0, arun = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        if (i == 0 || f[i] != 0) { run = 0.0; arun = 0.0; }
        e[i] = run;
        if (a) a[i] = arun;
        run = run + x[i];
        arun = arun + fabs(x[i]);
    }
}

int64_t mmv_oracle_seg_sum_flags_f64(const double *x, const uint8_t *f, int64_t n, double *out, double *a)
{
    int64_t k = 0;
    double zp = 0.0, ap = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        if (i == 0 || f[i] != 0) { zp = x[i]; ap = fabs(x[i]); }
        else                     { zp += x[i]; ap += fabs(x[i]); }
        if (i == n - 1 || f[i + 1] != 0) {
            out[k] = zp;
            if (a) a[k] = ap;
            ++k;
        }
    }
    return k;
}

void mmv_oracle_seg_sum_csr_f64(const double *x, const int32_t *off, int64_t nseg, double *out, double *a)
{
    for (int64_t r = 0; r < nseg; ++r) {
        double s = 0.0, sa = 0.0;
        for (int64_t i = off[r]; i < off[r + 1]; ++i) {
            s += x[i];
            sa += fabs(x[i]);
        }
        out[r] = s;
        if (a) a[r] = sa;
    }
}

/* ------------------------------------------------------------------------ */
/* CSR SpMV: y(r) = sum_k val(k) * x(col(k)) over the row's entries.          */
/* val is fp16 (bit patterns), x is fp32; both are decoded exactly to double */
/* so each product is exact in double; a(r) = sum |val(k) * x(col(k))|.       */
/* ------------------------------------------------------------------------ */
void mmv_oracle_spmv_csr(const int32_t *rowptr, const int32_t *col, const uint16_t *val,
                         const float *x, int64_t rows, double *y, double *a)
{
    for (int64_t r = 0; r < rows; ++r) {
        double s = 0.0, sa = 0.0;
        for (int64_t k = rowptr[r]; k < rowptr[r + 1]; ++k) {
            double t = half_bits_to_double(val[k]) * (double)x[col[k]];
            s += t;
            sa += fabs(t);
        }
        y[r] = s;
        if (a) a[r] = sa;
    }
}

/*
 * Element-wise product of two int8 vectors, int32 result (Section 4.3.1,
 * Corollary 4.5: z(i) = x(i) y(i)).  The paper obtains each product as the last
 * element of a segmented scan over the partial terms of the school method
 * (Lemma 4.4); the quantity itself is the plain product, which is what is
 * written here.  |x y| <= 2^14, so nothing wraps.
 */
void mmv_oracle_mult_i8(const int8_t *x, const int8_t *y, int64_t n, int32_t *z)
{
    for (int64_t i = 0; i < n; ++i) z[i] = (int32_t)x[i] * (int32_t)y[i];
}

