/*
 * gbs_oracle.c -- float64 CPU oracle for the rotate-and-quantize path of
 * "Gradual Binary Search and Dimension Expansion" (arXiv 2504.13989).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow,
 * by-the-definition restatement of what the path computes, written from the
 * paper, in double precision, sharing no code, header, table or constant with
 * the CUDA library.  Only the test-suite, the smoke check and the
 * cpu-baseline / reference leg of the benchmark may call it.
 *
 * What follows which passage of the paper
 *   - symmetric uniform quantizer  round(X/Delta)*Delta, Delta from max|X|
 *     and the bit-width ............................. Section 2.1 (Quantization)
 *   - per-token granularity ......................... Section 2.1
 *   - clipping ratio alpha (range shrunk to alpha*max) Section 3.1
 *   - Sylvester recursion H_2, H_4, H_{2^{n+1}} ..... Eq. (1) ("hadamard")
 *   - 1/sqrt(n) normalisation, H H^T = n I .......... Appendix A, proof of Lemma 1
 *   - Legendre symbol ............................... Section 2.3.3 (Paley algorithm)
 *   - Paley construction ............................ Algorithm 2
 *   - zero-pad dimension expansion .................. Section 4.2, Eq. (2) ("expand")
 *   - y = H x (column-vector convention) ............ Theorem 1 / Lemma 1
 *
 * Readings taken where the paper is silent or inconsistent:
 *   R1  levels: default D = 2^(b-1)-1, codes in [-D, D] (fits b bits);
 *       "literal" mode D = 2^b-1 is the formula exactly as printed.
 *   R2  clamp to [-D, D] when alpha < 1.
 *   R3  round = round-half-to-even.
 *   R4  Delta = alpha * max|y| / D.
 *   R5  an all-zero row/group gives codes 0 and Delta 0.
 *   R6  Legendre argument reduced into [0,p) first.
 *   R7  order 28 uses GF(27) = GF(3)[x]/(x^3+2x+1), element index
 *       e = c0 + 3 c1 + 9 c2, chi = quadratic character of the field.
 *   R8  composite order d' = m 2^k : H = H_m (x) H_{2^k}, flat index a*2^k + c.
 *   R9  padding zeros are appended at the tail (columns d .. d'-1).
 *   R10 packing: element j takes bits [j*b, (j+1)*b) of a little-endian
 *       bit-stream holding the low b bits of the two's-complement code.
 *       PARITY UNPINNED by the paper (it never packs); pinned only by a
 *       round trip and a hand-packed example.
 *
 * Every other function is pinned by tests that run without a GPU
 * (tests/test_oracle_pins.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_F32 0
#define ORACLE_BF16 1

/* ------------------------------------------------------------------ */
/* Legendre symbol, straight from the definition (Section 2.3.3):      */
/* +1 if some x has x^2 = a (mod p), a != 0; -1 if none; 0 if p | a.   */
/* ------------------------------------------------------------------ */
int oracle_legendre(long a, int p)
{
    long r = a % p;
    if (r < 0) r += p;               /* reading R6 */
    if (r == 0) return 0;
    for (long x = 1; x < p; ++x)
        if ((x * x) % p == r) return 1;
    return -1;
}

/* GF(27) arithmetic on indices e = c0 + 3 c1 + 9 c2 (reading R7). */
static void gf27_split(int e, int c[3]) { c[0] = e % 3; c[1] = (e / 3) % 3; c[2] = e / 9; }
static int gf27_join(const int c[3]) { return c[0] + 3 * c[1] + 9 * c[2]; }

int oracle_gf27_sub(int e, int f)
{
    int a[3], b[3], r[3];
    gf27_split(e, a); gf27_split(f, b);
    for (int i = 0; i < 3; ++i) r[i] = ((a[i] - b[i]) % 3 + 3) % 3;
    return gf27_join(r);
}

int oracle_gf27_mul(int e, int f)
{
    int a[3], b[3], t[5] = {0, 0, 0, 0, 0}, r[3];
    gf27_split(e, a); gf27_split(f, b);
    for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 3; ++j) t[i + j] += a[i] * b[j];
    /* x^3 = -2x - 1 = x + 2 (mod 3);  x^4 = x^2 + 2x */
    /* fold degree 4 then degree 3 */
    t[2] += t[4]; t[1] += 2 * t[4]; t[4] = 0;
    t[1] += t[3]; t[0] += 2 * t[3]; t[3] = 0;
    for (int i = 0; i < 3; ++i) r[i] = t[i] % 3;
    return gf27_join(r);
}

/* quadratic character of GF(27) by exhaustive squaring */
int oracle_gf27_chi(int e)
{
    if (e == 0) return 0;
    for (int x = 1; x < 27; ++x)
        if (oracle_gf27_mul(x, x) == e) return 1;
    return -1;
}

/* ------------------------------------------------------------------ */
/* H_m: m = 1 -> [1];  m = 28 -> Algorithm 2 over GF(27);              */
/* otherwise Algorithm 2 with p = m-1 prime, p = 3 (mod 4).            */
/* H is row-major m x m, entries +1/-1.  Returns 0, or -1 if no        */
/* construction applies.                                               */
/* ------------------------------------------------------------------ */
static int is_prime(int p)
{
    if (p < 2) return 0;
    for (int q = 2; q * q <= p; ++q) if (p % q == 0) return 0;
    return 1;
}

int oracle_hadamard_m(int m, int8_t *H)
{
    if (m == 1) { H[0] = 1; return 0; }
    int field27 = (m == 28);
    int p = m - 1;
    if (!field27 && !(is_prime(p) && p % 4 == 3)) return -1;
    /* Algorithm 2: all ones; first row/column and diagonal -1 (i >= 1);
       elsewhere the character of (i-1) - (j-1). */
    for (int i = 0; i < m * m; ++i) H[i] = 1;
    for (int i = 1; i < m; ++i) {
        H[i * m + 0] = -1;
        H[0 * m + i] = -1;
        for (int j = 1; j < m; ++j) {
            if (i == j) H[i * m + j] = -1;
            else if (field27) H[i * m + j] = (int8_t)oracle_gf27_chi(oracle_gf27_sub(i - 1, j - 1));
            else H[i * m + j] = (int8_t)oracle_legendre((long)(i - 1) - (long)(j - 1), p);
        }
    }
    return 0;
}

/* Sylvester matrix by the recursion of Eq. (1): H_1=[1], H_{2n}=[[H,H],[H,-H]]. */
int oracle_sylvester(int n, int8_t *H)
{
    if (n < 1 || (n & (n - 1))) return -1;
    H[0] = 1;
    for (int s = 1; s < n; s *= 2) {
        /* grow the s x s block held in the top-left corner (row stride n) */
        for (int i = 0; i < s; ++i)
            for (int j = 0; j < s; ++j) {
                int8_t v = H[i * n + j];
                H[i * n + (j + s)] = v;
                H[(i + s) * n + j] = v;
                H[(i + s) * n + (j + s)] = (int8_t)-v;
            }
    }
    return 0;
}

static int parity_and(unsigned a, unsigned b)
{
    unsigned v = a & b; int par = 0;
    while (v) { par ^= 1; v &= v - 1; }
    return par;
}

static int log2_exact(long n)
{
    int k = 0;
    if (n < 1) return -1;
    while ((1L << k) < n) ++k;
    return ((1L << k) == n) ? k : -1;
}

/* ------------------------------------------------------------------ */
/* Rotation by the definition: y = H_{d'} x_pad / sqrt(d'),            */
/* H_{d'}[(a,c),(a',c')] = H_m[a,a'] * (-1)^{popcount(c & c')}.        */
/* x has d entries; entries d..d'-1 are zero.  O(d'^2).                */
/* transpose != 0 applies H^T instead (the inverse rotation).          */
/* ------------------------------------------------------------------ */
int oracle_rotate_dense(const double *x, int d, int d_pad, int m, int transpose, double *y)
{
    if (m < 1 || d_pad % m) return -1;
    int n2 = d_pad / m, k = log2_exact(n2);
    if (k < 0 || d < 0 || d > d_pad) return -1;
    int8_t *Hm = (int8_t *)malloc((size_t)m * m);
    if (!Hm) return -2;
    if (oracle_hadamard_m(m, Hm)) { free(Hm); return -1; }
    double norm = 1.0 / sqrt((double)d_pad);
    for (int i = 0; i < d_pad; ++i) {
        int a = i / n2, c = i % n2;
        double acc = 0.0;
        for (int j = 0; j < d; ++j) {
            int a2 = j / n2, c2 = j % n2;
            int hm = transpose ? Hm[a2 * m + a] : Hm[a * m + a2];
            int s = parity_and((unsigned)c, (unsigned)c2) ? -hm : hm;
            acc += s * x[j];
        }
        y[i] = acc * norm;
    }
    free(Hm);
    return 0;
}

/* Same result through the fast transform the paper refers to ("FHT"):  */
/* the recursion of Eq. (1) unrolled into butterflies inside each block */
/* of 2^k, then the m x m mix across blocks.  Checked against the dense */
/* definition in the tests; used where O(d'^2) per row is too slow.     */
static int rotate_fast_with(const int8_t *Hm, const double *x, int d, int d_pad, int m,
                            int transpose, double *y, double *tmp)
{
    int n2 = d_pad / m;
    for (int j = 0; j < d; ++j) y[j] = x[j];
    for (int j = d; j < d_pad; ++j) y[j] = 0.0;
    for (int a = 0; a < m; ++a) {
        double *blk = y + (size_t)a * n2;
        for (int h = 1; h < n2; h *= 2)
            for (int base = 0; base < n2; base += 2 * h)
                for (int j = base; j < base + h; ++j) {
                    double u = blk[j], v = blk[j + h];
                    blk[j] = u + v; blk[j + h] = u - v;
                }
    }
    double norm = 1.0 / sqrt((double)d_pad);
    if (m == 1) {
        for (int j = 0; j < d_pad; ++j) y[j] *= norm;
        return 0;
    }
    for (int c = 0; c < n2; ++c) {
        for (int a = 0; a < m; ++a) {
            double acc = 0.0;
            for (int a2 = 0; a2 < m; ++a2) {
                int hm = transpose ? Hm[a2 * m + a] : Hm[a * m + a2];
                acc += hm * y[(size_t)a2 * n2 + c];
            }
            tmp[a] = acc;
        }
        for (int a = 0; a < m; ++a) y[(size_t)a * n2 + c] = tmp[a] * norm;
    }
    return 0;
}

int oracle_rotate_fast(const double *x, int d, int d_pad, int m, int transpose, double *y)
{
    if (m < 1 || d_pad % m) return -1;
    int n2 = d_pad / m;
    if (log2_exact(n2) < 0 || d < 0 || d > d_pad) return -1;
    int8_t *Hm = (int8_t *)malloc((size_t)m * m);
    double *tmp = (double *)malloc(sizeof(double) * (size_t)m);
    if (!Hm || !tmp) { free(Hm); free(tmp); return -2; }
    int rc = oracle_hadamard_m(m, Hm);
    if (!rc) rc = rotate_fast_with(Hm, x, d, d_pad, m, transpose, y, tmp);
    free(Hm); free(tmp);
    return rc;
}

/* ------------------------------------------------------------------ */
/* Quantizer (Section 2.1 with the clip ratio of Section 3.1).         */
/* group == 0: one Delta for the n values; else one per `group`        */
/* consecutive values.  literal != 0 uses D = 2^b - 1 (formula as      */
/* printed); default D = 2^(b-1) - 1.                                  */
/* q[j] integer codes, delta[g] scaling factors.                       */
/* ------------------------------------------------------------------ */
int oracle_levels(int bits, int literal)
{
    return literal ? ((1 << bits) - 1) : ((1 << (bits - 1)) - 1);
}

int oracle_quantize(const double *y, int n, int bits, int group, double alpha, int literal,
                    int32_t *q, double *delta)
{
    if (bits < 2 || bits > 8 || n < 1) return -1;
    int g = group ? group : n;
    if (n % g) return -1;
    double D = (double)oracle_levels(bits, literal);
    for (int s = 0; s < n / g; ++s) {
        const double *v = y + (size_t)s * g;
        double M = 0.0;
        for (int j = 0; j < g; ++j) { double a = fabs(v[j]); if (a > M) M = a; }
        double dl = alpha * M / D;                       /* reading R4 */
        delta[s] = dl;
        for (int j = 0; j < g; ++j) {
            double r = 0.0;
            if (dl > 0.0) {                              /* reading R5 */
                r = rint(v[j] / dl);                     /* half-to-even, R3 */
                if (r > D) r = D;                        /* R2 */
                if (r < -D) r = -D;
            }
            q[(size_t)s * g + j] = (int32_t)r;
        }
    }
    return 0;
}

/* Sum over the n values of (y - q*Delta)^2 for one clip ratio. */
double oracle_clip_error(const double *y, int n, int bits, int group, double alpha, int literal)
{
    int g = group ? group : n;
    double D = (double)oracle_levels(bits, literal), err = 0.0;
    for (int s = 0; s < n / g; ++s) {
        const double *v = y + (size_t)s * g;
        double M = 0.0;
        for (int j = 0; j < g; ++j) { double a = fabs(v[j]); if (a > M) M = a; }
        double dl = alpha * M / D;
        for (int j = 0; j < g; ++j) {
            double r = 0.0;
            if (dl > 0.0) {
                r = rint(v[j] / dl);
                if (r > D) r = D;
                if (r < -D) r = -D;
            }
            double e = v[j] - r * dl;
            err += e * e;
        }
    }
    return err;
}

/* Packing (reading R10). out must hold ceil(n*bits/8) bytes. */
void oracle_pack(const int32_t *q, long n, int bits, uint8_t *out)
{
    long nbytes = (n * bits + 7) / 8;
    memset(out, 0, (size_t)nbytes);
    uint32_t mask = (1u << bits) - 1u;
    for (long j = 0; j < n; ++j) {
        uint32_t f = ((uint32_t)q[j]) & mask;
        for (int t = 0; t < bits; ++t) {
            long bit = j * bits + t;
            if ((f >> t) & 1u) out[bit >> 3] |= (uint8_t)(1u << (bit & 7));
        }
    }
}

void oracle_unpack(const uint8_t *in, long n, int bits, int32_t *q)
{
    for (long j = 0; j < n; ++j) {
        uint32_t f = 0;
        for (int t = 0; t < bits; ++t) {
            long bit = j * bits + t;
            if ((in[bit >> 3] >> (bit & 7)) & 1u) f |= (1u << t);
        }
        if (f & (1u << (bits - 1))) f |= ~((1u << bits) - 1u);   /* sign-extend */
        q[j] = (int32_t)f;
    }
}

/* ------------------------------------------------------------------ */
/* Row-batched drivers (OpenMP over rows).                              */
/* ------------------------------------------------------------------ */
static double load_elem(const void *x, int dtype, size_t idx)
{
    if (dtype == ORACLE_F32) return (double)((const float *)x)[idx];
    uint32_t bits = ((uint32_t)((const uint16_t *)x)[idx]) << 16;   /* bf16 -> f32, exact */
    float f; memcpy(&f, &bits, 4);
    return (double)f;
}

/*
 * For each of n_rows rows (row r starts at element r*stride of x):
 * pad, rotate, quantize, pack.  Any output pointer may be NULL.
 *   y_out   [n_rows, d_pad]  rotated, normalised values
 *   q_out   [n_rows, d_pad]  integer codes
 *   packed  [n_rows, d_pad*bits/8] packed bytes
 *   delta   [n_rows, spr]    scaling factors, spr = group ? d_pad/group : 1
 * dense != 0 rotates by the O(d'^2) definition, else by the butterflies.
 */
int oracle_rotate_quantize_rows(const void *x, int dtype, long n_rows, long stride,
                                int d, int d_pad, int m, int bits, int group, double alpha,
                                int literal, int dense,
                                double *y_out, int32_t *q_out, uint8_t *packed, double *delta,
                                int nthreads)
{
    if (m < 1 || d_pad % m || log2_exact(d_pad / m) < 0 || d < 1 || d > d_pad) return -1;
    if (group && d_pad % group) return -1;
    int8_t *Hm = (int8_t *)malloc((size_t)m * m);
    if (!Hm) return -2;
    if (oracle_hadamard_m(m, Hm)) { free(Hm); return -1; }
    int spr = group ? d_pad / group : 1;
    long row_bytes = ((long)d_pad * bits) / 8;
    int fail = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#pragma omp parallel
#endif
    {
        double *xr = (double *)malloc(sizeof(double) * (size_t)d_pad);
        double *yr = (double *)malloc(sizeof(double) * (size_t)d_pad);
        double *tmp = (double *)malloc(sizeof(double) * (size_t)m);
        int32_t *qr = (int32_t *)malloc(sizeof(int32_t) * (size_t)d_pad);
        double *dl = (double *)malloc(sizeof(double) * (size_t)spr);
        if (!xr || !yr || !tmp || !qr || !dl) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            fail = 1;
        } else {
#ifdef _OPENMP
#pragma omp for schedule(static)
#endif
            for (long r = 0; r < n_rows; ++r) {
                for (int j = 0; j < d; ++j) xr[j] = load_elem(x, dtype, (size_t)r * stride + j);
                if (dense) oracle_rotate_dense(xr, d, d_pad, m, 0, yr);
                else rotate_fast_with(Hm, xr, d, d_pad, m, 0, yr, tmp);
                oracle_quantize(yr, d_pad, bits, group, alpha, literal, qr, dl);
                if (y_out) memcpy(y_out + (size_t)r * d_pad, yr, sizeof(double) * (size_t)d_pad);
                if (q_out) memcpy(q_out + (size_t)r * d_pad, qr, sizeof(int32_t) * (size_t)d_pad);
                if (packed) oracle_pack(qr, d_pad, bits, packed + (size_t)r * row_bytes);
                if (delta) memcpy(delta + (size_t)r * spr, dl, sizeof(double) * (size_t)spr);
            }
        }
        free(xr); free(yr); free(tmp); free(qr); free(dl);
    }
    free(Hm);
    return fail ? -2 : 0;
}

/*
 * Clip-ratio scoring: for each alpha_k, E_k = sum over rows and coordinates of
 * (y - yhat_k)^2 where yhat_k is the quantizer output under alpha_k.
 *   err_sum  [K]          totals (overwritten)
 *   err_rows [n_rows, K]  per-row sums, or NULL
 */
int oracle_clip_error_rows(const void *x, int dtype, long n_rows, long stride,
                           int d, int d_pad, int m, int bits, int group, int literal,
                           const double *alphas, int K, double *err_sum, double *err_rows,
                           int nthreads)
{
    if (m < 1 || d_pad % m || log2_exact(d_pad / m) < 0 || d < 1 || d > d_pad || K < 1) return -1;
    if (group && d_pad % group) return -1;
    int8_t *Hm = (int8_t *)malloc((size_t)m * m);
    double *rows = (double *)malloc(sizeof(double) * (size_t)n_rows * K);
    if (!Hm || !rows) { free(Hm); free(rows); return -2; }
    if (oracle_hadamard_m(m, Hm)) { free(Hm); free(rows); return -1; }
    int fail = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#pragma omp parallel
#endif
    {
        double *xr = (double *)malloc(sizeof(double) * (size_t)d_pad);
        double *yr = (double *)malloc(sizeof(double) * (size_t)d_pad);
        double *tmp = (double *)malloc(sizeof(double) * (size_t)m);
        if (!xr || !yr || !tmp) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            fail = 1;
        } else {
#ifdef _OPENMP
#pragma omp for schedule(static)
#endif
            for (long r = 0; r < n_rows; ++r) {
                for (int j = 0; j < d; ++j) xr[j] = load_elem(x, dtype, (size_t)r * stride + j);
                rotate_fast_with(Hm, xr, d, d_pad, m, 0, yr, tmp);
                for (int k = 0; k < K; ++k)
                    rows[(size_t)r * K + k] = oracle_clip_error(yr, d_pad, bits, group, alphas[k], literal);
            }
        }
        free(xr); free(yr); free(tmp);
    }
    if (!fail) {
        for (int k = 0; k < K; ++k) {
            double s = 0.0;
            for (long r = 0; r < n_rows; ++r) s += rows[(size_t)r * K + k];
            err_sum[k] = s;
        }
        if (err_rows) memcpy(err_rows, rows, sizeof(double) * (size_t)n_rows * K);
    }
    free(Hm); free(rows);
    return fail ? -2 : 0;
}

/*
 * Dequantize: yhat = q * Delta in the rotated domain (width d_pad); with
 * inverse != 0 additionally xhat = (H^T yhat / sqrt(d'))[0:d].
 * out is [n_rows, inverse ? d : d_pad].
 */
int oracle_dequantize_rows(const uint8_t *packed, const double *delta, long n_rows,
                           int d, int d_pad, int m, int bits, int group, int inverse,
                           double *out, int nthreads)
{
    if (m < 1 || d_pad % m || log2_exact(d_pad / m) < 0 || d < 1 || d > d_pad) return -1;
    if (group && d_pad % group) return -1;
    int8_t *Hm = (int8_t *)malloc((size_t)m * m);
    if (!Hm) return -2;
    if (oracle_hadamard_m(m, Hm)) { free(Hm); return -1; }
    int spr = group ? d_pad / group : 1, g = group ? group : d_pad;
    long row_bytes = ((long)d_pad * bits) / 8;
    int fail = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#pragma omp parallel
#endif
    {
        int32_t *qr = (int32_t *)malloc(sizeof(int32_t) * (size_t)d_pad);
        double *yh = (double *)malloc(sizeof(double) * (size_t)d_pad);
        double *xh = (double *)malloc(sizeof(double) * (size_t)d_pad);
        double *tmp = (double *)malloc(sizeof(double) * (size_t)m);
        if (!qr || !yh || !xh || !tmp) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            fail = 1;
        } else {
#ifdef _OPENMP
#pragma omp for schedule(static)
#endif
            for (long r = 0; r < n_rows; ++r) {
                oracle_unpack(packed + (size_t)r * row_bytes, d_pad, bits, qr);
                for (int j = 0; j < d_pad; ++j) yh[j] = qr[j] * delta[(size_t)r * spr + j / g];
                if (!inverse) {
                    memcpy(out + (size_t)r * d_pad, yh, sizeof(double) * (size_t)d_pad);
                } else {
                    rotate_fast_with(Hm, yh, d_pad, d_pad, m, 1, xh, tmp);
                    memcpy(out + (size_t)r * d, xh, sizeof(double) * (size_t)d);
                }
            }
        }
        free(qr); free(yh); free(xh); free(tmp);
    }
    free(Hm);
    return fail ? -2 : 0;
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
