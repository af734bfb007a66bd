/*
 * PeRQ rotate+quantize -- CPU ORACLE.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 statement of what the online path computes, written from the
 * paper's definitions.  It exists so that tests (and the benchmark's CPU-baseline leg)
 * have something independent to compare the CUDA library against.  It shares no code
 * with the CUDA library, is never linked into it, and the product never calls it.
 *
 * Every function cites the passage it follows.  Inputs are bf16 bit patterns (uint16),
 * widened exactly to double; all arithmetic is double unless stated.
 *
 * Parity pins (see tests/test_oracle_*.py): every function here is pinned by closed
 * forms / invariants / brute force except the storage conventions the paper does not
 * fix -- "parity unpinned" for: nibble order inside a byte, the all-zero-range
 * convention (scale 0, codes 0), sign of values that quantise to zero in E2M1, the
 * MX shared-exponent reading floor(log2 amax) - 2 versus 2^floor(log2(amax/6)), and the
 * tie-breaks of the greedy permutation.  perq_oracle_swiglu rounds the product once to bf16 (a reading: the
 * paper's figure gives the formula, not a storage precision).  perq_oracle_hadamard_base: "parity unpinned"
 * against the authors' base matrices of order 12 / 28 / 76, which the paper does not print (Paley's second
 * construction is taken; H H^T = n I, symmetry and the Kronecker structure are pinned).
 *
 * Rows are independent; `#pragma omp parallel for` over rows is the only parallelism.
 */
#include <fenv.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------------------------------------------------------------- helpers */

static double bf16_to_double(uint16_t h)
{
    uint32_t w = (uint32_t)h << 16; /* bf16 is the upper half of an IEEE binary32 */
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

static int popcount32(uint32_t v)
{
    int c = 0;
    while (v) { c += (int)(v & 1u); v >>= 1; }
    return c;
}

int perq_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------- Hadamard matrix
 * Notation paragraph: R is a normalised Hadamard matrix, columns of unit l2 norm and
 * entries +-1/sqrt(k).  The Sylvester construction in natural order has entry (k,i)
 * equal to (-1)^{popcount(k AND i)}.
 *
 * Appendix A.1 (non-power-of-2 rotation): d = k t with t the largest odd factor of d; R is
 * built from k' = log2(k) - 2 recursive (Sylvester) applications of a 4t-dimensional base
 * matrix, so the computation is k' radix-2 stages and 2^k' independent 4t-dimensional
 * rotations of ADJACENT inputs:  H_d = H_{2^k'} (x) H_{4t}, entry (k, i) =
 * (-1)^{popcount(k/4t AND i/4t)} * H_{4t}[k mod 4t][i mod 4t].
 * The paper does not print its base matrices (H_12, H_28, H_76): PARITY UNPINNED against the
 * authors' matrix.  Reading taken here: Paley's second construction for 4t = 2(q + 1), q a
 * prime with q = 1 (mod 4) -- q = 5, 13, 37 give exactly the three orders the paper's table of
 * non-power-of-2 dimensions needs (also 36 and 60).  With chi the quadratic character mod q
 * (chi(0) = 0, chi(a) = 1 for a non-zero square, -1 otherwise) and the symmetric conference
 * matrix S of order q + 1 (S_00 = 0, S_0j = S_j0 = 1, S_ij = chi(i - j) for i, j >= 1), every
 * zero of S becomes the 2x2 block [[1, -1], [-1, -1]] and every entry +-1 becomes
 * +-[[1, 1], [1, -1]].  What the mathematics fixes, H H^T = n I, is pinned in the tests.
 *
 * Both functions write the UNNORMALISED +-1 matrix, row-major signed bytes. */
int perq_oracle_hadamard_base(int32_t n, int8_t *H)
{
    if (n < 4 || n % 4 != 0 || !H) return 1;
    const int32_t q = n / 2 - 1;
    if (q % 4 != 1) return 1;
    for (int32_t f = 2; f * f <= q; ++f)
        if (q % f == 0) return 1;                       /* prime fields only */
    int8_t *chi = (int8_t *)malloc((size_t)q);
    if (!chi) return 3;
    for (int32_t a = 0; a < q; ++a) chi[a] = -1;
    chi[0] = 0;
    for (int32_t a = 1; a < q; ++a) chi[(a * a) % q] = 1;
    for (int32_t i = 0; i <= q; ++i) {
        for (int32_t j = 0; j <= q; ++j) {
            int s;
            if (i == 0 && j == 0) s = 0;
            else if (i == 0 || j == 0) s = 1;
            else s = chi[((i - j) % q + q) % q];
            int8_t *blk = H + (size_t)(2 * i) * n + 2 * j;
            if (s == 0) {
                blk[0] = 1;  blk[1] = -1;
                blk[n] = -1; blk[n + 1] = -1;
            } else {
                blk[0] = (int8_t)s; blk[1] = (int8_t)s;
                blk[n] = (int8_t)s; blk[n + 1] = (int8_t)-s;
            }
        }
    }
    free(chi);
    return 0;
}

/* order of the base matrix of a b-dimensional rotation: 1 for a power of two (Sylvester all the
 * way down), else 4t with t the odd part of b; 0 if b has no such factorisation (k < 4). */
static int32_t base_order(int32_t b)
{
    if (b < 1) return 0;
    int32_t t = b;
    while ((t & 1) == 0) t >>= 1;
    if (t == 1) return 1;
    return (b % (4 * t) == 0) ? 4 * t : 0;
}

int perq_oracle_hadamard_pm1(int32_t b, int8_t *H)
{
    const int32_t n = base_order(b);
    if (n == 0 || !H) return 1;
    int8_t *base = (int8_t *)malloc((size_t)n * n);
    if (!base) return 3;
    if (n == 1) base[0] = 1;
    else {
        const int rc = perq_oracle_hadamard_base(n, base);
        if (rc) { free(base); return rc; }
    }
    for (int32_t k = 0; k < b; ++k)
        for (int32_t i = 0; i < b; ++i) {
            const int8_t e = base[(size_t)(k % n) * n + (i % n)];
            H[(size_t)k * b + i] = (popcount32((uint32_t)((k / n) & (i / n))) & 1) ? (int8_t)-e : e;
        }
    free(base);
    return 0;
}

/* ---------------------------------------------------------------- permute + rotate
 * Notation paragraph: X is a row vector, d = n*b; P e_i = e_{pi(i)} so (X P)_i =
 * X_{pi(i)} (a gather); R~ = I_n (x) R acts on each contiguous block of b coordinates
 * (proof of the probabilistic proposition, coordinate form: X~_i = sum over k in the
 * block of i of X_k R~_{k,i}).
 *
 * y[t, j*b + i] = (1/sqrt(b)) * sum_{k<b} x'[t, j*b + k] * H[k][i],  x'[i] = x[perm[i]].
 * The sum is an explicit matrix-vector product (k ascending), no butterfly.
 * perm == NULL is the identity.  b may be any power of two >= 1 that divides d, or b = d for a
 * d that is not a power of two (Appendix A.1; the matrix of perq_oracle_hadamard_pm1). */
int perq_oracle_rotate(const uint16_t *x, const int32_t *perm, int64_t T, int32_t d,
                       int32_t b, double *y)
{
    if (!x || !y || T < 0 || d <= 0 || b < 1 || d % b != 0) return 1;
    if ((b & (b - 1)) != 0 && b != d) return 1;          /* other orders only as the full-vector rotation */
    if (perm)
        for (int32_t i = 0; i < d; ++i)
            if (perm[i] < 0 || perm[i] >= d) return 2;
    int8_t *H = (int8_t *)malloc((size_t)b * b);
    if (!H) return 3;
    if (perq_oracle_hadamard_pm1(b, H)) { free(H); return 1; }
    const double sqrt_b = sqrt((double)b);
    int fail = 0;
#pragma omp parallel
    {
        double *xp = (double *)malloc(sizeof(double) * (size_t)d);
        double *u = (double *)malloc(sizeof(double) * (size_t)b);
        if (!xp || !u) {
#pragma omp atomic write
            fail = 1;
        } else {
#pragma omp for schedule(static)
            for (int64_t t = 0; t < T; ++t) {
                const uint16_t *row = x + (size_t)t * d;
                for (int32_t i = 0; i < d; ++i)
                    xp[i] = bf16_to_double(row[perm ? perm[i] : i]);
                for (int32_t j = 0; j < d / b; ++j) {
                    for (int32_t i = 0; i < b; ++i) u[i] = 0.0;
                    for (int32_t k = 0; k < b; ++k) {
                        const double xk = xp[(size_t)j * b + k];
                        const int8_t *Hk = H + (size_t)k * b;
                        for (int32_t i = 0; i < b; ++i) u[i] += xk * (double)Hk[i];
                    }
                    for (int32_t i = 0; i < b; ++i)
                        y[(size_t)t * d + (size_t)j * b + i] = u[i] / sqrt_b;
                }
            }
        }
        free(xp);
        free(u);
    }
    free(H);
    return fail ? 3 : 0;
}

/* ---------------------------------------------------------------- packing
 * The paper has no storage format.  Two 4-bit codes per byte: byte k of a row holds
 * code[2k] in its low nibble and code[2k+1] in its high nibble. */
static void pack_row(const uint8_t *codes, int32_t d, uint8_t *out)
{
    for (int32_t k = 0; k < d / 2; ++k)
        out[k] = (uint8_t)((codes[2 * k] & 0xF) | ((codes[2 * k + 1] & 0xF) << 4));
}

/* ---------------------------------------------------------------- INT4
 * Sec. 3: step size s = ||X||_inf / (2^{q-1} - 1), q = 4, taken over the scale range
 * (the whole token when group == 0, else each contiguous `group` coordinates of the
 * rotated row).  Appendix B quantiser with zero point 0: q_i = clip(round(y_i / s),
 * -8, 7), round = nearest, ties to even.  The division uses the real (double) s; the
 * stored scale is s rounded to binary32.  A range whose max is 0 stores scale 0 and
 * codes 0.
 *
 * codes: packed [T, d/2]; scales: float [T] or [T, d/group];
 * v_pre (optional, may be NULL): the pre-rounding values y_i / s, [T, d]. */
int perq_oracle_quantize_int4(const double *y, int64_t T, int32_t d, int32_t group,
                              uint8_t *codes, float *scales, double *v_pre)
{
    if (!y || !codes || !scales || T < 0 || d <= 0 || d % 2 != 0 || group < 0) return 1;
    const int32_t g = group == 0 ? d : group;
    if (d % g != 0) return 1;
    if (fegetround() != FE_TONEAREST) return 4;
    const int32_t ng = d / g;
#pragma omp parallel
    {
        uint8_t *c = (uint8_t *)malloc((size_t)d);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < T; ++t) {
            const double *yr = y + (size_t)t * d;
            for (int32_t r = 0; r < ng; ++r) {
                double a = 0.0;
                for (int32_t i = 0; i < g; ++i) {
                    const double m = fabs(yr[(size_t)r * g + i]);
                    if (m > a) a = m;
                }
                const double s = a / 7.0;
                scales[(size_t)t * ng + r] = (a == 0.0) ? 0.0f : (float)s;
                for (int32_t i = 0; i < g; ++i) {
                    const size_t idx = (size_t)r * g + i;
                    double v = 0.0, q = 0.0;
                    if (a != 0.0) {
                        v = yr[idx] / s;
                        q = nearbyint(v); /* FE_TONEAREST: ties to even */
                        if (q > 7.0) q = 7.0;
                        if (q < -8.0) q = -8.0;
                    }
                    if (v_pre) v_pre[(size_t)t * d + idx] = v;
                    c[idx] = (uint8_t)((int)q & 0xF); /* two's complement nibble */
                }
            }
            pack_row(c, d, codes + (size_t)t * (d / 2));
        }
        free(c);
    }
    return 0;
}

/* ---------------------------------------------------------------- MXFP4
 * Appendix B, "(MX)FP4 Quantization": elements are E2M1 (e = 2, m = 1, per the OCP MX
 * specification the paper cites), one shared scale per 32 elements, rounded down to a
 * power of two.  Reading of the shared exponent (the printed formula is garbled):
 * E = floor(log2(max |y|)) - 2, where 2 is the exponent of the largest E2M1 value
 * 6 = 1.5 * 2^2; stored as E8M0 = clamp(E, -127, 127) + 127.
 * Elements: v = y * 2^-E (exact), magnitude rounded to the nearest of
 * {0, .5, 1, 1.5, 2, 3, 4, 6}, ties to the even code, |v| > 6 saturates to 6; the sign
 * bit of y is kept (code = sign << 3 | index).  An all-zero group stores E8M0 = 0.
 *
 * codes: packed [T, d/2]; e8m0: uint8 [T, d/32];
 * v_pre (optional): the pre-rounding scaled values y_i * 2^-E, [T, d]. */
static const double E2M1_GRID[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

static int e2m1_nearest_index(double mag)
{
    if (mag >= 6.0) return 7;
    for (int k = 0; k < 7; ++k) {
        const double lo = E2M1_GRID[k], hi = E2M1_GRID[k + 1];
        if (mag >= lo && mag <= hi) {
            const double mid = 0.5 * (lo + hi); /* exact: grid values are dyadic */
            if (mag < mid) return k;
            if (mag > mid) return k + 1;
            return (k % 2 == 0) ? k : k + 1; /* tie: the even code */
        }
    }
    return 7;
}

int perq_oracle_quantize_mxfp4(const double *y, int64_t T, int32_t d, uint8_t *codes,
                               uint8_t *e8m0, double *v_pre)
{
    if (!y || !codes || !e8m0 || T < 0 || d <= 0 || d % 32 != 0) return 1;
    const int32_t ng = d / 32;
#pragma omp parallel
    {
        uint8_t *c = (uint8_t *)malloc((size_t)d);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < T; ++t) {
            const double *yr = y + (size_t)t * d;
            for (int32_t r = 0; r < ng; ++r) {
                double a = 0.0;
                for (int32_t i = 0; i < 32; ++i) {
                    const double m = fabs(yr[(size_t)r * 32 + i]);
                    if (m > a) a = m;
                }
                int E = -127;
                if (a != 0.0) {
                    int e;
                    (void)frexp(a, &e);  /* a = m * 2^e, m in [0.5, 1)  =>  floor(log2 a) = e - 1 */
                    E = (e - 1) - 2;
                    if (E < -127) E = -127;
                    if (E > 127) E = 127;
                }
                e8m0[(size_t)t * ng + r] = (a == 0.0) ? 0 : (uint8_t)(E + 127);
                for (int32_t i = 0; i < 32; ++i) {
                    const size_t idx = (size_t)r * 32 + i;
                    const double v = ldexp(yr[idx], -E);
                    if (v_pre) v_pre[(size_t)t * d + idx] = v;
                    const int k = e2m1_nearest_index(fabs(v));
                    c[idx] = (uint8_t)((signbit(yr[idx]) ? 8 : 0) | k);
                }
            }
            pack_row(c, d, codes + (size_t)t * (d / 2));
        }
        free(c);
    }
    return 0;
}

/* ---------------------------------------------------------------- asymmetric INT4, per token
 * Appendix B: activations use "the standard asymmetric activation quantizer, where zero point
 * z = min(X) / s and scaling factor s = (max(X) - min(X)) / (2^q - 1) are dynamically defined
 * per-token", in Q(X) = s * (clip(round(X / s) - z, min A, max A) + z)  (the printed equation
 * adds z outside the product with s; it belongs inside).  The codes have to be integers of the
 * alphabet {0..15}, so z is read as the integer round(min(X) / s), ties to even like every
 * rounding here.  q = 4:
 *     s = (mx - mn) / 15,  z = rne(mn / s),  c_i = clip(rne(y_i / s) - z, 0, 15),  Q = s * (c_i + z).
 * A constant row (mx == mn, including all-zero) stores s = 0, z = 0 and codes 0.
 *
 * codes: packed [T, d/2] (unsigned nibbles); scale_zero: float [T, 2] = (s, z);
 * v_pre (optional): y_i / s, [T, d]. */
int perq_oracle_quantize_int4_asym(const double *y, int64_t T, int32_t d, uint8_t *codes,
                                   float *scale_zero, double *v_pre)
{
    if (!y || !codes || !scale_zero || T < 0 || d <= 0 || d % 2 != 0) return 1;
    if (fegetround() != FE_TONEAREST) return 4;
#pragma omp parallel
    {
        uint8_t *c = (uint8_t *)malloc((size_t)d);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < T; ++t) {
            const double *yr = y + (size_t)t * d;
            double mx = yr[0], mn = yr[0];
            for (int32_t i = 1; i < d; ++i) {
                if (yr[i] > mx) mx = yr[i];
                if (yr[i] < mn) mn = yr[i];
            }
            const double s = (mx - mn) / 15.0;
            const double z = (s == 0.0) ? 0.0 : nearbyint(mn / s);
            scale_zero[2 * t] = (float)s;
            scale_zero[2 * t + 1] = (float)z;
            for (int32_t i = 0; i < d; ++i) {
                double v = 0.0, q = 0.0;
                if (s != 0.0) {
                    v = yr[i] / s;
                    q = nearbyint(v) - z;
                    if (q > 15.0) q = 15.0;
                    if (q < 0.0) q = 0.0;
                }
                if (v_pre) v_pre[(size_t)t * d + i] = v;
                c[i] = (uint8_t)q;
            }
            pack_row(c, d, codes + (size_t)t * (d / 2));
        }
        free(c);
    }
    return 0;
}

/* ---------------------------------------------------------------- FP4 with a per-token scale
 * Appendix B, "(MX)FP4 Quantization": "For FP4 activations, scaling factor
 * s = ||X||_inf / (2^{q-1} - 1) is defined dynamically per-token", elements E2M1 as above.
 * With q = 4 the step is the row maximum over 7 (the same scale as the INT4 quantiser of
 * Sec. 3), so the largest element maps to 7 and saturates to 6, like the (6, 8) band of MXFP4.
 * Elements: v = y / s in double, magnitude to the nearest of {0, .5, 1, 1.5, 2, 3, 4, 6}, ties to
 * the even code, |v| > 6 saturates; the sign bit of y is kept.  A zero row stores scale 0 and
 * sign-only codes.
 *
 * codes: packed [T, d/2]; scales: float [T]; v_pre (optional): y_i / s, [T, d]. */
int perq_oracle_quantize_fp4(const double *y, int64_t T, int32_t d, uint8_t *codes, float *scales,
                             double *v_pre)
{
    if (!y || !codes || !scales || T < 0 || d <= 0 || d % 2 != 0) return 1;
#pragma omp parallel
    {
        uint8_t *c = (uint8_t *)malloc((size_t)d);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < T; ++t) {
            const double *yr = y + (size_t)t * d;
            double a = 0.0;
            for (int32_t i = 0; i < d; ++i) {
                const double m = fabs(yr[i]);
                if (m > a) a = m;
            }
            const double s = a / 7.0;
            scales[t] = (a == 0.0) ? 0.0f : (float)s;
            for (int32_t i = 0; i < d; ++i) {
                const double v = (a == 0.0) ? 0.0 : yr[i] / s;
                if (v_pre) v_pre[(size_t)t * d + i] = v;
                const int k = e2m1_nearest_index(fabs(v));
                c[i] = (uint8_t)((signbit(yr[i]) ? 8 : 0) | k);
            }
            pack_row(c, d, codes + (size_t)t * (d / 2));
        }
        free(c);
    }
    return 0;
}

/* ---------------------------------------------------------------- gated activation in front of the path
 * Fig. "permutation-equivariance" (the feedforward network of a transformer block): the online rotation's
 * input is h = Swish(x W_gate) (.) (x W_up), an elementwise product of the Swish of one projection with the
 * other; Swish(g) = g * sigmoid(g) = g / (1 + exp(-g)).  Here the two projections are given (bf16) and h is
 * what a model would store: the real-valued product rounded ONCE to bf16, round to nearest even.
 *
 * double_to_bf16_rne rounds a finite double directly to bf16 (no intermediate float: two roundings could
 * differ from one).  bf16 has 8 significant bits and the exponent range of binary32 (normal from 2^-126,
 * subnormal quantum 2^-133); magnitudes that round beyond the largest finite bf16 become infinity. */
static uint16_t double_to_bf16_rne(double v)
{
    uint16_t sign = (uint16_t)(signbit(v) ? 0x8000u : 0u);
    double a = fabs(v);
    if (a == 0.0) return sign;
    int e;
    (void)frexp(a, &e);                       /* a = m * 2^e, m in [0.5, 1): exponent of the leading bit is e - 1 */
    int lead = e - 1;
    if (lead < -126) lead = -126;             /* subnormal range: fixed quantum 2^-133 */
    double q = nearbyint(ldexp(a, 7 - lead)); /* units of 2^(lead-7); ties to even under FE_TONEAREST */
    if (q >= 256.0) { q = 128.0; lead += 1; } /* rounded up to the next power of two */
    if (lead > 127) return (uint16_t)(sign | 0x7F80u);
    uint32_t qi = (uint32_t)q;                /* 0 .. 255; below 128 only in the subnormal range */
    if (qi < 128u) return (uint16_t)(sign | qi);
    return (uint16_t)(sign | ((uint32_t)(lead + 127) << 7) | (qi - 128u));
}

int perq_oracle_swiglu(const uint16_t *gate, const uint16_t *up, int64_t T, int32_t d, uint16_t *h)
{
    if (T < 0 || d <= 0 || !gate || !up || !h) return 1;
    fesetround(FE_TONEAREST);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        for (int32_t i = 0; i < d; ++i) {
            const double g = bf16_to_double(gate[(size_t)t * d + i]);
            const double u = bf16_to_double(up[(size_t)t * d + i]);
            const double swish = g / (1.0 + exp(-g));
            h[(size_t)t * d + i] = double_to_bf16_rne(swish * u);
        }
    }
    return 0;
}

/* ---------------------------------------------------------------- whole path
 * (X P) R~ then Q(.), Fig. "perq-pipeline" / Sec. 4 overview.  fmt: 0 = INT4, 1 = MXFP4,
 * 3 = FP4 with a per-token scale, 4 = asymmetric INT4 per token (2 is not a quantiser).
 * y_out (optional) receives the rotated row, v_pre (optional) the pre-rounding values. */
int perq_oracle_rotate_quantize(const uint16_t *x, const int32_t *perm, int64_t T, int32_t d,
                                int32_t b, int32_t fmt, int32_t group, uint8_t *codes,
                                void *scales, double *y_out, double *v_pre)
{
    if (T < 0 || d <= 0) return 1;
    double *y = y_out ? y_out : (double *)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1) * d);
    if (!y) return 3;
    int rc = perq_oracle_rotate(x, perm, T, d, b, y);
    if (rc == 0) {
        if (fmt == 0) rc = perq_oracle_quantize_int4(y, T, d, group, codes, (float *)scales, v_pre);
        else if (fmt == 1) rc = perq_oracle_quantize_mxfp4(y, T, d, codes, (uint8_t *)scales, v_pre);
        else if (fmt == 3) rc = perq_oracle_quantize_fp4(y, T, d, codes, (float *)scales, v_pre);
        else if (fmt == 4) rc = perq_oracle_quantize_int4_asym(y, T, d, codes, (float *)scales, v_pre);
        else rc = 1;
    }
    if (!y_out) free(y);
    return rc;
}

/* ---------------------------------------------------------------- calibration statistic
 * Algorithm 1 (MassDiff) uses the per-coordinate mean magnitude (1/m) sum_k |X_i^(k)|
 * and the per-block mean l1 norm (1/m) sum_k ||X^(k)_{B_j}||_1; the block proposition
 * bounds ||X R~||_inf by max_j ||X_{j}||_1 / sqrt(b).
 *
 * chan_abs_sum[c]        = sum_t |x[t, c]|                 (original channel order)
 * block_l1_mean[j]       = (1/T) sum_t L[t, j]             L[t, j] = sum_{i<b} |x'[t, j*b+i]|
 * token_max_block_l1[t]  = max_j L[t, j]                   x' = gather(x, perm)
 * Any output pointer may be NULL. */
int perq_oracle_block_l1_stats(const uint16_t *x, const int32_t *perm, int64_t T, int32_t d,
                               int32_t b, double *chan_abs_sum, double *block_l1_mean,
                               double *token_max_block_l1)
{
    if (!x || T < 0 || d <= 0 || b < 1 || d % b != 0) return 1;
    if (perm)
        for (int32_t i = 0; i < d; ++i)
            if (perm[i] < 0 || perm[i] >= d) return 2;
    const int32_t n = d / b;
    if (chan_abs_sum) for (int32_t c = 0; c < d; ++c) chan_abs_sum[c] = 0.0;
    if (block_l1_mean) for (int32_t j = 0; j < n; ++j) block_l1_mean[j] = 0.0;
    for (int64_t t = 0; t < T; ++t) {
        const uint16_t *row = x + (size_t)t * d;
        if (chan_abs_sum)
            for (int32_t c = 0; c < d; ++c) chan_abs_sum[c] += fabs(bf16_to_double(row[c]));
        double mx = 0.0;
        for (int32_t j = 0; j < n; ++j) {
            double L = 0.0;
            for (int32_t i = 0; i < b; ++i) {
                const int32_t src = perm ? perm[(size_t)j * b + i] : j * b + i;
                L += fabs(bf16_to_double(row[src]));
            }
            if (block_l1_mean) block_l1_mean[j] += L;
            if (L > mx) mx = L;
        }
        if (token_max_block_l1) token_max_block_l1[t] = mx;
    }
    if (block_l1_mean && T > 0)
        for (int32_t j = 0; j < n; ++j) block_l1_mean[j] /= (double)T;
    return 0;
}

/* ---------------------------------------------------------------- per-token diagnostics
 * The quantities the paper plots per token (the figures on delta, on the block bound versus the
 * block size, and on the bound versus the quantization error), before their normalisation by
 * ||X||_inf.  With x' = gather(x, perm), blocks of b, y = x' R~ (block Hadamard) and Q the 4-bit
 * symmetric quantiser of Sec. 3 with one step per token (s = ||y||_inf / 7, round to nearest even):
 *
 *   out[t][0] = ||x||_inf                       out[t][1] = ||x||_1
 *   out[t][2] = max_j ||x'_{j}||_1              (b * max_j delta_{j} ||x'_{j}||_inf, block proposition)
 *   out[t][3] = ||y||_inf                       out[t][4] = ||y - Q(y)||_2
 *
 * so that delta = out1 / (d out0) (full-vector proposition), the normalised block bound is
 * out2 / (b out0), the outlier suppression ratio out3 / out0 and the normalised error out4 / out0.
 * A zero row gives five zeros. */
int perq_oracle_token_diagnostics(const uint16_t *x, const int32_t *perm, int64_t T, int32_t d,
                                  int32_t b, double *out)
{
    if (!x || !out || T < 0 || d <= 0 || b < 1 || (b & (b - 1)) != 0 || d % b != 0) return 1;
    if (fegetround() != FE_TONEAREST) return 4;
    double *y = (double *)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1) * (size_t)d);
    if (!y) return 3;
    int rc = perq_oracle_rotate(x, perm, T, d, b, y);
    if (rc) { free(y); return rc; }
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        const uint16_t *row = x + (size_t)t * d;
        const double *yr = y + (size_t)t * d;
        double xinf = 0.0, x1 = 0.0, bmax = 0.0;
        for (int32_t i = 0; i < d; ++i) {
            const double a = fabs(bf16_to_double(row[i]));
            if (a > xinf) xinf = a;
            x1 += a;
        }
        for (int32_t j = 0; j < d / b; ++j) {
            double l1 = 0.0;
            for (int32_t i = 0; i < b; ++i)
                l1 += fabs(bf16_to_double(row[perm ? perm[(size_t)j * b + i] : (size_t)j * b + i]));
            if (l1 > bmax) bmax = l1;
        }
        double yinf = 0.0;
        for (int32_t i = 0; i < d; ++i)
            if (fabs(yr[i]) > yinf) yinf = fabs(yr[i]);
        double e2 = 0.0;
        if (yinf > 0.0) {
            const double s = yinf / 7.0;
            for (int32_t i = 0; i < d; ++i) {
                double q = nearbyint(yr[i] / s);
                if (q > 7.0) q = 7.0;
                if (q < -8.0) q = -8.0;
                const double e = yr[i] - s * q;
                e2 += e * e;
            }
        }
        double *o = out + (size_t)t * 5;
        o[0] = xinf; o[1] = x1; o[2] = bmax; o[3] = yinf; o[4] = sqrt(e2);
    }
    free(y);
    return 0;
}

/* ---------------------------------------------------------------- MassDiff (Algorithm 1)
 * Visit coordinates in descending mean magnitude; put each into the not-yet-full block
 * whose running mean l1 norm is smallest; drop a block from the candidates once it holds
 * b coordinates; return the blocks concatenated.  The argmin's "+ |X_i|" term is common
 * to all blocks, so only the running block sums matter, and since the mean is a positive
 * multiple of the sum the channel sums can stand in for the means.
 * Unfixed by the paper: sort ties -> lower channel index first; argmin ties -> lower
 * block index.  perm[j*b + r] = the r-th coordinate assigned to block j. */
int perq_oracle_massdiff_perm(const double *chan_abs_sum, int32_t d, int32_t b, int32_t *perm)
{
    if (!chan_abs_sum || !perm || d <= 0 || b < 1 || d % b != 0) return 1;
    const int32_t n = d / b;
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * (size_t)d);
    double *mass = (double *)calloc((size_t)n, sizeof(double));
    int32_t *fill = (int32_t *)calloc((size_t)n, sizeof(int32_t));
    if (!order || !mass || !fill) { free(order); free(mass); free(fill); return 3; }
    for (int32_t i = 0; i < d; ++i) order[i] = i;
    /* stable insertion sort, descending: equal values keep ascending index order */
    for (int32_t i = 1; i < d; ++i) {
        const int32_t c = order[i];
        int32_t p = i - 1;
        while (p >= 0 && chan_abs_sum[order[p]] < chan_abs_sum[c]) { order[p + 1] = order[p]; --p; }
        order[p + 1] = c;
    }
    for (int32_t s = 0; s < d; ++s) {
        const int32_t c = order[s];
        int32_t best = -1;
        for (int32_t j = 0; j < n; ++j) {
            if (fill[j] >= b) continue;              /* block j is full: not in J */
            if (best < 0 || mass[j] < mass[best]) best = j;
        }
        perm[(size_t)best * b + fill[best]] = c;
        fill[best] += 1;
        mass[best] += chan_abs_sum[c];
    }
    free(order); free(mass); free(fill);
    return 0;
}

/* ---------------------------------------------------------------- comparison permutations
 * Appendix C, paragraph "Permutations" (Table "permute_fn_ablations"): "absmax" permutes coordinates in
 * descending order of the maximum absolute value observed over the calibration sample; "ZigZag" assigns
 * coordinates to blocks in a zigzag pattern over a coordinate-wise l-infinity statistic (the cited method's
 * strategy; Sec. 4.2 mentions it as the alternative to MassDiff).  The paper prints neither procedure.
 * Readings taken here (parity unpinned against the authors' code): both visit channels by descending
 * statistic, equal values by ascending channel; absmax returns that order; ZigZag deals the visiting order to
 * the n = d / b blocks back and forth -- ranks 0..n-1 to blocks 0..n-1, ranks n..2n-1 to blocks n-1..0, and so
 * on -- so that every block receives one channel of every round and block j's r-th slot is round r.
 *
 * chan_abs_max[c] = max_t |x[t, c]| is the statistic of both. */
int perq_oracle_chan_abs_max(const uint16_t *x, int64_t T, int32_t d, double *chan_abs_max)
{
    if (T < 0 || d <= 0 || !x || !chan_abs_max) return 1;
    for (int32_t c = 0; c < d; ++c) chan_abs_max[c] = 0.0;
    for (int64_t t = 0; t < T; ++t)
        for (int32_t c = 0; c < d; ++c) {
            const double a = fabs(bf16_to_double(x[(size_t)t * d + c]));
            if (a > chan_abs_max[c]) chan_abs_max[c] = a;
        }
    return 0;
}

/* visiting order: descending statistic, equal values by ascending channel (insertion sort: stable) */
static void descending_order(const double *stat, int32_t d, int32_t *order)
{
    for (int32_t i = 0; i < d; ++i) {
        int32_t k = i;
        while (k > 0 && stat[order[k - 1]] < stat[i]) { order[k] = order[k - 1]; --k; }
        order[k] = i;
    }
}

int perq_oracle_absmax_perm(const double *chan_abs_max, int32_t d, int32_t *perm)
{
    if (d <= 0 || !chan_abs_max || !perm) return 1;
    descending_order(chan_abs_max, d, perm);
    return 0;
}

int perq_oracle_zigzag_perm(const double *chan_abs_max, int32_t d, int32_t b, int32_t *perm)
{
    if (d <= 0 || b <= 0 || d % b != 0 || !chan_abs_max || !perm) return 1;
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * (size_t)d);
    if (!order) return 3;
    descending_order(chan_abs_max, d, order);
    const int32_t n = d / b;
    for (int32_t r = 0; r < d; ++r) {
        const int32_t round = r / n, pos = r % n;
        const int32_t block = (round % 2 == 0) ? pos : n - 1 - pos;
        perm[(size_t)block * b + round] = order[r];
    }
    free(order);
    return 0;
}
