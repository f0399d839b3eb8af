/*
 * AMXFP4 reference ("oracle"): a plain, slow CPU restatement of the format and
 * of the quantized matrix product in arXiv 2411.09909.
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists to check the CUDA library and to be
 * timed as a CPU baseline.  The CUDA library shares no code with it and never
 * calls it.
 *
 * Format (Section 4.2, Eq. 1; Section 4.3): an element is an FP4 E2M1 number
 * (1 sign, 2 exponent, 1 mantissa bit: magnitudes 0, 0.5, 1, 1.5, 2, 3, 4, 6).
 * Elements are grouped along the last axis (32 per group, Section 2.1 and the
 * MX configuration table of Appendix A.1).  Each group carries TWO shared
 * scales in FP8 E5M2 ("1-5-2", Section 4.2 "FP8"): one used by the elements
 * whose sign bit is 0, one by the elements whose sign bit is 1.  The decoded
 * value is  (-1)^s * E2M1(E, M) * scale_{s}.
 *
 * Quantization (direct cast, no calibration).  The paper gives the procedure
 * only through Algorithm 1 (the MX quantizer) and the worked example of
 * Appendix B.3.  The reading used here, which reproduces the three value sets
 * printed in that example:
 *   1. per group, pmax = largest element with sign 0, nmax = largest |element|
 *      with sign 1 (0 when that side is empty);
 *   2. scale_side = E5M2 nearest to max_side / 6, ties to the even mantissa,
 *      saturating at the largest finite E5M2 (57344), with subnormals;
 *   3. element magnitude = E2M1 nearest to |x| / scale_side, ties to the even
 *      code, clamped at 6 (Algorithm 1: "quantize(V_i / X), clamping normal
 *      numbers"); 0 when scale_side is 0;
 *   4. the element's sign bit is the input's sign bit, also when the magnitude
 *      rounds to 0.
 * The tie rules in 2 and 3, the handling of scale under/overflow and rule 4 are
 * not fixed by the paper (parity unpinned for those choices alone: the oracle
 * defines them); everything else is pinned by the tests.
 *
 * All arithmetic on values is fp64.  x is a bf16 number (8 significant bits)
 * or, for the paper's example, an fp32 number; an E5M2 scale has 3 significant
 * bits.  A quotient that is mathematically a rounding midpoint is therefore
 * exactly representable and fp64 division returns it exactly; any other
 * quotient is at least 2^-24 (relative) away from every midpoint, far more
 * than the fp64 rounding error, so rounding the fp64 quotient equals rounding
 * the exact one.
 *
 * Also here, for the pins only: the MX power-of-two "floor" scale rule of
 * Algorithm 1 (symmetric and per-sign), and the softmax step that sits between
 * the two attention products.
 */
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---------------------------------------------------------------- E2M1 -- */

/* Magnitude of the 3-bit code EEM: exponent bias 1, subnormal when EE == 0. */
static const double E2M1_MAG[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

double amx_oracle_e2m1_value(int code4)
{
    double m = E2M1_MAG[code4 & 7];
    return (code4 & 8) ? -m : m;
}

/* Nearest E2M1 magnitude code to r >= 0, ties to the even code, clamp at 6. */
int amx_oracle_e2m1_encode(double r)
{
    if (r > 6.0)
        r = 6.0;                              /* clamp first: keeps the distances below exact */
    int best = 0;
    double best_d = fabs(r - E2M1_MAG[0]);
    for (int c = 1; c < 8; ++c) {
        double d = fabs(r - E2M1_MAG[c]);
        if (d < best_d || (d == best_d && (c & 1) == 0)) {
            best = c;
            best_d = d;
        }
    }
    return best;
}

/* ---------------------------------------------------------------- E5M2 -- */

/* Value of an E5M2 byte: 1 sign, 5 exponent (bias 15), 2 mantissa bits. */
double amx_oracle_e5m2_value(uint8_t code)
{
    int e = (code >> 2) & 31, m = code & 3;
    double v;
    if (e == 0)
        v = ldexp((double)m, -16);            /* subnormal: m/4 * 2^-14 */
    else if (e == 31)
        v = m ? NAN : INFINITY;               /* never produced by the quantizer */
    else
        v = ldexp(1.0 + m / 4.0, e - 15);
    return (code & 0x80) ? -v : v;
}

/* E5M2 code nearest to q >= 0; ties to even; saturate at 57344 (0x7B). */
uint8_t amx_oracle_e5m2_encode(double q)
{
    if (!(q > 0.0))
        return 0;
    int ex;
    (void)frexp(q, &ex);                      /* q = f * 2^ex, f in [0.5, 1) */
    int e = ex - 1;                           /* floor(log2 q) */
    if (e < -14)
        e = -14;                              /* subnormal spacing below 2^-14 */
    double quantum = ldexp(1.0, e - 2);       /* spacing of E5M2 in this binade */
    double t = q / quantum;                   /* exact: power-of-two divisor */
    double lo = floor(t), frac = t - lo;
    double n = lo;
    if (frac > 0.5 || (frac == 0.5 && fmod(lo, 2.0) == 1.0))
        n = lo + 1.0;
    if (n == 8.0) {                           /* rounded up into the next binade */
        n = 4.0;
        e += 1;
    }
    if (e > 15)
        return 0x7B;                          /* 1.75 * 2^15 = 57344 */
    if (n < 4.0)                              /* only possible with e == -14 */
        return (uint8_t)n;
    return (uint8_t)(((e + 15) << 2) | ((int)n - 4));
}

/* ------------------------------------------------------------- helpers -- */

static double bf16_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/*
 * One group of n values -> n 4-bit codes and the two scale bytes.
 * v holds the values, sgn the sign bits (kept apart so that -0.0 survives).
 */
static void quantize_group(const double *v, const int *sgn, int n,
                           uint8_t *code4, uint8_t *scale_pos, uint8_t *scale_neg)
{
    double pmax = 0.0, nmax = 0.0;
    for (int i = 0; i < n; ++i) {
        double a = fabs(v[i]);
        if (sgn[i]) { if (a > nmax) nmax = a; }
        else        { if (a > pmax) pmax = a; }
    }
    uint8_t sp = amx_oracle_e5m2_encode(pmax / 6.0);
    uint8_t sn = amx_oracle_e5m2_encode(nmax / 6.0);
    double vp = amx_oracle_e5m2_value(sp), vn = amx_oracle_e5m2_value(sn);
    for (int i = 0; i < n; ++i) {
        double s = sgn[i] ? vn : vp;
        int mag = (s > 0.0) ? amx_oracle_e2m1_encode(fabs(v[i]) / s) : 0;
        code4[i] = (uint8_t)((sgn[i] << 3) | mag);
    }
    *scale_pos = sp;
    *scale_neg = sn;
}

/* ------------------------------------------------------------ quantize -- */

/*
 * x: bf16 bit patterns [rows][ld] (ld >= K, elements), groups of gs along K.
 * codes:  [rows][K/2], element 2j in the low nibble of byte j.
 * scales: [rows][K/gs][2] = {positive-side E5M2, negative-side E5M2}.
 * Returns 0, or -1 when K % gs != 0 or K is odd.
 */
int amx_oracle_quantize(const uint16_t *x, int64_t rows, int64_t K, int64_t ld, int gs,
                        uint8_t *codes, uint8_t *scales)
{
    if (gs <= 0 || K % gs != 0 || (K & 1))
        return -1;
    int64_t G = K / gs;
#pragma omp parallel
    {
        double *v = (double *)malloc(sizeof(double) * gs);
        int *sg = (int *)malloc(sizeof(int) * gs);
        uint8_t *c = (uint8_t *)malloc(gs);
#pragma omp for schedule(static)
        for (int64_t r = 0; r < rows; ++r) {
            for (int64_t g = 0; g < G; ++g) {
                const uint16_t *xg = x + r * ld + g * gs;
                for (int i = 0; i < gs; ++i) {
                    v[i] = bf16_to_double(xg[i]);
                    sg[i] = xg[i] >> 15;
                }
                uint8_t sp, sn;
                quantize_group(v, sg, gs, c, &sp, &sn);
                for (int i = 0; i < gs; ++i) {
                    int64_t k = g * gs + i;
                    uint8_t *byte = codes + r * (K / 2) + k / 2;
                    if (k & 1) *byte = (uint8_t)((*byte & 0x0F) | (c[i] << 4));
                    else       *byte = (uint8_t)((*byte & 0xF0) | c[i]);
                }
                scales[(r * G + g) * 2 + 0] = sp;
                scales[(r * G + g) * 2 + 1] = sn;
            }
        }
        free(v); free(sg); free(c);
    }
    return 0;
}

/*
 * The two symmetric formats the paper compares AMXFP4 with, in the same storage
 * layout (both scale bytes of a group hold the one shared scale, so the decoder
 * and the matrix product need no change):
 *   mode 1  one FP8 E5M2 scale per group, nearest to max|x| / 6 - Section 4.2's
 *           FP8 shared scale without Section 4.3's split by sign;
 *   mode 2  MXFP4 - Algorithm 1: shared_exp = floor(log2(max|x|)) - 2 (2 = the
 *           largest E2M1 exponent), X = 2^shared_exp, elements nearest E2M1 of
 *           x / X with clamping.  X is stored as the E5M2 byte of the same power
 *           of two; a shared_exp above 15 is stored as 2^15 and one below -16 as
 *           a zero scale (Algorithm 1's 8-bit exponent reaches further: a range
 *           difference only, outside [2^-14, 2^18) group maxima).
 * Element rounding, sign bit and zero-scale rules are those of the quantizer
 * above.
 */
/* Scale byte of one side (or of the whole group) from its largest magnitude.
 * rule 0: E5M2 nearest to max / 6 (Section 4.2);
 * rule 1: Algorithm 1, 2^(floor(log2 max) - 2);
 * rule 2: the same with the exponent rounded instead of floored (appendix
 *         "Determining PoT Shared Scale: Floor vs. Round"), read as
 *         2^(round(log2 max) - 2): one more than the floor when max is at
 *         least sqrt(2) times its power of two. */
static uint8_t variant_scale_byte(double amax, int rule)
{
    if (rule == 0)
        return amx_oracle_e5m2_encode(amax / 6.0);
    if (!(amax > 0.0))
        return 0;
    int e;
    double f = 2.0 * frexp(amax, &e);          /* amax = f * 2^(e-1), 1 <= f < 2 */
    int shared_exp = (e - 1) - 2;              /* floor(log2(amax)) - emax_elem */
    if (rule == 2 && f * f >= 2.0)             /* log2 f >= 1/2 (f*f is exact: f has 8 bits) */
        shared_exp += 1;
    if (shared_exp > 15) shared_exp = 15;
    return shared_exp < -16 ? 0 : amx_oracle_e5m2_encode(ldexp(1.0, shared_exp));
}

/* modes: 1 symmetric FP8 scale, 2 MXFP4 (power-of-two floor), 3 per-sign
 * power-of-two floor ("AMXFP4, shared scale PoT" of Appendix B.3), 4 symmetric
 * power-of-two round, 5 per-sign power-of-two round. */
int amx_oracle_quantize_variant(const uint16_t *x, int64_t rows, int64_t K, int64_t ld, int gs,
                                int mode, uint8_t *codes, uint8_t *scales)
{
    if (gs <= 0 || K % gs != 0 || (K & 1) || mode < 1 || mode > 5)
        return -1;
    const int per_sign = (mode == 3 || mode == 5);
    const int rule = mode == 1 ? 0 : (mode == 2 || mode == 3) ? 1 : 2;
    int64_t G = K / gs;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t g = 0; g < G; ++g) {
            const uint16_t *xg = x + r * ld + g * gs;
            double pmax = 0.0, nmax = 0.0;
            for (int i = 0; i < gs; ++i) {
                double a = fabs(bf16_to_double(xg[i]));
                if (xg[i] >> 15) { if (a > nmax) nmax = a; }
                else             { if (a > pmax) pmax = a; }
            }
            uint8_t sb[2];
            if (per_sign) {
                sb[0] = variant_scale_byte(pmax, rule);
                sb[1] = variant_scale_byte(nmax, rule);
            } else {
                sb[0] = sb[1] = variant_scale_byte(pmax > nmax ? pmax : nmax, rule);
            }
            for (int i = 0; i < gs; ++i) {
                int sign = xg[i] >> 15;
                double sv = amx_oracle_e5m2_value(sb[sign]);
                int mag = sv > 0.0 ? amx_oracle_e2m1_encode(fabs(bf16_to_double(xg[i])) / sv) : 0;
                uint8_t c = (uint8_t)((sign << 3) | mag);
                int64_t k = g * gs + i;
                uint8_t *byte = codes + r * (K / 2) + k / 2;
                if (k & 1) *byte = (uint8_t)((*byte & 0x0F) | (c << 4));
                else       *byte = (uint8_t)((*byte & 0xF0) | c);
            }
            scales[(r * G + g) * 2 + 0] = sb[0];
            scales[(r * G + g) * 2 + 1] = sb[1];
        }
    return 0;
}

/* Same quantizer on fp64 inputs, one code per byte (used by the pins). */
int amx_oracle_quantize_f64(const double *x, int64_t rows, int64_t K, int gs,
                            uint8_t *code4, uint8_t *scales)
{
    if (gs <= 0 || K % gs != 0)
        return -1;
    int64_t G = K / gs;
    int *sg = (int *)malloc(sizeof(int) * gs);
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t g = 0; g < G; ++g) {
            const double *xg = x + r * K + g * gs;
            for (int i = 0; i < gs; ++i)
                sg[i] = signbit(xg[i]) ? 1 : 0;
            quantize_group(xg, sg, gs, code4 + r * K + g * gs,
                           &scales[(r * G + g) * 2], &scales[(r * G + g) * 2 + 1]);
        }
    free(sg);
    return 0;
}

/* ---------------------------------------------------------- dequantize -- */

/* Eq. 1: value = (-1)^s * E2M1 * (s ? negative scale : positive scale). */
int amx_oracle_dequantize(const uint8_t *codes, const uint8_t *scales,
                          int64_t rows, int64_t K, int gs, double *out)
{
    if (gs <= 0 || K % gs != 0 || (K & 1))
        return -1;
    int64_t G = K / gs;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            uint8_t byte = codes[r * (K / 2) + k / 2];
            int c = (k & 1) ? (byte >> 4) : (byte & 15);
            const uint8_t *sc = scales + (r * G + k / gs) * 2;
            double s = amx_oracle_e5m2_value((c & 8) ? sc[1] : sc[0]);
            out[r * K + k] = amx_oracle_e2m1_value(c) * s;
        }
    return 0;
}

/* --------------------------------------------------- quantization error -- */

/*
 * Squared error of a quantized tensor against its bf16 source, split the way
 * the appendix on power-of-two scales (floor vs. round) splits it: an element
 * whose magnitude exceeds the largest value its side can represent
 * (|x| > 6 * scale of its side) contributes to the max-clamping error, every
 * other element to the rounding error.
 * out[0] = sum x^2, out[1] = sum (x - xhat)^2 over all elements,
 * out[2] = the part of out[1] from clamped elements, out[3] = their count.
 * Plain fp64 sums in index order.
 */
int amx_oracle_quant_error(const uint16_t *x, int64_t rows, int64_t K, int64_t ld,
                           const uint8_t *codes, const uint8_t *scales, int gs, double *out)
{
    if (gs <= 0 || K % gs != 0 || (K & 1))
        return -1;
    int64_t G = K / gs;
    double sx = 0.0, se = 0.0, sc_err = 0.0, n_clamped = 0.0;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            double v = bf16_to_double(x[r * ld + k]);
            uint8_t byte = codes[r * (K / 2) + k / 2];
            int c = (k & 1) ? (byte >> 4) : (byte & 15);
            const uint8_t *sc = scales + (r * G + k / gs) * 2;
            double s = amx_oracle_e5m2_value((c & 8) ? sc[1] : sc[0]);
            double e = v - amx_oracle_e2m1_value(c) * s;
            sx += v * v;
            se += e * e;
            if (fabs(v) > 6.0 * s) {
                sc_err += e * e;
                n_clamped += 1.0;
            }
        }
    out[0] = sx; out[1] = se; out[2] = sc_err; out[3] = n_clamped;
    return 0;
}

/* ---------------------------------------------------------------- GEMM -- */

/*
 * C[i][n] = sum_k Ahat[row_i][k] * What[n][k], Ahat and What the decoded
 * operands (Section 4.3: each product uses the scale its own sign selects),
 * accumulated in fp64 in index order and rounded once to fp32.
 * rows_idx (nullable) lists which rows of A to compute: n_rows of them; with
 * NULL the rows are 0..n_rows-1.  C is [n_rows][N].
 */
int amx_oracle_gemm(const uint8_t *codesA, const uint8_t *scalesA,
                    const uint8_t *codesW, const uint8_t *scalesW,
                    int64_t M, int64_t N, int64_t K, int gs,
                    const int64_t *rows_idx, int64_t n_rows, float *C)
{
    if (gs <= 0 || K % gs != 0 || (K & 1))
        return -1;
    double *What = (double *)malloc(sizeof(double) * (size_t)N * (size_t)K);
    if (!What)
        return -2;
    amx_oracle_dequantize(codesW, scalesW, N, K, gs, What);
    int64_t G = K / gs;
    int bad = 0;
#pragma omp parallel
    {
        double *a = (double *)malloc(sizeof(double) * (size_t)K);
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < n_rows; ++i) {
            int64_t r = rows_idx ? rows_idx[i] : i;
            if (r < 0 || r >= M) {
#pragma omp atomic write
                bad = 1;
                continue;
            }
            amx_oracle_dequantize(codesA + r * (K / 2), scalesA + r * G * 2, 1, K, gs, a);
            for (int64_t n = 0; n < N; ++n) {
                const double *w = What + n * K;
                double acc = 0.0;
                for (int64_t k = 0; k < K; ++k)
                    acc += a[k] * w[k];
                C[i * N + n] = (float)acc;
            }
        }
        free(a);
    }
    free(What);
    return bad ? -3 : 0;
}

/* --------------------------------------- Algorithm 1 (pins only) -------- */

/*
 * MX quantizer with the power-of-two "floor" scale of Algorithm 1:
 *   shared_exp = floor(log2(max |V_i|)) - emax_elem,  emax_elem = 2 for E2M1,
 *   X = 2^shared_exp,  P_i = nearest E2M1 of V_i / X with clamping.
 * asym = 0: one scale from the largest magnitude of the group (MXFP4);
 * asym = 1: the same rule applied to each sign separately (the example's
 *           "AMXFP4, shared scale PoT").
 * Writes the decoded ("fake-quantized") values, which is what the example prints.
 */
int amx_oracle_fakequant_pot_floor(const double *x, int64_t rows, int64_t K, int gs,
                                   int asym, double *out)
{
    if (gs <= 0 || K % gs != 0)
        return -1;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t g0 = 0; g0 < K; g0 += gs) {
            const double *v = x + r * K + g0;
            double mx[2] = {0.0, 0.0};
            for (int i = 0; i < gs; ++i) {
                int s = asym ? (signbit(v[i]) ? 1 : 0) : 0;
                if (fabs(v[i]) > mx[s]) mx[s] = fabs(v[i]);
            }
            double X[2];
            for (int s = 0; s < 2; ++s)
                X[s] = mx[s] > 0.0 ? ldexp(1.0, (int)floor(log2(mx[s])) - 2) : 0.0;
            for (int i = 0; i < gs; ++i) {
                int sb = signbit(v[i]) ? 1 : 0;
                double Xs = X[asym ? sb : 0];
                double q = Xs > 0.0 ? E2M1_MAG[amx_oracle_e2m1_encode(fabs(v[i]) / Xs)] * Xs : 0.0;
                out[r * K + g0 + i] = sb ? -q : q;
            }
        }
    return 0;
}

/* ------------------------------------------- attention glue (config 5) -- */

/*
 * Row softmax of alpha * S in fp64, then each probability rounded to bf16
 * (nearest, ties to even).  The paper quantizes the normalised self-attention
 * map (Appendix C, quantization settings); the quantizer's input type is bf16,
 * so the map is rounded to bf16 before it is grouped along the key axis.
 */
static uint16_t double_to_bf16_rne(double p)
{
    if (!(p > 0.0))
        return 0;
    int ex;
    (void)frexp(p, &ex);
    int e = ex - 1;
    if (e < -126) e = -126;
    double quantum = ldexp(1.0, e - 7);
    double t = p / quantum, lo = floor(t), frac = t - lo;
    if (frac > 0.5 || (frac == 0.5 && fmod(lo, 2.0) == 1.0)) lo += 1.0;
    float f = (float)(lo * quantum);          /* exact: at most 8 significant bits */
    uint32_t u;
    memcpy(&u, &f, 4);
    return (uint16_t)(u >> 16);
}

int amx_oracle_softmax_bf16(const float *S, int64_t rows, int64_t cols, double alpha,
                            uint16_t *P)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const float *s = S + r * cols;
        double mx = -INFINITY, sum = 0.0;
        for (int64_t c = 0; c < cols; ++c)
            if (alpha * s[c] > mx) mx = alpha * s[c];
        for (int64_t c = 0; c < cols; ++c)
            sum += exp(alpha * s[c] - mx);
        for (int64_t c = 0; c < cols; ++c)
            P[r * cols + c] = double_to_bf16_rne(exp(alpha * s[c] - mx) / sum);
    }
    return 0;
}

/*
 * The same with a causal mask: row r is query row0 + r and sees the keys (columns) 0 .. row0 + r only; the
 * others get probability 0 (bf16 +0).  The paper's decoder-only models attend causally; the mask is applied to
 * the logits before the softmax, as usual.
 */
int amx_oracle_softmax_bf16_causal(const float *S, int64_t rows, int64_t cols, double alpha,
                                   int64_t row0, uint16_t *P)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const float *s = S + r * cols;
        int64_t seen = row0 + r + 1;
        if (seen > cols) seen = cols;
        double mx = -INFINITY, sum = 0.0;
        for (int64_t c = 0; c < seen; ++c)
            if (alpha * s[c] > mx) mx = alpha * s[c];
        for (int64_t c = 0; c < seen; ++c)
            sum += exp(alpha * s[c] - mx);
        for (int64_t c = 0; c < cols; ++c)
            P[r * cols + c] = c < seen ? double_to_bf16_rne(exp(alpha * s[c] - mx) / sum) : 0;
    }
    return 0;
}

int amx_oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}
