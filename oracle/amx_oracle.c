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

/* ------------------------------------------------- NVFP4 / ANVFP4 -- */

/*
 * The "recently deployed commercial" format the paper compares with in Section 5
 * (table of NVFP4 / ANVFP4 results): FP4 E2M1 elements in groups of 16 with a
 * double scaling - one FP32 scale for the whole tensor and one FP8 E4M3 scale per
 * group.  ANVFP4 is the paper's asymmetric variant: two E4M3 scales per group, one
 * per sign, as in AMXFP4.  The paper names the parts but no arithmetic; the reading
 * used here (recorded in the design notes):
 *   tensor scale  t = max|x| / (448 * 6): the largest group scale then sits at the
 *                 top of the E4M3 range (448) and the largest element at 6;
 *                 t = 1 for an all-zero tensor;
 *   group scale   E4M3 nearest (ties to even, saturating at 448, with subnormals)
 *                 to (max_side / 6) / t;
 *   element       E2M1 nearest (ties to even, clamped at 6) to x / (scale * t);
 *                 sign bit = the input's sign bit; magnitude 0 under a zero scale;
 *   decoded value (-1)^s * E2M1 * E4M3(scale_s) * t.
 * Precision of the DECISIONS: with a 24-bit tensor scale the quotients above are not
 * exactly representable and can lie within 2^-30 of a rounding boundary, which no
 * fp32 arithmetic resolves.  So that a device implementation can take every
 * decision exactly as this reference does, the decisions are taken in IEEE fp32,
 * in this order (each operation rounded to nearest even):
 *     t     = amax / 2688
 *     rt    = 1 / t
 *     g     = (max_side * fl(1/6)) * rt              -> E4M3 byte
 *     d     = E4M3(byte) * t,   rd = 1 / d
 *     q     = x * rd                                  -> E2M1 code
 * The tests pin this against exact rational arithmetic: the two agree except for
 * quotients within 2^-20 (relative) of a boundary, and agree everywhere on inputs
 * for which the fp32 operations are exact.
 */

/* Value of an E4M3 byte (OCP FP8 E4M3: bias 7, no infinities, 0x7F / 0xFF = NaN). */
double amx_oracle_e4m3_value(uint8_t code)
{
    int e = (code >> 3) & 15, m = code & 7;
    double v;
    if (e == 15 && m == 7)
        v = NAN;
    else if (e == 0)
        v = ldexp((double)m, -9);             /* subnormal: m/8 * 2^-6 */
    else
        v = ldexp(1.0 + m / 8.0, e - 7);
    return (code & 0x80) ? -v : v;
}

/* E4M3 byte nearest to q >= 0; ties to even; saturate at 448 (0x7E). */
uint8_t amx_oracle_e4m3_encode(double q)
{
    if (!(q > 0.0))
        return 0;
    int ex;
    (void)frexp(q, &ex);
    int e = ex - 1;                           /* floor(log2 q) */
    if (e < -6)
        e = -6;                               /* subnormal spacing below 2^-6 */
    double quantum = ldexp(1.0, e - 3);
    double t = q / quantum;                   /* exact: power-of-two divisor */
    double lo = floor(t), frac = t - lo, n = lo;
    if (frac > 0.5 || (frac == 0.5 && fmod(lo, 2.0) == 1.0))
        n = lo + 1.0;
    if (n == 16.0) {
        n = 8.0;
        e += 1;
    }
    if (e > 8 || (e == 8 && n > 14.0))
        return 0x7E;                          /* 1.75 * 2^8 = 448 */
    if (n < 8.0)                              /* only possible with e == -6 */
        return (uint8_t)n;
    return (uint8_t)(((e + 7) << 3) | ((int)n - 8));
}

static float bf16_to_float(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/*
 * x: bf16 bit patterns [rows][ld]; groups of 16 along K (K % 16 == 0).
 * asym = 0: NVFP4 (one scale per group, stored in both bytes); 1: ANVFP4.
 * codes [rows][K/2], scales [rows][K/16][2] (E4M3 bytes: positive side, negative
 * side), *tensor_scale = t.
 */
int amx_oracle_quantize_nv(const uint16_t *x, int64_t rows, int64_t K, int64_t ld, int asym,
                           uint8_t *codes, uint8_t *scales, float *tensor_scale)
{
    if (K <= 0 || K % 16 != 0)
        return -1;
    float amax = 0.0f;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            float a = fabsf(bf16_to_float(x[r * ld + k]));
            if (a > amax) amax = a;
        }
    const volatile float t = amax > 0.0f ? amax / 2688.0f : 1.0f;
    const volatile float rt = 1.0f / t;
    const volatile float sixth = 1.0f / 6.0f;
    *tensor_scale = t;
    int64_t G = K / 16;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t g = 0; g < G; ++g) {
            const uint16_t *xg = x + r * ld + g * 16;
            float pmax = 0.0f, nmax = 0.0f;
            for (int i = 0; i < 16; ++i) {
                float a = fabsf(bf16_to_float(xg[i]));
                if (xg[i] >> 15) { if (a > nmax) nmax = a; }
                else             { if (a > pmax) pmax = a; }
            }
            if (!asym)
                pmax = nmax = (pmax > nmax ? pmax : nmax);
            uint8_t byte[2];
            float rd[2];
            for (int side = 0; side < 2; ++side) {
                volatile float g1 = (side ? nmax : pmax) * sixth;   /* every product rounded to fp32 */
                volatile float g2 = g1 * rt;
                byte[side] = amx_oracle_e4m3_encode((double)g2);
                volatile float d = (float)amx_oracle_e4m3_value(byte[side]) * t;
                volatile float inv = 1.0f / d;
                rd[side] = byte[side] ? inv : 0.0f;
            }
            for (int i = 0; i < 16; ++i) {
                int sgn = xg[i] >> 15;
                volatile float q = fabsf(bf16_to_float(xg[i])) * rd[sgn];
                int mag = byte[sgn] ? amx_oracle_e2m1_encode((double)q) : 0;
                uint8_t c = (uint8_t)((sgn << 3) | mag);
                int64_t k = g * 16 + i;
                uint8_t *b = codes + r * (K / 2) + k / 2;
                if (k & 1) *b = (uint8_t)((*b & 0x0F) | (c << 4));
                else       *b = (uint8_t)((*b & 0xF0) | c);
            }
            scales[(r * G + g) * 2 + 0] = byte[0];
            scales[(r * G + g) * 2 + 1] = byte[1];
        }
    return 0;
}

/* out[r][k] = (-1)^s * E2M1 * E4M3(scale_s) * t, in fp64 (the first product is exact). */
int amx_oracle_dequantize_nv(const uint8_t *codes, const uint8_t *scales, float tensor_scale,
                             int64_t rows, int64_t K, double *out)
{
    if (K <= 0 || K % 16 != 0)
        return -1;
    int64_t G = K / 16;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            uint8_t byte = codes[r * (K / 2) + k / 2];
            int c = (k & 1) ? (byte >> 4) : (byte & 15);
            double s = amx_oracle_e4m3_value(scales[(r * G + k / 16) * 2 + ((c >> 3) & 1)]);
            out[r * K + k] = amx_oracle_e2m1_value(c) * s * (double)tensor_scale;
        }
    return 0;
}

/*
 * C[i][n] = tA * tW * sum_k (E2M1 * E4M3)_A[rows[i]][k] * (E2M1 * E4M3)_W[n][k], fp64 sums,
 * rounded once to fp32.  rows == NULL: all M rows.
 */
int amx_oracle_gemm_nv(const uint8_t *codesA, const uint8_t *scalesA, float tA,
                       const uint8_t *codesW, const uint8_t *scalesW, float tW,
                       int64_t M, int64_t N, int64_t K, const int64_t *rows, int64_t n_rows, float *C)
{
    if (K <= 0 || K % 16 != 0)
        return -1;
    int64_t G = K / 16;
    double *w = (double *)malloc(sizeof(double) * (size_t)N * (size_t)K);
    if (!w)
        return -2;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) {
            uint8_t byte = codesW[n * (K / 2) + k / 2];
            int c = (k & 1) ? (byte >> 4) : (byte & 15);
            w[n * K + k] = amx_oracle_e2m1_value(c) * amx_oracle_e4m3_value(scalesW[(n * G + k / 16) * 2 + ((c >> 3) & 1)]);
        }
#pragma omp parallel
    {
        double *a = (double *)malloc(sizeof(double) * (size_t)K);
#pragma omp for schedule(static)
        for (int64_t i = 0; i < n_rows; ++i) {
            int64_t m = rows ? rows[i] : i;
            if (m < 0 || m >= M) continue;
            for (int64_t k = 0; k < K; ++k) {
                uint8_t byte = codesA[m * (K / 2) + k / 2];
                int c = (k & 1) ? (byte >> 4) : (byte & 15);
                a[k] = amx_oracle_e2m1_value(c) * amx_oracle_e4m3_value(scalesA[(m * G + k / 16) * 2 + ((c >> 3) & 1)]);
            }
            for (int64_t n = 0; n < N; ++n) {
                double acc = 0.0;
                for (int64_t k = 0; k < K; ++k) acc += a[k] * w[n * K + k];
                C[i * N + n] = (float)(acc * (double)tA * (double)tW);
            }
        }
        free(a);
    }
    free(w);
    return 0;
}

/* ------------------------------------ FP16 shared scales (scale-encoding ablation) -- */

/*
 * The appendix's ablation of the shared-scale encoding compares the FP8 scale with
 * a 16-bit floating-point one, for the symmetric FP4 format and for the asymmetric
 * one, at group sizes 16 to 128.  Here: the quantizer of Sections 4.2-4.3 with
 * every "nearest E5M2" replaced by "nearest IEEE binary16" (ties to even, subnormals
 * kept, saturating at 65504; a quotient that rounds to zero gives a zero scale and
 * zero magnitudes, as in the FP8 quantizer).  Element rounding, clamping and the
 * sign bit are unchanged.
 * Layout: codes as everywhere, scales uint16 [rows][K/gs][2] = binary16 bit
 * patterns {positive side, negative side}; the symmetric format stores the one
 * scale of max|x| / 6 in both.
 */

/* Value of a binary16 bit pattern (never an infinity or NaN from the quantizer). */
double amx_oracle_f16_value(uint16_t bits)
{
    int e = (bits >> 10) & 31, m = bits & 1023;
    double v;
    if (e == 0)
        v = ldexp((double)m, -24);            /* subnormal: m/1024 * 2^-14 */
    else if (e == 31)
        v = m ? NAN : INFINITY;
    else
        v = ldexp(1.0 + m / 1024.0, e - 15);
    return (bits & 0x8000) ? -v : v;
}

/* binary16 pattern nearest to q >= 0; ties to even; saturate at 65504 (0x7BFF). */
uint16_t amx_oracle_f16_encode(double q)
{
    if (!(q > 0.0))
        return 0;
    int ex;
    (void)frexp(q, &ex);
    int e = ex - 1;                           /* floor(log2 q) */
    if (e < -14)
        e = -14;                              /* subnormal spacing below 2^-14 */
    double quantum = ldexp(1.0, e - 10);
    double t = q / quantum;                   /* exact: power-of-two divisor */
    double lo = floor(t), frac = t - lo, n = lo;
    if (frac > 0.5 || (frac == 0.5 && fmod(lo, 2.0) == 1.0))
        n = lo + 1.0;
    if (n == 2048.0) {                        /* rounded up into the next binade */
        n = 1024.0;
        e += 1;
    }
    if (e > 15)
        return 0x7BFF;
    if (n < 1024.0)                           /* only possible with e == -14 */
        return (uint16_t)n;
    return (uint16_t)(((e + 15) << 10) | ((int)n - 1024));
}

/*
 * asym = 1: one scale per sign (AMXFP4 with FP16 scales); 0: one per group.
 * e4m3 = 1: the ablation's other FP8 scale, "1-4-3": the scale is the nearest FP8 E4M3 value (ties to even,
 * subnormals kept, saturating at 448) instead of the nearest binary16; every E4M3 value is a binary16 value, so
 * it is stored as that value's binary16 pattern in the same layout and everything downstream is unchanged.
 */
int amx_oracle_quantize_f16s(const uint16_t *x, int64_t rows, int64_t K, int64_t ld, int gs, int asym, int e4m3,
                             uint8_t *codes, uint16_t *scales)
{
    if (gs <= 0 || K % gs != 0 || (K & 1))
        return -1;
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
            if (!asym)
                pmax = nmax = (pmax > nmax ? pmax : nmax);
            uint16_t sb[2];
            if (e4m3) {
                sb[0] = amx_oracle_f16_encode(amx_oracle_e4m3_value(amx_oracle_e4m3_encode(pmax / 6.0)));
                sb[1] = amx_oracle_f16_encode(amx_oracle_e4m3_value(amx_oracle_e4m3_encode(nmax / 6.0)));
            } else {
                sb[0] = amx_oracle_f16_encode(pmax / 6.0);
                sb[1] = amx_oracle_f16_encode(nmax / 6.0);
            }
            for (int i = 0; i < gs; ++i) {
                int sign = xg[i] >> 15;
                double sv = amx_oracle_f16_value(sb[sign]);
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

/* Eq. 1 with binary16 scales. */
int amx_oracle_dequantize_f16s(const uint8_t *codes, const uint16_t *scales,
                               int64_t rows, int64_t K, int gs, double *out)
{
    if (gs <= 0 || K % gs != 0 || (K & 1))
        return -1;
    int64_t G = K / gs;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            uint8_t byte = codes[r * (K / 2) + k / 2];
            int c = (k & 1) ? (byte >> 4) : (byte & 15);
            double s = amx_oracle_f16_value(scales[(r * G + k / gs) * 2 + ((c >> 3) & 1)]);
            out[r * K + k] = amx_oracle_e2m1_value(c) * s;
        }
    return 0;
}

/* C[m][n] = sum_k Ahat[m][k] * What[n][k]: fp64 sums in index order, rounded once to fp32. */
int amx_oracle_gemm_f16s(const uint8_t *codesA, const uint16_t *scalesA,
                         const uint8_t *codesW, const uint16_t *scalesW,
                         int64_t M, int64_t N, int64_t K, int gs, float *C)
{
    if (gs <= 0 || K % gs != 0 || (K & 1))
        return -1;
    double *a = (double *)malloc(sizeof(double) * (size_t)M * (size_t)K);
    double *w = (double *)malloc(sizeof(double) * (size_t)N * (size_t)K);
    if (!a || !w) {
        free(a); free(w);
        return -2;
    }
    amx_oracle_dequantize_f16s(codesA, scalesA, M, K, gs, a);
    amx_oracle_dequantize_f16s(codesW, scalesW, N, K, gs, w);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) acc += a[m * K + k] * w[n * K + k];
            C[m * N + n] = (float)acc;
        }
    free(a); free(w);
    return 0;
}

/* amx_oracle_quant_error with binary16 scales (same four sums). */
int amx_oracle_quant_error_f16s(const uint16_t *x, int64_t rows, int64_t K, int64_t ld,
                                const uint8_t *codes, const uint16_t *scales, int gs, double *out)
{
    if (gs <= 0 || K % gs != 0 || (K & 1))
        return -1;
    int64_t G = K / gs;
    double x2 = 0.0, e2 = 0.0, c2 = 0.0, cnt = 0.0;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            double v = bf16_to_double(x[r * ld + k]);
            uint8_t byte = codes[r * (K / 2) + k / 2];
            int c = (k & 1) ? (byte >> 4) : (byte & 15);
            double s = amx_oracle_f16_value(scales[(r * G + k / gs) * 2 + ((c >> 3) & 1)]);
            double e = v - amx_oracle_e2m1_value(c) * s;
            x2 += v * v;
            e2 += e * e;
            if (fabs(v) > 6.0 * s) {
                c2 += e * e;
                cnt += 1.0;
            }
        }
    out[0] = x2; out[1] = e2; out[2] = c2; out[3] = cnt;
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
