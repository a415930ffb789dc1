/*
 * mxq oracle -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.
 *
 * A plain, slow, CPU-only statement of what the MXFP4 weight-only linear path
 * of ML-SpecQD (arXiv 2503.13565) computes.  It exists so that the CUDA
 * library can be checked against something that can be compared with the
 * paper by eye.  It shares no code, header, table or helper with the CUDA
 * sources, and nothing in the product may call it: only the tests, the smoke
 * check and the benchmark's cpu_baseline / reference legs do.
 *
 * Everything here is written for clarity: one element at a time, double
 * precision, no blocking, no intrinsics.  The only concession to size is an
 * OpenMP "parallel for" over independent output rows, which changes no
 * arithmetic and no summation order.
 *
 * What each function follows:
 *   oq_quantize        Sec. III-D-3, the two-step direct cast: a shared
 *                      power-of-two scale X taken from the block maximum, then
 *                      v/X rounded to E2M1 and clamped to the largest normal
 *                      with the sign kept.
 *   oq_dequantize      the value an (E2M1 code, E8M0 scale) pair stands for,
 *                      same section: the element has one sign bit, two
 *                      exponent bits and one mantissa bit; the scale byte is
 *                      the biased exponent field of a binary32, read unsigned.
 *   oq_linear          the plain definition Y = X * dequant(W)^T that the GEMM
 *                      microkernel of Sec. III-D-3 must reproduce.  Eq. 2 says
 *                      that scaling a 32-long partial sum equals scaling every
 *                      weight in it, so the oracle scales every weight.
 *   oq_greedy_accept   Sec. III-A and Sec. III-B: of N drafted tokens the
 *                      target keeps the first G that agree with its own greedy
 *                      choice, drops everything after the first mismatch, and
 *                      contributes one more token of its own (G+1 produced).
 *
 * Parity pins live in tests/test_oracle_*.py; no function here is unpinned.
 *
 * Conventions (BF16 = upper 16 bits of an IEEE binary32):
 *   W      [N][K]     uint16 BF16 bit patterns, row-major, K % 32 == 0
 *   codes  [N][K/2]   byte j of a row = code(2j) | code(2j+1) << 4
 *   scales [N][K/32]  E8M0 byte: 2^(byte-127); 0xFF = NaN
 *   code   = sign<<3 | e1<<2 | e0<<1 | m  (E2M1, exponent bias 1)
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>

#define MX_BLOCK 32

/* ---- BF16 helpers (own, not shared with the CUDA side) ------------------ */

static double bf16_bits_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f; /* binary32 -> binary64 is exact */
}

static int bf16_bits_nonfinite(uint16_t b)
{
    return (b & 0x7F80u) == 0x7F80u; /* exponent field all ones: Inf or NaN */
}

/* ---- E2M1 ---------------------------------------------------------------- */

/* Value of the 3-bit magnitude field (e1 e0 m), exponent bias 1:
 *   e == 0: subnormal, m * 2^(1-1) * 1/2          -> 0, 0.5
 *   e >= 1: (1 + m/2) * 2^(e-1)                    -> 1, 1.5, 2, 3, 4, 6      */
static double e2m1_magnitude(unsigned mag3)
{
    unsigned e = (mag3 >> 1) & 3u, m = mag3 & 1u;
    if (e == 0)
        return 0.5 * (double)m;
    return ldexp(1.0 + 0.5 * (double)m, (int)e - 1);
}

/* Round a non-negative real r to E2M1 the way a floating-point format rounds:
 * pick the binade, divide by the spacing of representable numbers in that
 * binade, round to the nearest integer with ties to even, multiply back.
 * Results above the largest normal (6) are clamped to it (Sec. III-D-3).
 * Returns the 3-bit magnitude code.                                         */
static unsigned e2m1_round_magnitude(double r)
{
    double spacing, q, val;
    unsigned code;

    if (!(r < 8.0)) /* also catches anything absurdly large: clamp */
        return 7u;
    if (r < 1.0)
        spacing = 0.5; /* subnormal range shares the spacing of [1,2) */
    else if (r < 2.0)
        spacing = 0.5;
    else if (r < 4.0)
        spacing = 1.0;
    else
        spacing = 2.0;
    q = nearbyint(r / spacing); /* default rounding mode: nearest, ties to even */
    val = q * spacing;          /* may have carried into the next binade       */
    if (val > 6.0)
        val = 6.0; /* clamp to max normal */
    /* name the representable value */
    if (val == 0.0) code = 0u;
    else if (val == 0.5) code = 1u;
    else if (val == 1.0) code = 2u;
    else if (val == 1.5) code = 3u;
    else if (val == 2.0) code = 4u;
    else if (val == 3.0) code = 5u;
    else if (val == 4.0) code = 6u;
    else code = 7u; /* 6.0 */
    return code;
}

/* ---- direct cast (Sec. III-D-3) ------------------------------------------ */

/* One block of 32 BF16 values -> 32 codes + one scale byte.
 * Returns 1 if the block held an Inf/NaN (reading: such a block gets scale
 * 0xFF and all-zero codes), else 0.                                          */
static int quantize_block(const uint16_t *v, uint8_t code_out[MX_BLOCK], uint8_t *scale_out)
{
    int k, shared_exp;
    double amax = 0.0;

    for (k = 0; k < MX_BLOCK; ++k) {
        if (bf16_bits_nonfinite(v[k])) {
            for (int j = 0; j < MX_BLOCK; ++j) code_out[j] = 0;
            *scale_out = 0xFF;
            return 1;
        }
    }
    /* step (i): X = 2^floor(log2(max|v|)) / 2^emax, emax = 2 because the
     * largest power of two E2M1 can hold is 4 (its largest normal is 6).     */
    for (k = 0; k < MX_BLOCK; ++k) {
        double a = fabs(bf16_bits_to_double(v[k]));
        if (a > amax) amax = a;
    }
    if (amax == 0.0) {
        shared_exp = -127; /* reading: an all-zero block takes the smallest scale */
    } else {
        int e;
        (void)frexp(amax, &e);   /* amax = f * 2^e, f in [0.5,1)  => floor(log2 amax) = e-1 */
        shared_exp = (e - 1) - 2;
        if (shared_exp < -127) shared_exp = -127; /* E8M0 cannot go lower */
        if (shared_exp > 127) shared_exp = 127;   /* never reached from BF16 */
    }
    *scale_out = (uint8_t)(shared_exp + 127);

    /* step (ii): v / X -> E2M1, round to nearest even, clamp, keep the sign  */
    for (k = 0; k < MX_BLOCK; ++k) {
        double x = bf16_bits_to_double(v[k]);
        double r = ldexp(fabs(x), -shared_exp); /* exact: power-of-two scaling in binary64 */
        unsigned sign = (v[k] >> 15) & 1u;      /* the sign bit itself, so -0 stays -0     */
        code_out[k] = (uint8_t)((sign << 3) | e2m1_round_magnitude(r));
    }
    return 0;
}

/* W[N][K] BF16 bits -> codes[N][K/2], scales[N][K/32].
 * Returns the number of blocks that contained Inf/NaN.                       */
int64_t oq_quantize(const uint16_t *W, int64_t N, int64_t K, uint8_t *codes, uint8_t *scales)
{
    int64_t bad = 0;
    int64_t nblk = K / MX_BLOCK;
#pragma omp parallel for reduction(+ : bad) schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t j = 0; j < nblk; ++j) {
            uint8_t c[MX_BLOCK];
            uint8_t s;
            bad += quantize_block(W + n * K + j * MX_BLOCK, c, &s);
            scales[n * nblk + j] = s;
            for (int i = 0; i < MX_BLOCK / 2; ++i)
                codes[n * (K / 2) + j * (MX_BLOCK / 2) + i] = (uint8_t)(c[2 * i] | (c[2 * i + 1] << 4));
        }
    }
    return bad;
}

/* ---- dequantisation ------------------------------------------------------- */

static double dequant_one(unsigned code4, uint8_t scale_byte)
{
    double mag, s;
    if (scale_byte == 0xFF)
        return NAN;
    mag = e2m1_magnitude(code4 & 7u);
    s = ldexp(1.0, (int)scale_byte - 127);
    return (code4 & 8u) ? -(mag * s) : (mag * s);
}

static unsigned code_at(const uint8_t *codes_row, int64_t k)
{
    uint8_t byte = codes_row[k >> 1];
    return (k & 1) ? (unsigned)(byte >> 4) : (unsigned)(byte & 0x0F);
}

/* codes/scales -> out[N][K] doubles (each exactly the represented value) */
void oq_dequantize(const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K, double *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k)
            out[n * K + k] = dequant_one(code_at(codes + n * (K / 2), k), scales[n * (K / MX_BLOCK) + k / MX_BLOCK]);
}

/* ---- weight-only-quantised linear layer ---------------------------------- */

/* y64[m][n] = sum_k x[m][k] * w^[n][k]   and   A[m][n] = sum_k |x[m][k] * w^[n][k]|
 * in binary64, plain k order.  A may be NULL.                                 */
void oq_linear(const uint16_t *X, int64_t M, const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K,
               double *y64, double *A)
{
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        const uint8_t *crow = codes + n * (K / 2);
        const uint8_t *srow = scales + n * (K / MX_BLOCK);
        for (int64_t m = 0; m < M; ++m) {
            double acc = 0.0, accabs = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double w = dequant_one(code_at(crow, k), srow[k / MX_BLOCK]);
                double p = bf16_bits_to_double(X[m * K + k]) * w;
                acc += p;
                accabs += fabs(p);
            }
            y64[m * N + n] = acc;
            if (A) A[m * N + n] = accabs;
        }
    }
}

/* Same sum for a chosen list of output rows only (used to check full-size GPU
 * outputs on a sample): rows[i] in [0,N), y64/A are [M][nrows].              */
void oq_linear_rows(const uint16_t *X, int64_t M, const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K,
                    const int64_t *rows, int64_t nrows, double *y64, double *A)
{
    (void)N;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < nrows; ++i) {
        int64_t n = rows[i];
        const uint8_t *crow = codes + n * (K / 2);
        const uint8_t *srow = scales + n * (K / MX_BLOCK);
        for (int64_t m = 0; m < M; ++m) {
            double acc = 0.0, accabs = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double w = dequant_one(code_at(crow, k), srow[k / MX_BLOCK]);
                double p = bf16_bits_to_double(X[m * K + k]) * w;
                acc += p;
                accabs += fabs(p);
            }
            y64[m * nrows + i] = acc;
            if (A) A[m * nrows + i] = accabs;
        }
    }
}

/* ---- greedy verification (Sec. III-A, III-B) ------------------------------ */

static double logit_at(const void *logits, int is_bf16, int64_t i)
{
    if (is_bf16)
        return bf16_bits_to_double(((const uint16_t *)logits)[i]);
    return (double)((const float *)logits)[i];
}

/* out[r] = index of the largest entry of row r, scanning upward and replacing
 * only on strictly greater: the lowest index wins ties and a NaN never wins
 * (a row with nothing above -inf yields 0).                                  */
void oq_argmax(const void *logits, int is_bf16, int64_t rows, int64_t V, int32_t *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        double best = -INFINITY;
        int64_t idx = 0;
        for (int64_t v = 0; v < V; ++v) {
            double x = logit_at(logits, is_bf16, r * V + v);
            if (x > best) {
                best = x;
                idx = v;
            }
        }
        out[r] = (int32_t)idx;
    }
}

/* draft[B][T], verifier[B][R] (R == T or T+1).
 * accept_len[b] = first i with draft[b][i] != verifier[b][i], else T.
 * next_token[b] = verifier[b][G] if G < R else -1.                          */
void oq_greedy_accept_tokens(const int32_t *draft, const int32_t *verifier, int64_t B, int64_t T, int64_t R,
                             int32_t *accept_len, int32_t *next_token)
{
    for (int64_t b = 0; b < B; ++b) {
        int64_t G = T;
        for (int64_t i = 0; i < T; ++i) {
            /* row i of the verifier is the target's own choice for the slot
             * draft token i fills; a draft position with no verifier row
             * cannot be confirmed                                           */
            if (i >= R || draft[b * T + i] != verifier[b * R + i]) {
                G = i;
                break;
            }
        }
        accept_len[b] = (int32_t)G;
        next_token[b] = (G < R) ? verifier[b * R + G] : -1;
    }
}

/* logits [B][R][V] -> accept_len[B], next_token[B]; verifier_out may be NULL */
void oq_greedy_accept(const void *logits, int is_bf16, int64_t B, int64_t R, int64_t V, const int32_t *draft,
                      int64_t T, int32_t *verifier_scratch, int32_t *accept_len, int32_t *next_token)
{
    oq_argmax(logits, is_bf16, B * R, V, verifier_scratch);
    oq_greedy_accept_tokens(draft, verifier_scratch, B, T, R, accept_len, next_token);
}

/* how many threads the parallel loops above will use */
#ifdef _OPENMP
#include <omp.h>
int oq_threads(void) { return omp_get_max_threads(); }
void oq_set_threads(int n) { if (n > 0) omp_set_num_threads(n); }
#else
int oq_threads(void) { return 1; }
void oq_set_threads(int n) { (void)n; }
#endif
