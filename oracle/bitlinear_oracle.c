/*
 * BitLinear forward (BitNet b1.58) -- CPU ORACLE.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition of what the BitLinear forward
 * computes.  It exists so that tests can compare the CUDA library against it
 * and so that the benchmark can time a CPU baseline.  Nothing in the product
 * path may call it, and it shares no code, header, table or constant with the
 * CUDA kernels.
 *
 * What follows the paper, and where:
 *   - absmean weight quantisation  ............ Section 2, Eq. 1, Eq. 2, Eq. 3
 *   - per-token symmetric activation quantisation to [-Qb, Qb], no zero point
 *     ........................................... Section 2, paragraph after Eq. 3
 *   - integer-only matrix product ................ Section 1 ("only involves integer addition")
 *   - 2-bit storage of ternary weights ........... Section 3, "Memory and Latency"
 *
 * Readings taken where the paper is silent (each repeated next to its code):
 *   R1  eps enters additively in Eq. 1 and is a caller argument.
 *   R2  gamma (Eq. 3) is the order-free EXACT sum of |W| in 2^-64 fixed point
 *       (each term truncated to a multiple of 2^-64), divided in double.
 *   R3  round() is round-half-to-even.
 *   R4  Qb = 127; clip to [-127, 127].
 *   R5  beta_t = max_k |x_tk| over the K features of token t.
 *   R6  beta_t is clamped below by 1e-5f; s_t = 127/beta_t is formed once and
 *       every element takes ONE fp32 multiply before rounding.
 *   R7  dequantisation scale is (gamma*beta_t)/127 with the plain gamma.
 *   R8  output is round-to-nearest-even bfloat16 of float(acc)*scale.
 *   R9  storage layout of the 2-bit codes (see oracle_pack_weights).
 *   R10 one gamma per weight matrix.
 *   T1  a second storage format with five weights per byte in base 3 (see oracle_pack_weights_trits).
 *
 * Parity pins (tests/test_oracle_pins.py): hand-worked cases for Eq. 1-3 and
 * the activation quantiser including rounding ties, closed-form Gaussian
 * statistics, textbook int32 matmul via numpy, brute-force double-precision
 * matmul of the dequantised operands, algebraic invariants, exactness of gamma
 * against math.fsum, pack/unpack round trip, and a pure-Python restatement
 * (oracle/np_restatement.py) on small shapes.
 * Parity unpinned: the bf16 output tolerance itself (1e-2 rel / 1e-3 abs) is
 * not fixed by the paper.
 *
 * Build for parity:  gcc -O2 -fno-fast-math -ffp-contract=off -shared -fPIC
 * Build for timing:  same source with -O3 -fopenmp (outer loops only).
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <fenv.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG -1
#define ORACLE_ERR_RANGE -8 /* non-finite value or |w| >= 2^24 */

#define QB 127          /* R4 */
#define BETA_FLOOR 1e-5f /* R6 */

/* ---------- bfloat16 helpers (bf16 = upper 16 bits of an IEEE fp32) ---------- */

static float bf16_to_float(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* R8: round-to-nearest-even from fp32 to bf16 (finite inputs). */
static uint16_t float_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    uint32_t lower = u & 0xFFFFu;
    uint32_t upper = u >> 16;
    if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u)))
        upper += 1u;
    return (uint16_t)upper;
}

/* ---------- Eq. 3 with reading R2: exact sum of |W| ---------- */

/*
 * floor(|v| * 2^64) as an unsigned 128-bit integer.  An fp32 magnitude is
 * sig * 2^(e-150) with a 24-bit integer significand, so the scaled value is
 * sig * 2^(e-86): a left shift when e >= 86, a truncating right shift below.
 * Caller guarantees e < 151, i.e. |v| < 2^24.
 */
static unsigned __int128 fix64_of_magnitude(uint32_t magnitude_bits)
{
    uint32_t e = magnitude_bits >> 23;
    uint32_t frac = magnitude_bits & 0x7FFFFFu;
    uint32_t sig = e ? (frac | 0x800000u) : frac; /* subnormals: no hidden bit */
    int shift = (int)(e ? e : 1u) - 86;
    if (shift >= 0)
        return ((unsigned __int128)sig) << shift;
    if (-shift >= 24)
        return 0;
    return (unsigned __int128)(sig >> (-shift));
}

int oracle_absmean(const float *W, int64_t N, int64_t K, float *gamma)
{
    if (!W || !gamma || N <= 0 || K <= 0)
        return ORACLE_ERR_ARG;
    unsigned __int128 total = 0;
    for (int64_t i = 0; i < N * K; ++i) {
        uint32_t u;
        memcpy(&u, &W[i], sizeof u);
        u &= 0x7FFFFFFFu; /* |W_ij| */
        if ((u >> 23) >= 151u)
            return ORACLE_ERR_RANGE;
        total += fix64_of_magnitude(u);
    }
    uint64_t hi = (uint64_t)(total >> 64);
    uint64_t lo = (uint64_t)total;
    double sum = ((double)hi * 18446744073709551616.0 + (double)lo) * (1.0 / 18446744073709551616.0);
    double mean = sum / (double)(N * K);
    *gamma = (float)mean;
    return ORACLE_OK;
}

/* ---------- Eq. 1 and Eq. 2 ---------- */

/* Eq. 2: RoundClip(x, a, b) = max(a, min(b, round(x))), round = half-to-even (R3). */
static int round_clip(float x, int a, int b)
{
    float r = rintf(x); /* FE_TONEAREST: ties to even */
    if (r != r) return 0; /* 0/0 (all-zero matrix with eps = 0): the weight is 0 */
    if (r < (float)a) return a;
    if (r > (float)b) return b;
    return (int)r;
}

/*
 * Eq. 1: W~ = RoundClip(W / (gamma + eps), -1, 1), gamma from Eq. 3.
 * T receives the ternary values row-major [N][K].
 */
int oracle_quantize_weights(const float *W, int64_t N, int64_t K, float eps, int8_t *T, float *gamma)
{
    if (!T)
        return ORACLE_ERR_ARG;
    int rc = oracle_absmean(W, N, K, gamma);
    if (rc != ORACLE_OK)
        return rc;
    float denom = *gamma + eps; /* R1 */
#ifdef _OPENMP
#pragma omp parallel for
#endif
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k)
            T[n * K + k] = (int8_t)round_clip(W[n * K + k] / denom, -1, 1);
    return ORACLE_OK;
}

/* ---------- R9: 2-bit storage ---------- */

static int64_t col_tiles(int64_t K) { return (K + 63) / 64; }
static int64_t row_blocks(int64_t N) { return (N + 63) / 64; }

int64_t oracle_packed_bytes(int64_t N, int64_t K)
{
    if (N <= 0 || K <= 0 || (N % 16) != 0)
        return -1;
    return row_blocks(N) * col_tiles(K) * 1024;
}

/*
 * Where weight (n, k) lives.  The matrix is cut into tiles of 64 rows by 64
 * columns, 1024 bytes each, stored one after another with the column-tile index
 * running fastest.  One BYTE holds the codes of four rows at the same column.
 * Within a tile, with r = n mod 64 and c = k mod 64, split
 *     r = 16*f + 8*h + g        (f = 0..3, h = 0..1, g = 0..7)
 *     c = 16*tq + 8*s + 4*hi + b  (tq = 0..3, s = 0..1, hi = 0..1, b = 0..3)
 * and the code occupies bits [2*f, 2*f + 1] of byte
 *     512*s + 16*(4*g + tq) + 4*(2*hi + h) + b
 * of the tile.  The stored code is t + 1, so it is 0, 1 or 2; 3 never appears.
 * Rows N..(multiple of 64) and columns K..(multiple of 64) hold code 1 (weight
 * zero).
 */
static void locate(int64_t n, int64_t k, int64_t KB, int64_t *byte_index, int *bit)
{
    int64_t tile = (n / 64) * KB + (k / 64);
    int r = (int)(n % 64), c = (int)(k % 64);
    int f = r / 16, h = (r % 16) / 8, g = r % 8;
    int tq = c / 16, s = (c % 16) / 8, hi = (c % 8) / 4, b = c % 4;
    *byte_index = tile * 1024 + 512 * s + 16 * (4 * g + tq) + 4 * (2 * hi + h) + b;
    *bit = 2 * f;
}

int oracle_pack_weights(const int8_t *T, int64_t N, int64_t K, uint8_t *packed)
{
    if (!T || !packed || N <= 0 || K <= 0 || (N % 16) != 0)
        return ORACLE_ERR_ARG;
    int64_t KB = col_tiles(K), NB = row_blocks(N);
    memset(packed, 0, (size_t)(NB * KB * 1024));
    for (int64_t n = 0; n < NB * 64; ++n) {
        for (int64_t k = 0; k < KB * 64; ++k) {
            int t = (n < N && k < K) ? T[n * K + k] : 0;
            if (t < -1 || t > 1)
                return ORACLE_ERR_ARG;
            uint32_t code = (uint32_t)(t + 1);
            int64_t at;
            int bit;
            locate(n, k, KB, &at, &bit);
            packed[at] |= (uint8_t)(code << bit);
        }
    }
    return ORACLE_OK;
}

int oracle_unpack_weights(const uint8_t *packed, int64_t N, int64_t K, int8_t *T)
{
    if (!T || !packed || N <= 0 || K <= 0 || (N % 16) != 0)
        return ORACLE_ERR_ARG;
    int64_t KB = col_tiles(K);
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t k = 0; k < K; ++k) {
            int64_t at;
            int bit;
            locate(n, k, KB, &at, &bit);
            int code = (packed[at] >> bit) & 3;
            if (code == 3)
                return ORACLE_ERR_ARG;
            T[n * K + k] = (int8_t)(code - 1);
        }
    }
    return ORACLE_OK;
}

/* ---------- base-3 storage: five weights per byte (1.6 bits per weight) ----------
 *
 * A ternary weight carries log2 3 = 1.58 bits (the paper's title; Section 1), and the paper notes that its 2-bit kernel
 * leaves room (Section 3, "Memory and Latency").  Reading T1: five codes c = t + 1 in {0, 1, 2} share one byte as the
 * base-3 number c0 + 3 c1 + 9 c2 + 27 c3 + 81 c4 (0..242).  The matrix is cut into tiles of 80 rows by 64 columns, 1024
 * bytes each, stored one after another with the column-tile index running fastest.  Within a tile, with r = n mod 80
 * and c = k mod 64, split
 *     r = 16*f + 8*h + g          (f = 0..4, h = 0..1, g = 0..7)
 *     c = 16*tq + 8*s + 4*hi + b  (tq = 0..3, s = 0..1, hi = 0..1, b = 0..3)
 * and the weight is digit f of byte 512*s + 16*(4*g + tq) + 4*(2*hi + h) + b of the tile (the byte positions of the
 * 2-bit format; the five rows of a byte are 16 apart).  Rows N..(multiple of 80) and columns K..(multiple of 64) hold
 * code 1 (weight zero), so a byte of padding is 121.
 */
static int64_t trit_row_blocks(int64_t N) { return (N + 79) / 80; }

int64_t oracle_packed_bytes_trits(int64_t N, int64_t K)
{
    if (N <= 0 || K <= 0 || (N % 16) != 0)
        return -1;
    return trit_row_blocks(N) * col_tiles(K) * 1024;
}

static const int POW3[5] = {1, 3, 9, 27, 81};

static void locate_trit(int64_t n, int64_t k, int64_t KB, int64_t *byte_index, int *digit)
{
    int64_t tile = (n / 80) * KB + (k / 64);
    int r = (int)(n % 80), c = (int)(k % 64);
    int f = r / 16, h = (r % 16) / 8, g = r % 8;
    int tq = c / 16, s = (c % 16) / 8, hi = (c % 8) / 4, b = c % 4;
    *byte_index = tile * 1024 + 512 * s + 16 * (4 * g + tq) + 4 * (2 * hi + h) + b;
    *digit = f;
}

int oracle_pack_weights_trits(const int8_t *T, int64_t N, int64_t K, uint8_t *packed)
{
    if (!T || !packed || N <= 0 || K <= 0 || (N % 16) != 0)
        return ORACLE_ERR_ARG;
    int64_t KB = col_tiles(K), NB = trit_row_blocks(N);
    memset(packed, 0, (size_t)(NB * KB * 1024));
    for (int64_t n = 0; n < NB * 80; ++n) {
        for (int64_t k = 0; k < KB * 64; ++k) {
            int t = (n < N && k < K) ? T[n * K + k] : 0;
            if (t < -1 || t > 1)
                return ORACLE_ERR_ARG;
            int64_t at;
            int digit;
            locate_trit(n, k, KB, &at, &digit);
            packed[at] = (uint8_t)(packed[at] + (t + 1) * POW3[digit]);
        }
    }
    return ORACLE_OK;
}

int oracle_unpack_weights_trits(const uint8_t *packed, int64_t N, int64_t K, int8_t *T)
{
    if (!T || !packed || N <= 0 || K <= 0 || (N % 16) != 0)
        return ORACLE_ERR_ARG;
    int64_t KB = col_tiles(K);
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t k = 0; k < K; ++k) {
            int64_t at;
            int digit;
            locate_trit(n, k, KB, &at, &digit);
            if (packed[at] > 242)
                return ORACLE_ERR_ARG;
            T[n * K + k] = (int8_t)((packed[at] / POW3[digit]) % 3 - 1);
        }
    }
    return ORACLE_OK;
}

/* ---------- activation quantiser (Section 2, after Eq. 3; R4, R5, R6) ---------- */

int oracle_quantize_acts(const uint16_t *X_bf16, int64_t M, int64_t K,
                         int8_t *Xq, float *beta, int32_t *rowsum)
{
    if (!X_bf16 || !Xq || !beta || !rowsum || M < 0 || K <= 0)
        return ORACLE_ERR_ARG;
#ifdef _OPENMP
#pragma omp parallel for
#endif
    for (int64_t t = 0; t < M; ++t) {
        float amax = 0.0f;
        for (int64_t k = 0; k < K; ++k) {
            float a = fabsf(bf16_to_float(X_bf16[t * K + k]));
            if (a > amax) amax = a;
        }
        float b = amax > BETA_FLOOR ? amax : BETA_FLOOR; /* R6 */
        float s = (float)QB / b;                          /* one IEEE divide per token */
        int32_t sum = 0;
        for (int64_t k = 0; k < K; ++k) {
            float scaled = bf16_to_float(X_bf16[t * K + k]) * s; /* one multiply per element */
            int q = round_clip(scaled, -QB, QB);
            Xq[t * K + k] = (int8_t)q;
            sum += q;
        }
        beta[t] = b;
        rowsum[t] = sum;
    }
    return ORACLE_OK;
}

/* ---------- RMSNorm in front of the activation quantiser ----------
 *
 * The paper builds its models from "LLaMA-alike components", RMSNorm among them (Section 2, "LLaMA-alike
 * Components"), and gives no formula for it: what stands in front of a BitLinear is taken here as the textbook
 * RMSNorm, x_k = h_k / sqrt(mean_k(h_k^2) + eps_n) * g_k, followed by the activation quantiser above.
 * Because the normalised values decide integers, the arithmetic is fixed (readings, not the paper's):
 *   N1  the sum of squares is EXACT integer arithmetic, hence order-free: with E the exponent field of the
 *       token's largest |h_k| (a bfloat16: 8-bit exponent field e, 8-bit significand m with its hidden bit; e = 0
 *       counts as 1 without hidden bit), h_k^2 = m_k^2 * 4^(e_k - 134), and the token's sum is
 *           S = sum_k floor( m_k^2 * 2^30 / 4^(E - e_k) )        (terms with E - e_k > 23 are 0)
 *       in units of 4^(E - 134) * 2^-30: every term is below 2^46, so S < 2^63 for K <= 2^17.  What a term loses is
 *       below 2^-44 of the largest square, far below fp32 resolution, and the sum does not depend on the scale
 *       of h.  Infinities and NaNs are refused;
 *   N2  mean = (float)( (double)S / (double)K * 2^(2E - 298) ) (the conversion of S rounds to nearest even, the power
 *       of two is exact); r = 1.0f / sqrtf(max(mean + eps_n, 2^-126)): fp32 add, IEEE square root, IEEE divide
 *       (the floor, the smallest normal fp32, only matters for an all-zero token or one whose mean square
 *       underflows fp32 with eps_n = 0: r stays finite there);
 *   N3  x_k = (h_k * r) * g_k: two fp32 multiplications in this order, no fused multiply-add;
 *   N4  the quantiser then works on the fp32 x_k exactly as on bfloat16 inputs (R4, R5, R6).
 * Parity pins (tests/test_oracle_pins.py): a hand case, agreement of x with a double-precision evaluation of the
 * formula and with torch's rms_norm, scale invariance for eps_n = 0, reduction to the plain quantiser.
 */
/* N1, N2 for one token of K bfloat16 values: *mean = the fp32 mean square.  Returns 0, or 1 if the token holds an
 * infinity or a NaN. */
static int token_mean_square(const uint16_t *h, int64_t K, float *mean)
{
    /* N1: exponent field of the largest magnitude, then the integer sum */
    unsigned E = 0;
    for (int64_t k = 0; k < K; ++k) {
        unsigned e = (h[k] >> 7) & 0xFFu;
        if (e == 255u) return 1;
        if (e < 1u) e = 1u;
        if (e > E) E = e;
    }
    uint64_t S = 0;
    for (int64_t k = 0; k < K; ++k) {
        unsigned bits = h[k];
        unsigned e = (bits >> 7) & 0xFFu;
        uint64_t m = bits & 0x7Fu;
        if (e) m |= 0x80u; else e = 1u;
        unsigned twice = 2u * (E - e);
        if (twice <= 46u) S += ((m * m) << 30) >> twice;
    }
    *mean = (float)(ldexp((double)S / (double)K, 2 * (int)E - 298)); /* N2 */
    return 0;
}

/* The mean square alone, per token (for the pins: compared with the exactly rounded mean of the exact squares). */
int oracle_rmsnorm_mean_square(const uint16_t *H_bf16, int64_t M, int64_t K, float *mean)
{
    if (!H_bf16 || !mean || M < 0 || K <= 0)
        return ORACLE_ERR_ARG;
    for (int64_t t = 0; t < M; ++t)
        if (token_mean_square(H_bf16 + t * K, K, &mean[t]))
            return ORACLE_ERR_RANGE;
    return ORACLE_OK;
}

int oracle_rmsnorm_quantize_acts(const uint16_t *H_bf16, const float *gain, float eps_n, int64_t M, int64_t K,
                                 int8_t *Xq, float *beta, int32_t *rowsum, float *x_out /* may be NULL: [M][K] */)
{
    if (!H_bf16 || !gain || !Xq || !beta || !rowsum || M < 0 || K <= 0 || !(eps_n >= 0.0f))
        return ORACLE_ERR_ARG;
    int status = ORACLE_OK;
#ifdef _OPENMP
#pragma omp parallel for
#endif
    for (int64_t t = 0; t < M; ++t) {
        float mean;
        if (token_mean_square(H_bf16 + t * K, K, &mean)) {
#ifdef _OPENMP
#pragma omp critical
#endif
            status = ORACLE_ERR_RANGE;
            continue;
        }
        float d = mean + eps_n;
        if (!(d > 1.17549435e-38f)) d = 1.17549435e-38f; /* an all-zero or vanishing token: r stays finite */
        float r = 1.0f / sqrtf(d);
        float amax = 0.0f;
        for (int64_t k = 0; k < K; ++k) {
            float x = (bf16_to_float(H_bf16[t * K + k]) * r) * gain[k]; /* N3 */
            if (x_out) x_out[t * K + k] = x;
            float a = fabsf(x);
            if (a > amax) amax = a;
        }
        float b = amax > BETA_FLOOR ? amax : BETA_FLOOR; /* R6 */
        float s = (float)QB / b;
        int32_t acc = 0;
        for (int64_t k = 0; k < K; ++k) {
            float x = (bf16_to_float(H_bf16[t * K + k]) * r) * gain[k];
            int q = round_clip(x * s, -QB, QB);
            Xq[t * K + k] = (int8_t)q;
            acc += q;
        }
        beta[t] = b;
        rowsum[t] = acc;
    }
    return status;
}

/* ---------- SwiGLU in front of the activation quantiser ----------
 *
 * SwiGLU is another of the paper's "LLaMA-alike components" (Section 2), again without a formula: the input of the
 * down projection is taken here as the textbook h_k = silu(g_k) * u_k, silu(g) = g * sigmoid(g) = g / (1 + e^-g), of
 * the gate and up projections' outputs g and u (bfloat16, as BitLinear writes them), followed by the activation
 * quantiser above.  The values decide integers, so the arithmetic is fixed in fp32 (readings, not the paper's):
 *   G1  e^t for t = -g by range reduction and a Taylor polynomial, every step one IEEE fp32 operation:
 *           z = t * log2(e)         (log2(e) as fp32),           n = z rounded to the nearest integer, ties to even,
 *           r = fma(n, -ln2_hi, t), r = fma(n, -ln2_lo, r)       (ln 2 = ln2_hi + ln2_lo, ln2_hi with 9 trailing zero bits),
 *           p = 1 + r + r^2/2 + ... + r^7/5040                   (Horner's scheme, seven fused multiply-adds from the top),
 *           e^t = p * 2^n                                        (exact: t is kept within [-87, 87], so 2^n and the
 *                                                                 product are normal numbers);
 *   G2  sigmoid(g) = 1 / (1 + e^-g): one fp32 addition and one IEEE division; for g > 87 it is 1, for g < -87 it
 *       is 0 (the true value is within 2^-125 of that);
 *   G3  h_k = (g_k * sigmoid(g_k)) * u_k: two fp32 multiplications in this order;
 *   G4  the quantiser then works on the fp32 h_k exactly as on bfloat16 inputs (R4, R5, R6).  Infinities and NaNs in
 *       g or u, and a product h_k that overflows fp32, are refused.
 * Parity pins (tests/test_oracle_pins.py): agreement of h with a double-precision evaluation of the definition and
 * with torch's silu, hand cases (g = 0, the saturated ends), reduction to the plain quantiser for saturated gates,
 * odd symmetry in u.
 */
static float sigmoid_f32(float g)
{
    float t = -g;
    if (t > 87.0f) return 0.0f;
    if (t < -87.0f) return 1.0f;
    float z = t * 1.44269502162933349609375f;                 /* log2(e) rounded to fp32 */
    float n = rintf(z);                                       /* default rounding mode: ties to even */
    float r = fmaf(n, -0.693145751953125f, t);                /* ln2_hi */
    r = fmaf(n, -1.42860676533018704503775e-06f, r);          /* ln2_lo = fp32(ln 2 - ln2_hi) */
    float p = fmaf(r, 1.0f / 5040.0f, 1.0f / 720.0f);
    p = fmaf(p, r, 1.0f / 120.0f);
    p = fmaf(p, r, 1.0f / 24.0f);
    p = fmaf(p, r, 1.0f / 6.0f);
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    float e = ldexpf(p, (int)n);
    return 1.0f / (1.0f + e);
}

int oracle_swiglu_quantize_acts(const uint16_t *G_bf16, const uint16_t *U_bf16, int64_t M, int64_t K,
                                int8_t *Xq, float *beta, int32_t *rowsum, float *h_out /* may be NULL: [M][K] */)
{
    if (!G_bf16 || !U_bf16 || !Xq || !beta || !rowsum || M < 0 || K <= 0)
        return ORACLE_ERR_ARG;
    int status = ORACLE_OK;
#ifdef _OPENMP
#pragma omp parallel for
#endif
    for (int64_t t = 0; t < M; ++t) {
        float amax = 0.0f;
        int bad = 0;
        for (int64_t k = 0; k < K; ++k) {
            float g = bf16_to_float(G_bf16[t * K + k]), u = bf16_to_float(U_bf16[t * K + k]);
            if (!isfinite(g) || !isfinite(u)) {
                bad = 1;
                break;
            }
            float h = (g * sigmoid_f32(g)) * u; /* G3 */
            if (!isfinite(h)) {
                bad = 1;
                break;
            }
            if (h_out) h_out[t * K + k] = h;
            float a = fabsf(h);
            if (a > amax) amax = a;
        }
        if (bad) {
#ifdef _OPENMP
#pragma omp critical
#endif
            status = ORACLE_ERR_RANGE;
            continue;
        }
        float b = amax > BETA_FLOOR ? amax : BETA_FLOOR; /* R6 */
        float s = (float)QB / b;
        int32_t acc = 0;
        for (int64_t k = 0; k < K; ++k) {
            float g = bf16_to_float(G_bf16[t * K + k]), u = bf16_to_float(U_bf16[t * K + k]);
            float h = (g * sigmoid_f32(g)) * u;
            int q = round_clip(h * s, -QB, QB);
            Xq[t * K + k] = (int8_t)q;
            acc += q;
        }
        beta[t] = b;
        rowsum[t] = acc;
    }
    return status;
}

/* ---------- integer matrix product: the plain definition ---------- */

/* acc[t][n] = sum_k Xq[t][k] * T[n][k], exact in int32 (|acc| <= 127*K). */
int oracle_matmul_i32(const int8_t *Xq, const int8_t *T, int64_t M, int64_t K, int64_t N, int32_t *acc)
{
    if (!Xq || !T || !acc || M < 0 || K <= 0 || N <= 0)
        return ORACLE_ERR_ARG;
#ifdef _OPENMP
#pragma omp parallel for
#endif
    for (int64_t t = 0; t < M; ++t) {
        for (int64_t n = 0; n < N; ++n) {
            int32_t s = 0;
            for (int64_t k = 0; k < K; ++k)
                s += (int32_t)Xq[t * K + k] * (int32_t)T[n * K + k];
            acc[t * N + n] = s;
        }
    }
    return ORACLE_OK;
}

/* ---------- dequantisation (R7, R8) ---------- */

int oracle_dequant(const int32_t *acc, const float *beta, float gamma, int64_t M, int64_t N, uint16_t *Y_bf16)
{
    if (!acc || !beta || !Y_bf16 || M < 0 || N <= 0)
        return ORACLE_ERR_ARG;
#ifdef _OPENMP
#pragma omp parallel for
#endif
    for (int64_t t = 0; t < M; ++t) {
        float scale = (gamma * beta[t]) / (float)QB;
        for (int64_t n = 0; n < N; ++n)
            Y_bf16[t * N + n] = float_to_bf16_rne((float)acc[t * N + n] * scale);
    }
    return ORACLE_OK;
}

/* ---------- activations of fewer bits ----------
 *
 * The paper's outlook (Section 4, on long sequences) expects the activations to go from 8 bits to 4 bits or fewer.
 * The same forward with b-bit activations, 2 <= b <= 8 (readings, not the paper's):
 *   B1  Q_b = 2^(b-1) - 1 (b = 8: the 127 of R4; b = 4: 7), symmetric, no zero point;
 *   B2  beta, the one divide s = Q_b / beta per token, one multiply per element, round half to even and the clip
 *       to [-Q_b, Q_b] as in R5, R6; the codes are still delivered one per byte;
 *   B3  dequantisation by (gamma * beta_t) / Q_b, as in R7, R8.
 * Parity pins (tests/test_oracle_pins.py): a hand case with ties, equality with the 8-bit functions for b = 8, the
 * value set, the error bound |x - q * beta / Q_b| <= beta / (2 Q_b), the double-precision product.
 */
int oracle_quantize_acts_bits(const uint16_t *X_bf16, int64_t M, int64_t K, int bits,
                              int8_t *Xq, float *beta, int32_t *rowsum)
{
    if (!X_bf16 || !Xq || !beta || !rowsum || M < 0 || K <= 0 || bits < 2 || bits > 8)
        return ORACLE_ERR_ARG;
    const int qb = (1 << (bits - 1)) - 1; /* B1 */
#ifdef _OPENMP
#pragma omp parallel for
#endif
    for (int64_t t = 0; t < M; ++t) {
        float amax = 0.0f;
        for (int64_t k = 0; k < K; ++k) {
            float a = fabsf(bf16_to_float(X_bf16[t * K + k]));
            if (a > amax) amax = a;
        }
        float b = amax > BETA_FLOOR ? amax : BETA_FLOOR;
        float s = (float)qb / b; /* B2 */
        int32_t sum = 0;
        for (int64_t k = 0; k < K; ++k) {
            int q = round_clip(bf16_to_float(X_bf16[t * K + k]) * s, -qb, qb);
            Xq[t * K + k] = (int8_t)q;
            sum += q;
        }
        beta[t] = b;
        rowsum[t] = sum;
    }
    return ORACLE_OK;
}

int oracle_dequant_bits(const int32_t *acc, const float *beta, float gamma, int64_t M, int64_t N, int bits,
                        uint16_t *Y_bf16)
{
    if (!acc || !beta || !Y_bf16 || M < 0 || N <= 0 || bits < 2 || bits > 8)
        return ORACLE_ERR_ARG;
    const int qb = (1 << (bits - 1)) - 1;
#ifdef _OPENMP
#pragma omp parallel for
#endif
    for (int64_t t = 0; t < M; ++t) {
        float scale = (gamma * beta[t]) / (float)qb; /* B3 */
        for (int64_t n = 0; n < N; ++n)
            Y_bf16[t * N + n] = float_to_bf16_rne((float)acc[t * N + n] * scale);
    }
    return ORACLE_OK;
}

/* ---------- the whole forward for an already ternarised weight matrix ---------- */

/*
 * Y = dequant( quantize_acts(X) x T^T ).  Scratch buffers are the caller's:
 * Xq [M*K], beta [M], rowsum [M], acc [M*N].
 */
int oracle_forward(const int8_t *T, float gamma, const uint16_t *X_bf16,
                   int64_t M, int64_t K, int64_t N,
                   int8_t *Xq, float *beta, int32_t *rowsum, int32_t *acc, uint16_t *Y_bf16)
{
    int rc = oracle_quantize_acts(X_bf16, M, K, Xq, beta, rowsum);
    if (rc != ORACLE_OK) return rc;
    rc = oracle_matmul_i32(Xq, T, M, K, N, acc);
    if (rc != ORACLE_OK) return rc;
    return oracle_dequant(acc, beta, gamma, M, N, Y_bf16);
}

/* Timing aid (no arithmetic): how many threads the outer loops of the timing build use from now on. */
void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    extern void omp_set_num_threads(int);
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
