/*
 * tpq_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, scalar CPU statement of the low-bit tensor-parallel
 * synchronisation codec of "Towards Low-bit Communication for Tensor Parallel
 * LLM Inference" (arXiv 2411.07942).  It exists only so that the CUDA library
 * can be compared against something written independently from the paper; it
 * shares no code, header, table or constant generator with the CUDA path and
 * must never be called from it.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may load it.
 *
 * Each function follows the paper's steps in the paper's order:
 *   Section 3 "Calibration", Eq. (1)-(2)      -> tpqo_colminmax, tpqo_calibrate
 *   Section 3 (range R = 2 max(-m, M))        -> tpqo_ranges
 *   Section 3 "Selecting High Precision Features" -> tpqo_ranges (R-bar), tpqo_select
 *   Section 3 (symmetric Int4)                -> tpqo_params, tpqo_quantize_pack
 *   Figure 2 caption, Section 5 (all-gather + local reduction) -> tpqo_dequant_reduce
 *   Section 4 (k = floor(E/64), bits per value) -> tpqo_payload_bytes
 *
 * Where the paper is silent, the reading taken is stated at the function.
 * Pin status (what checks each function against something other than itself)
 * is listed in oracle/README.md; the Int4 grid constant (15 levels-minus-one),
 * the degenerate-range floor and the payload byte layout have no counterpart
 * in the paper and are "parity unpinned" by it: they are pinned only by
 * hand-derived fixtures and a second, independently written NumPy statement.
 *
 * Precision: BF16 values are 16-bit patterns widened exactly to binary32.
 * Every calibration / parameter / quantiser operation is ONE IEEE-754 binary32
 * operation, round-to-nearest-even, never contracted (compile with
 * -ffp-contract=off, no -ffast-math).  The reduction reference is binary64.
 *
 * BF16 arrays are uint16_t, row-major, with an explicit row stride in elements.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* code widths other than 4 (definitions below, beside their Int4 forms) */
void tpqo_params_b(const float *R, int64_t n, int bits, float *s, float *inv_s);
int64_t tpqo_lp_bytes_b(int64_t T, int64_t E, int64_t k, int bits);
int64_t tpqo_payload_bytes_b(int64_t T, int64_t E, int64_t k, int bits);
int tpqo_quantize_one_b(uint16_t x_bf16, float inv_s, int bits);
void tpqo_quantize_pack_b(const uint16_t *y, int64_t T, int64_t E, int64_t stride, const int32_t *hp_idx, int64_t k,
                          const float *inv_s, int bits, uint8_t *payload);
void tpqo_dequant_reduce_b(const uint8_t *const *payloads, int64_t N, int64_t T, int64_t E, const int32_t *hp_idx,
                           int64_t k, const float *s, int bits, double *ref64, float *chain32);
void tpqo_linear_bf16(const uint16_t *x, const uint16_t *w, int64_t T, int64_t K, int64_t E, uint16_t *y);
void tpqo_dequant_reduce_bias_b(const uint8_t *const *payloads, int64_t N, int64_t T, int64_t E, const int32_t *hp_idx,
                                int64_t k, const float *s, int bits, const float *bias, double *ref64, float *chain32);

#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------------------------------------------------------------- helpers */

static float bf16_widen(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* binary32 -> BF16, round-to-nearest-even (NaN stays NaN). */
static uint16_t bf16_round(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u)
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/* Total order on non-NaN BF16 patterns with -0 < +0, so that the column
 * minimum and maximum do not depend on the order in which rows are visited. */
static int32_t bf16_order(uint16_t h)
{
    int32_t mag = (int32_t)(h & 0x7fffu);
    return (h & 0x8000u) ? -mag - 1 : mag;
}

int tpqo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------ calibration */

/* Section 3, Eq. (1)-(2): min(Y_{.,j}) and max(Y_{.,j}) over the S tokens of
 * ONE sequence, for every feature j.  Outputs are binary32 (exact widenings). */
void tpqo_colminmax(const uint16_t *y, int64_t S, int64_t E, int64_t stride,
                    float *mn, float *mx)
{
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < E; ++j) {
        uint16_t lo = y[j], hi = y[j];
        for (int64_t t = 1; t < S; ++t) {
            uint16_t v = y[t * stride + j];
            if (bf16_order(v) < bf16_order(lo)) lo = v;
            if (bf16_order(v) > bf16_order(hi)) hi = v;
        }
        mn[j] = bf16_widen(lo);
        mx[j] = bf16_widen(hi);
    }
}

/* Section 3, Eq. (1)-(2) with the first-sequence rule: fold n_seq sequences of
 * one device into its running (m, M).  *count = sequences folded so far for
 * this device (0 means the next one is "the first sequence").
 * Reading where the paper is silent: state kept in binary32; the update is
 * evaluated literally left to right, c = fl(1 - gamma),
 * m <- fl( fl(c*m) + fl(gamma*min) ); one EMA step per sequence, sequences in
 * the order given. */
void tpqo_calibrate(float *m, float *M, int64_t *count,
                    const uint16_t *y, int64_t n_seq, int64_t S, int64_t E,
                    int64_t stride, float gamma)
{
    float *mn = (float *)malloc(sizeof(float) * (size_t)E);
    float *mx = (float *)malloc(sizeof(float) * (size_t)E);
    volatile float c = 1.0f - gamma;
    for (int64_t q = 0; q < n_seq; ++q) {
        tpqo_colminmax(y + q * S * stride, S, E, stride, mn, mx);
        if (*count == 0) {
            for (int64_t j = 0; j < E; ++j) { m[j] = mn[j]; M[j] = mx[j]; }
        } else {
            for (int64_t j = 0; j < E; ++j) {
                volatile float a = c * m[j];
                volatile float b = gamma * mn[j];
                m[j] = a + b;
                volatile float a2 = c * M[j];
                volatile float b2 = gamma * mx[j];
                M[j] = a2 + b2;
            }
        }
        *count += 1;
    }
    free(mn);
    free(mx);
}

/* Section 3: R^(i)_j = 2 max(-m^(i)_j, M^(i)_j) for every device i and feature
 * j, and the aggregated range R-bar_j = sum_i R^(i)_j.
 * Reading: binary32; the sum runs over devices in ascending order. */
void tpqo_ranges(const float *m, const float *M, int64_t N, int64_t E,
                 float *R, float *Rbar)
{
    for (int64_t i = 0; i < N; ++i)
        for (int64_t j = 0; j < E; ++j) {
            float a = -m[i * E + j];
            float b = M[i * E + j];
            float A = (a > b) ? a : b;
            R[i * E + j] = 2.0f * A;
        }
    for (int64_t j = 0; j < E; ++j) {
        volatile float acc = R[j];
        for (int64_t i = 1; i < N; ++i)
            acc = acc + R[i * E + j];
        Rbar[j] = acc;
    }
}

/* Section 3 "Selecting High Precision Features": the k features with the
 * largest R-bar_j; the set is the same for every sequence and device.
 * Reading: equal R-bar -> the lower feature index wins; the set is returned
 * sorted by feature index, ascending.  Written as k rounds of "take the best
 * remaining feature" so that it is visibly the definition of top-k. */
void tpqo_select(const float *Rbar, int64_t E, int64_t k, int32_t *hp_idx)
{
    unsigned char *taken = (unsigned char *)calloc((size_t)E, 1);
    for (int64_t r = 0; r < k; ++r) {
        int64_t best = -1;
        for (int64_t j = 0; j < E; ++j) {
            if (taken[j]) continue;
            if (best < 0 || Rbar[j] > Rbar[best]) best = j;  /* strict: lower j wins ties */
        }
        if (best < 0) break;          /* k > E: everything is taken already */
        taken[best] = 1;
    }
    int64_t n = 0;
    for (int64_t j = 0; j < E; ++j)
        if (taken[j]) hp_idx[n++] = (int32_t)j;
    free(taken);
}

/* Section 4: k = floor(E / 64). */
int64_t tpqo_default_k(int64_t E) { return E / 64; }

/* Symmetric Int4 parameters from the range (Section 3 says only "symmetric",
 * "Int4" and gives the range).  Reading: step s = R / (2^4 - 1), zero-point 0,
 * codes -8..7; a degenerate range is floored at s = 2^-23 so that 1/s is
 * finite; the quantiser multiplies by the stored reciprocal fl(1/s). */
void tpqo_params(const float *R, int64_t n, float *s, float *inv_s) { tpqo_params_b(R, n, 4, s, inv_s); }

/* The same at another code width b (Section 4 / Figure 3 evaluate the method "at lower and higher
 * precision"): step s = R / (2^b - 1), codes -2^(b-1) .. 2^(b-1)-1. */
void tpqo_params_b(const float *R, int64_t n, int bits, float *s, float *inv_s)
{
    const float floor_s = 1.1920928955078125e-07f; /* 2^-23 */
    const float levels = (float)((1 << bits) - 1);
    for (int64_t a = 0; a < n; ++a) {
        volatile float v = R[a] / levels;
        if (!(v >= floor_s)) v = floor_s;
        s[a] = v;
        volatile float r = 1.0f / v;
        inv_s[a] = r;
    }
}

/* ------------------------------------------------------- payload geometry */

/* Section 4 counts (E-k) 4-bit codes and k BF16 values per token.
 * Layout (ours; the paper gives only the count): one flat stream of 4-bit
 * codes for all T tokens in (token, slot) order, low nibble first, zero padded
 * to a multiple of 16 bytes; then T x k BF16 values (selected features
 * ascending).
 *
 * Slot order of the L = E-k codes of a token ("hole filling"): slot c holds
 * feature c, unless feature c is a selected one; the selected features below L
 * ("holes", ascending) are filled, in order, with the unselected features
 * at or above L (ascending).  There are equally many of both, so every slot is
 * used and most features keep their own index as slot. */
void tpqo_slot_order(int64_t E, const int32_t *hp_idx, int64_t k, int32_t *slot_feature /* [E-k] */)
{
    int64_t L = E - k;
    unsigned char *sel = (unsigned char *)calloc((size_t)(E > 0 ? E : 1), 1);
    for (int64_t h = 0; h < k; ++h) sel[hp_idx[h]] = 1;
    int64_t next_filler = L;          /* next candidate feature at or above L */
    for (int64_t c = 0; c < L; ++c) {
        if (!sel[c]) {
            slot_feature[c] = (int32_t)c;
        } else {
            while (sel[next_filler]) ++next_filler;
            slot_feature[c] = (int32_t)next_filler++;
        }
    }
    free(sel);
}

int64_t tpqo_lp_bytes(int64_t T, int64_t E, int64_t k) { return tpqo_lp_bytes_b(T, E, k, 4); }

int64_t tpqo_payload_bytes(int64_t T, int64_t E, int64_t k) { return tpqo_payload_bytes_b(T, E, k, 4); }

/* Width b: T(E-k) codes of b bits each, one flat little-endian bit stream (code p occupies bits
 * [p b, p b + b) of the stream, bit 0 = least significant bit of byte 0), padded to 16 bytes. */
int64_t tpqo_lp_bytes_b(int64_t T, int64_t E, int64_t k, int bits)
{
    int64_t nbits = T * (E - k) * bits;
    int64_t bytes = (nbits + 7) / 8;
    return (bytes + 15) / 16 * 16;
}

int64_t tpqo_payload_bytes_b(int64_t T, int64_t E, int64_t k, int bits)
{
    return tpqo_lp_bytes_b(T, E, k, bits) + 2 * T * k;
}

/* ------------------------------------------------------- compression C^(i) */

/* One symmetric Int4 code: u = fl(x * inv_s); clamp to [-8, 7]; round half to
 * even.  Two roundings (the product, then the integer), never a fused one. */
int tpqo_quantize_one(uint16_t x_bf16, float inv_s) { return tpqo_quantize_one_b(x_bf16, inv_s, 4); }

/* Width b: clamp to [-2^(b-1), 2^(b-1) - 1]. */
int tpqo_quantize_one_b(uint16_t x_bf16, float inv_s, int bits)
{
    const float lo = -(float)(1 << (bits - 1)), hi = (float)((1 << (bits - 1)) - 1);
    volatile float u = bf16_widen(x_bf16) * inv_s;
    float v = u;
    if (v < lo) v = lo;
    if (v > hi) v = hi;
    /* round half to even without relying on the floating-point environment */
    float fl = floorf(v);
    float d = v - fl;                 /* exact for |v| <= 128 */
    int q = (int)fl;
    if (d > 0.5f || (d == 0.5f && (q & 1))) q += 1;
    return q;
}

/* Section 3 + Figure 2: one device's [T][E] partial sums -> payload.
 * hp_idx: the k selected features, ascending; inv_s: this device's E
 * reciprocals (entries at selected features are unused). */
void tpqo_quantize_pack(const uint16_t *y, int64_t T, int64_t E, int64_t stride,
                        const int32_t *hp_idx, int64_t k, const float *inv_s,
                        uint8_t *payload)
{
    tpqo_quantize_pack_b(y, T, E, stride, hp_idx, k, inv_s, 4, payload);
}

void tpqo_quantize_pack_b(const uint16_t *y, int64_t T, int64_t E, int64_t stride,
                          const int32_t *hp_idx, int64_t k, const float *inv_s, int bits,
                          uint8_t *payload)
{
    int64_t L = E - k;
    int64_t lp_bytes = tpqo_lp_bytes_b(T, E, k, bits);
    const unsigned cmask = (1u << bits) - 1u;
    int32_t *lp_idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)(L > 0 ? L : 1));
    tpqo_slot_order(E, hp_idx, k, lp_idx);      /* lp_idx[c] = feature held by slot c */
    memset(payload, 0, (size_t)lp_bytes);
    uint16_t *hp = (uint16_t *)(payload + lp_bytes);
    /* rows are independent; 8 rows of codes always end on a byte boundary, so
     * the threads take 8 rows at a time and never share a byte. */
    int64_t rows_per_chunk = 8;
    int64_t n_chunks = (T + rows_per_chunk - 1) / rows_per_chunk;
#pragma omp parallel for schedule(static)
    for (int64_t ch = 0; ch < n_chunks; ++ch) {
        int64_t t0 = ch * rows_per_chunk;
        int64_t t1 = t0 + rows_per_chunk < T ? t0 + rows_per_chunk : T;
        for (int64_t t = t0; t < t1; ++t) {
            for (int64_t c = 0; c < L; ++c) {
                int64_t j = lp_idx[c];
                int q = tpqo_quantize_one_b(y[t * stride + j], inv_s[j], bits);
                int64_t bit = (t * L + c) * bits;          /* first bit of the code in the stream */
                unsigned u = ((unsigned)q & cmask) << (bit & 7);   /* at most 15 bits: spans <= 2 bytes */
                payload[bit >> 3] |= (uint8_t)(u & 0xFFu);
                if (u >> 8) payload[(bit >> 3) + 1] |= (uint8_t)(u >> 8);
            }
            for (int64_t h = 0; h < k; ++h)
                hp[t * k + h] = y[t * stride + hp_idx[h]];
        }
    }
    free(lp_idx);
}

/* ---------------------------------------------- decompression + reduction */

/* Figure 2 caption / Section 5: dequantise each device's payload and sum over
 * the N devices, features back in their original order.
 *   ref64   : the sum in binary64 (every product q*s is exact) -- the reference
 *   chain32 : binary32 chain acc = fma(q_i, s_i, acc), i ascending (selected
 *             features: acc = fl(acc + y_i)); a secondary, stricter comparison
 * s is [N][E] (entries at selected features unused).  Either output may be NULL. */
void tpqo_dequant_reduce(const uint8_t *const *payloads, int64_t N, int64_t T,
                         int64_t E, const int32_t *hp_idx, int64_t k,
                         const float *s, double *ref64, float *chain32)
{
    tpqo_dequant_reduce_b(payloads, N, T, E, hp_idx, k, s, 4, ref64, chain32);
}

void tpqo_dequant_reduce_b(const uint8_t *const *payloads, int64_t N, int64_t T,
                           int64_t E, const int32_t *hp_idx, int64_t k,
                           const float *s, int bits, double *ref64, float *chain32)
{
    tpqo_dequant_reduce_bias_b(payloads, N, T, E, hp_idx, k, s, bits, NULL, ref64, chain32);
}

/* Section 2: the synchronised layer output is f(x) = sum_i f^(i)(x^(i)) + b.  With a bias b[E] (binary32)
 * the reference adds it in binary64 and the chain adds it last, chain32 = fl(acc32 + b_j); bias == NULL
 * leaves the sum as it is. */
void tpqo_dequant_reduce_bias_b(const uint8_t *const *payloads, int64_t N, int64_t T,
                                int64_t E, const int32_t *hp_idx, int64_t k,
                                const float *s, int bits, const float *bias, double *ref64, float *chain32)
{
    int64_t L = E - k;
    int64_t lp_bytes = tpqo_lp_bytes_b(T, E, k, bits);
    const unsigned cmask = (1u << bits) - 1u, sign = 1u << (bits - 1);
    int32_t *pos = (int32_t *)malloc(sizeof(int32_t) * (size_t)E); /* >=0: code slot c; <0: -(h+1) */
    {
        int32_t *slot_feature = (int32_t *)malloc(sizeof(int32_t) * (size_t)(L > 0 ? L : 1));
        tpqo_slot_order(E, hp_idx, k, slot_feature);
        for (int64_t c = 0; c < L; ++c) pos[slot_feature[c]] = (int32_t)c;
        for (int64_t h = 0; h < k; ++h) pos[hp_idx[h]] = -(int32_t)(h + 1);
        free(slot_feature);
    }
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        for (int64_t j = 0; j < E; ++j) {
            double acc64 = 0.0;
            float acc32 = 0.0f;
            for (int64_t i = 0; i < N; ++i) {
                const uint8_t *pl = payloads[i];
                if (pos[j] >= 0) {
                    int64_t bit = (t * L + pos[j]) * bits;
                    unsigned w = pl[bit >> 3];
                    if ((bit & 7) + bits > 8) w |= (unsigned)pl[(bit >> 3) + 1] << 8;
                    unsigned u = (w >> (bit & 7)) & cmask;
                    int q = (u & sign) ? (int)u - (int)(cmask + 1u) : (int)u;   /* two's complement, b bits */
                    float si = s[i * E + j];
                    acc64 += (double)q * (double)si;
                    acc32 = fmaf((float)q, si, acc32);
                } else {
                    int64_t h = -pos[j] - 1;
                    const uint16_t *hp = (const uint16_t *)(pl + lp_bytes);
                    float v = bf16_widen(hp[t * k + h]);
                    acc64 += (double)v;
                    volatile float tmp = acc32 + v;
                    acc32 = tmp;
                }
            }
            if (bias) {
                acc64 += (double)bias[j];
                volatile float tmp = acc32 + bias[j];
                acc32 = tmp;
            }
            if (ref64) ref64[t * E + j] = acc64;
            if (chain32) chain32[t * E + j] = acc32;
        }
    }
    free(pos);
}

/* BF16 rounding of a binary64 / binary32 array (for the BF16-output check). */
void tpqo_round_bf16_f32(const float *x, int64_t n, uint16_t *out)
{
    for (int64_t a = 0; a < n; ++a) out[a] = bf16_round(x[a]);
}

/* ------------------------------------------------------------------------------------------------
 * Section 2: the layer ahead of the synchronisation point on device i, f^(i)(x^(i)) = x^(i) W^(i),
 * x: [T][K], W^T stored as w: [E][K] (one row per output feature), all BF16; the output is BF16 too
 * (the models of Section 4 run in BF16).  Written as the definition: every product of two BF16 values is
 * exact in binary64, the K products are summed in binary64 in index order, and the sum is rounded ONCE,
 * from binary64, to the nearest BF16 (ties to even).  (Reading: the paper does not say how the layer
 * accumulates; a BF16 layer is specified by its rounded exact result, and an implementation that
 * accumulates in binary32 may differ from it by one BF16 unit in the last place.)
 * ---------------------------------------------------------------------------------------------- */
static uint16_t bf16_round_f64(double v)
{
    if (v != v) return 0x7FC0;
    if (v == 0.0) return signbit(v) ? 0x8000 : 0x0000;
    const double a = fabs(v);
    if (a >= 3.3961775292304601e38) return signbit(v) ? 0xFF80 : 0x7F80; /* >= max BF16 + half a unit: infinity */
    int e;
    (void)frexp(a, &e);          /* a = f * 2^e, 0.5 <= f < 1: the leading bit has weight 2^(e-1) */
    int q = e - 1 - 7;           /* weight of the last kept bit (8 significant bits) */
    if (q < -133) q = -133;      /* subnormal BF16: fixed spacing 2^-133 */
    const double r = nearbyint(ldexp(a, -q)); /* default rounding mode: nearest, ties to even; the scaling is exact */
    const float f = (float)ldexp(signbit(v) ? -r : r, q); /* exactly representable in binary32 */
    uint32_t u;
    memcpy(&u, &f, 4);
    return (uint16_t)(u >> 16);
}

void tpqo_linear_bf16(const uint16_t *x, const uint16_t *w, int64_t T, int64_t K, int64_t E, uint16_t *y)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t)
        for (int64_t j = 0; j < E; ++j) {
            double acc = 0.0;
            for (int64_t c = 0; c < K; ++c) acc += (double)bf16_widen(x[t * K + c]) * (double)bf16_widen(w[j * K + c]);
            y[t * E + j] = bf16_round_f64(acc);
        }
}
