/*
 * CPU oracle for the binarized 2-D convolution path (LceQuantize, LceBConv2d,
 * LceBMaxPool2d, LceDequantize and the fp32 residual add).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is the plain definition of
 * every operation, written as nested loops in +-1 integer arithmetic: nothing is
 * bit-packed inside the convolution, no XOR, no popcount, no blocking, no
 * fusion.  It shares no code, header, table or helper with the CUDA library and
 * neither includes the other.  Only tests, the smoke check and the benchmark's
 * cpu-baseline leg may call it.
 *
 * Conventions (paper, Section 3.2 "Operator implementations"):
 *   - LceQuantize: a 0 bit stands for +1.0, a 1 bit for -1.0; channels are
 *     packed along the channel axis, padded up to a multiple of 32.
 *   - LceBConv2d: padded locations hold zero words, i.e. +1.0 ("one-padding");
 *     zero-padding is the variant that needs a correction, here simply the
 *     definition with the out-of-image taps left out.
 *   - output transform: per-channel fp32 multiplier and bias after the fused
 *     activation, or a compare against per-channel thresholds for bit-packed
 *     output.
 *   - LceBMaxPool2d: max over the window of the +-1 values.
 * Readings where the paper is silent:
 *   - sign: bit = (x < 0), so +0.0, -0.0 and NaN binarize to +1;
 *   - channel c lives in word c/32, bit c%32 (least significant bit = lowest
 *     channel); channel-pad bits are 0; K counts true channels only;
 *   - "same" padding is TensorFlow's: out = ceil(in/stride), total pad
 *     max((out-1)*stride + k - in, 0), floor(half) before, the rest after;
 *   - float output y = fmaf((float)act(acc), multiplier[c], bias[c]), one
 *     rounding; bit-packed output bit = (acc < threshold[c]).
 *
 * "parity unpinned": the bit ORDER inside a word (LSB = lowest channel) is not
 * fixed by the paper; it is pinned only by this oracle's own one-hot tests.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

enum { ORACLE_PAD_VALID = 0, ORACLE_PAD_SAME_ONE = 1, ORACLE_PAD_SAME_ZERO = 2 };
enum { ORACLE_ACT_NONE = 0, ORACLE_ACT_RELU = 1 };

/* ---- geometry --------------------------------------------------------- */

/* Output extent along one axis (TensorFlow VALID / SAME rules). */
int32_t oracle_out_size(int32_t in, int32_t k, int32_t stride, int32_t padding)
{
    if (padding == ORACLE_PAD_VALID) {
        if (in < k) return 0;
        return (in - k) / stride + 1;
    }
    return (in + stride - 1) / stride;
}

/* Padding placed BEFORE the first input element along one axis. */
int32_t oracle_pad_before(int32_t in, int32_t k, int32_t stride, int32_t padding)
{
    if (padding == ORACLE_PAD_VALID) return 0;
    int32_t out = oracle_out_size(in, k, stride, padding);
    int32_t total = (out - 1) * stride + k - in;
    if (total < 0) total = 0;
    return total / 2;
}

/* ---- LceQuantize / LceDequantize -------------------------------------- */

/* s = -1 where x < 0, +1 elsewhere (value sign; +-0.0 and NaN give +1). */
void oracle_sign(const float *x, int8_t *s, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) s[i] = (x[i] < 0.0f) ? (int8_t)-1 : (int8_t)1;
}

/* x: fp32 [rows][channels] -> out: uint32 [rows][ceil(channels/32)]. */
void oracle_bitpack(const float *x, int64_t rows, int32_t channels, uint32_t *out)
{
    int32_t words = (channels + 31) / 32;
    for (int64_t r = 0; r < rows; ++r) {
        for (int32_t j = 0; j < words; ++j) out[r * words + j] = 0u;
        for (int32_t c = 0; c < channels; ++c) {
            int is_minus_one = (x[r * (int64_t)channels + c] < 0.0f);
            if (is_minus_one) out[r * words + c / 32] |= (uint32_t)1 << (c % 32);
        }
    }
}

/* Same packing rule applied to +-1 int8 values (bit 1 <=> -1). */
void oracle_bitpack_pm1(const int8_t *s, int64_t rows, int32_t channels, uint32_t *out)
{
    int32_t words = (channels + 31) / 32;
    for (int64_t r = 0; r < rows; ++r) {
        for (int32_t j = 0; j < words; ++j) out[r * words + j] = 0u;
        for (int32_t c = 0; c < channels; ++c)
            if (s[r * (int64_t)channels + c] == -1)
                out[r * words + c / 32] |= (uint32_t)1 << (c % 32);
    }
}

/* words: uint32 [rows][ceil(channels/32)] -> s: int8 [rows][channels] in {-1,+1}. */
void oracle_unpack_pm1(const uint32_t *words, int64_t rows, int32_t channels, int8_t *s)
{
    int32_t nw = (channels + 31) / 32;
    for (int64_t r = 0; r < rows; ++r)
        for (int32_t c = 0; c < channels; ++c) {
            uint32_t bit = (words[r * nw + c / 32] >> (c % 32)) & 1u;
            s[r * (int64_t)channels + c] = bit ? (int8_t)-1 : (int8_t)1;
        }
}

/* LceDequantize: packed -> +-1.0f. */
void oracle_unpack_f32(const uint32_t *words, int64_t rows, int32_t channels, float *out)
{
    int32_t nw = (channels + 31) / 32;
    for (int64_t r = 0; r < rows; ++r)
        for (int32_t c = 0; c < channels; ++c) {
            uint32_t bit = (words[r * nw + c / 32] >> (c % 32)) & 1u;
            out[r * (int64_t)channels + c] = bit ? -1.0f : 1.0f;
        }
}

/* ---- LceBConv2d: the accumulator -------------------------------------- */

/* One accumulator value by the definition:
 *   acc = sum over (ky,kx,c) of v(iy,ix,c) * w[o][ky][kx][c],
 *   v = a inside the image; outside: +1 (one-padding) or 0 (zero-padding).
 * a: int8 [N][H][W][Cin] in {-1,+1};  w: int8 [Cout][KH][KW][Cin] in {-1,+1}. */
static int32_t acc_at(const int8_t *a, const int8_t *w,
                      int32_t H, int32_t W, int32_t Cin,
                      int32_t KH, int32_t KW, int32_t sh, int32_t sw,
                      int32_t pt, int32_t pl, int32_t padding,
                      int32_t n, int32_t oh, int32_t ow, int32_t o)
{
    int32_t acc = 0;
    for (int32_t ky = 0; ky < KH; ++ky) {
        for (int32_t kx = 0; kx < KW; ++kx) {
            int32_t iy = oh * sh - pt + ky;
            int32_t ix = ow * sw - pl + kx;
            const int8_t *wp = w + (((int64_t)o * KH + ky) * KW + kx) * Cin;
            if (iy >= 0 && iy < H && ix >= 0 && ix < W) {
                const int8_t *ap = a + (((int64_t)n * H + iy) * W + ix) * Cin;
                for (int32_t c = 0; c < Cin; ++c) acc += (int32_t)ap[c] * (int32_t)wp[c];
            } else if (padding == ORACLE_PAD_SAME_ONE) {
                for (int32_t c = 0; c < Cin; ++c) acc += (int32_t)wp[c]; /* (+1) * w */
            }
            /* zero-padding: the tap contributes nothing */
        }
    }
    return acc;
}

/* acc: int32 [N][OH][OW][Cout]. Returns 0, or -1 if the output would be empty. */
int oracle_bconv2d_acc(const int8_t *a, const int8_t *w,
                       int32_t N, int32_t H, int32_t W, int32_t Cin, int32_t Cout,
                       int32_t KH, int32_t KW, int32_t sh, int32_t sw, int32_t padding,
                       int32_t *acc)
{
    int32_t OH = oracle_out_size(H, KH, sh, padding);
    int32_t OW = oracle_out_size(W, KW, sw, padding);
    int32_t pt = oracle_pad_before(H, KH, sh, padding);
    int32_t pl = oracle_pad_before(W, KW, sw, padding);
    if (OH <= 0 || OW <= 0) return -1;
    int64_t rows = (int64_t)N * OH;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        int32_t n = (int32_t)(r / OH), oh = (int32_t)(r % OH);
        for (int32_t ow = 0; ow < OW; ++ow)
            for (int32_t o = 0; o < Cout; ++o)
                acc[(((int64_t)n * OH + oh) * OW + ow) * Cout + o] =
                    acc_at(a, w, H, W, Cin, KH, KW, sh, sw, pt, pl, padding, n, oh, ow, o);
    }
    return 0;
}

/* The same definition at a list of sampled output coordinates
 * idx: int32 [count][4] = (n, oh, ow, o);  acc: int32 [count]. */
int oracle_bconv2d_acc_at(const int8_t *a, const int8_t *w,
                          int32_t N, int32_t H, int32_t W, int32_t Cin, int32_t Cout,
                          int32_t KH, int32_t KW, int32_t sh, int32_t sw, int32_t padding,
                          const int32_t *idx, int64_t count, int32_t *acc)
{
    int32_t OH = oracle_out_size(H, KH, sh, padding);
    int32_t OW = oracle_out_size(W, KW, sw, padding);
    int32_t pt = oracle_pad_before(H, KH, sh, padding);
    int32_t pl = oracle_pad_before(W, KW, sw, padding);
    for (int64_t i = 0; i < count; ++i) {
        int32_t n = idx[4 * i], oh = idx[4 * i + 1], ow = idx[4 * i + 2], o = idx[4 * i + 3];
        if (n < 0 || n >= N || oh < 0 || oh >= OH || ow < 0 || ow >= OW || o < 0 || o >= Cout)
            return -1;
        acc[i] = acc_at(a, w, H, W, Cin, KH, KW, sh, sw, pt, pl, padding, n, oh, ow, o);
    }
    return 0;
}

/* ---- LceBConv2d: output transforms ------------------------------------ */

/* y = fmaf((float)act(acc), multiplier[c], bias[c]); acc: [rows][Cout]. */
void oracle_transform_float(const int32_t *acc, int64_t rows, int32_t Cout,
                            const float *multiplier, const float *bias,
                            int32_t activation, float *out)
{
    for (int64_t r = 0; r < rows; ++r)
        for (int32_t c = 0; c < Cout; ++c) {
            int32_t v = acc[r * Cout + c];
            if (activation == ORACLE_ACT_RELU && v < 0) v = 0;
            out[r * Cout + c] = fmaf((float)v, multiplier[c], bias[c]);
        }
}

/* bit[c] = (acc < threshold[c]); 32 output channels per word, pad bits 0. */
void oracle_transform_bits(const int32_t *acc, int64_t rows, int32_t Cout,
                           const int32_t *threshold, uint32_t *out)
{
    int32_t words = (Cout + 31) / 32;
    for (int64_t r = 0; r < rows; ++r) {
        for (int32_t j = 0; j < words; ++j) out[r * words + j] = 0u;
        for (int32_t c = 0; c < Cout; ++c)
            if (acc[r * Cout + c] < threshold[c])
                out[r * words + c / 32] |= (uint32_t)1 << (c % 32);
    }
}

/* ---- LceBMaxPool2d ----------------------------------------------------- */

/* Max over the window of the +-1 values; out-of-image taps are skipped.
 * s: int8 [N][H][W][C] -> out: int8 [N][OH][OW][C]; padding VALID or SAME. */
int oracle_maxpool_pm1(const int8_t *s, int32_t N, int32_t H, int32_t W, int32_t C,
                       int32_t PH, int32_t PW, int32_t sh, int32_t sw, int32_t padding,
                       int8_t *out)
{
    int32_t OH = oracle_out_size(H, PH, sh, padding);
    int32_t OW = oracle_out_size(W, PW, sw, padding);
    int32_t pt = oracle_pad_before(H, PH, sh, padding);
    int32_t pl = oracle_pad_before(W, PW, sw, padding);
    if (OH <= 0 || OW <= 0) return -1;
    for (int32_t n = 0; n < N; ++n)
        for (int32_t oh = 0; oh < OH; ++oh)
            for (int32_t ow = 0; ow < OW; ++ow)
                for (int32_t c = 0; c < C; ++c) {
                    int32_t best = -2; /* below every +-1 value */
                    for (int32_t ky = 0; ky < PH; ++ky)
                        for (int32_t kx = 0; kx < PW; ++kx) {
                            int32_t iy = oh * sh - pt + ky, ix = ow * sw - pl + kx;
                            if (iy < 0 || iy >= H || ix < 0 || ix >= W) continue;
                            int32_t v = s[(((int64_t)n * H + iy) * W + ix) * C + c];
                            if (v > best) best = v;
                        }
                    out[(((int64_t)n * OH + oh) * OW + ow) * C + c] = (int8_t)best;
                }
    return 0;
}

/* ---- fp32 residual add -------------------------------------------------- */

void oracle_add_f32(const float *a, const float *b, float *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = a[i] + b[i];
}
