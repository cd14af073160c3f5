// Shared by the tiled XOR/POPC kernels (bconv_kxk.cuh, bconv_1x1.cuh) and their host side
// (bconv_tiled.cu): thread-tile constants, the kernel parameter block, the layout of the weight
// operands in shared memory and in the load-time packed image, the per-channel inner loop and the
// output transform (paper Section 3.2).  Internal to that translation unit (anonymous namespace).
#pragma once

#include "common.cuh"
#include "csa.cuh"

namespace lce {
namespace {


#ifndef LCE_WARPS
#define LCE_WARPS 4
#endif
constexpr int kWarps = LCE_WARPS;
constexpr int kThreads = 32 * kWarps;    // a warp = 4 pixels x 8 channel groups
constexpr int kPixPerStep = 4 * kWarps;  // pixels the CTA works on at a time
constexpr int kChanPerCta = 64;
constexpr int kChanPerThread = 8;
constexpr int kChanGroups = kChanPerCta / kChanPerThread;
constexpr int kWRow = 12;           // 9 carry-save operand words per (channel word, channel) + 3 pad
constexpr int kWGroupStride = kChanPerThread * kWRow + 4;  // +4 words: the 8 channel groups hit distinct banks
#ifdef LCE_NO_TAIL
constexpr bool kTailStep = false;
#else
constexpr bool kTailStep = true;
#endif
constexpr int kMaxTaps = 25;                               // 5x5 is the largest tiled filter
constexpr int kWsumWords = kChanPerCta * kMaxTaps;         // per-tap weight sums of a channel block

struct TiledParams {
    const uint32_t *in;
    const float *in_f32;       // KxK kernel: float activations, binarized while staged (then `in` is unused)
    const uint32_t *w;         // plain packed weights [Cout][3][3][Cw]
    const uint32_t *w_image;   // packed-weights image (see image_block_words), or nullptr
    const float *mult;
    const float *bias;
    const int32_t *thr;
    void *out;                 // may be null for float output when only the packed sign is wanted
    const float *residual;     // float output only: added after the multiply-add (or nullptr)
    uint32_t *out_packed;      // float output only: LceQuantize of the float result (or nullptr)
    int32_t N, H, W, Cin, Cw, Cout, Cow, OH, OW, pt, pl;
    int32_t tile_pixels;  // flat output pixels per tile, a multiple of kPixPerStep * TP
    int32_t n_tiles;      // ceil(M / tile_pixels); CTA x works on tiles x, x + gridDim.x, ...
    int32_t M, Hp, Wp, pitch, plane;
    int32_t cw_shift;     // log2(Cw) when Cw is a power of two, else -1
    int32_t half_block;   // KxK kernel: index of the channel block with at most 32 real channels, or -1
    int32_t full_blocks, ctas_full, ctas_half;  // KxK kernel: 1-D grid = full_blocks x ctas_full CTAs, then ctas_half
    int32_t range_full, range_half;             // KxK kernel: flat output pixels per CTA of a full / the half block
    int32_t stride;       // pointwise kernel only
    int32_t n9, rem3, cwp; // pointwise kernel: nine-word groups, leftover triples, padded words per pixel
    int32_t padding, out_type, activation;
};

// Shared-memory / packed-image offset (in words) of the operands of (channel word, channel).
__host__ __device__ __forceinline__ int32_t w_offset(int cw, int ch)
{
    return cw * kChanGroups * kWGroupStride + (ch >> 3) * kWGroupStride + (ch & 7) * kWRow;
}
// One channel block of the packed image: operands of every nine-word group, then the per-tap sums.
__host__ __device__ __forceinline__ int64_t image_block_words(int groups)
{
    return (int64_t)groups * kChanGroups * kWGroupStride + kWsumWords;
}
// nine-word groups per channel word of a KSxKS filter: taps beyond KS*KS count as zero words
__host__ __device__ constexpr int groups_per_word(int ks) { return (ks * ks + 8) / 9; }

template <int BYTE_OFF>
__device__ __forceinline__ uint4 lds128(uint32_t saddr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4+%5];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(saddr), "n"(BYTE_OFF));
    return v;
}
template <int BYTE_OFF>
__device__ __forceinline__ uint32_t lds32(uint32_t saddr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(saddr), "n"(BYTE_OFF));
    return v;
}
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src)
{
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}

template <int J>
__device__ __forceinline__ void load_w_triples(uint32_t saddr, Triple (&wt)[3])
{
    const uint4 q0 = lds128<J * 48>(saddr);
    const uint4 q1 = lds128<J * 48 + 16>(saddr);
    const uint32_t q2 = lds32<J * 48 + 32>(saddr);
    wt[0].all = q0.x; wt[0].pair = q0.y; wt[0].first = q0.z;
    wt[1].all = q0.w; wt[1].pair = q1.x; wt[1].first = q1.y;
    wt[2].all = q1.z; wt[2].pair = q1.w; wt[2].first = q2;
}

template <int J, int TP>
struct ChannelLoop {
    // channel J of the thread: weight operands from shared memory once, then all TP pixels
    __device__ __forceinline__ static void run(uint32_t w_saddr, const Triple (&at)[TP][3], const Weights124 &k,
                                               uint32_t (&acc)[TP][kChanPerThread])
    {
        Triple wt[3];
        load_w_triples<J>(w_saddr, wt);
#ifdef LCE_SERIAL_PIXELS
#pragma unroll
        for (int i = 0; i < TP; ++i) popc9_mad(at[i], wt, k, acc[i][J]);
#else
        popc9_mad_pixels<TP, kChanPerThread, J>(at, wt, k, acc);
#endif
        ChannelLoop<J + 1, TP>::run(w_saddr, at, k, acc);
    }
};
template <int TP>
struct ChannelLoop<kChanPerThread, TP> {
    __device__ __forceinline__ static void run(uint32_t, const Triple (&)[TP][3], const Weights124 &,
                                               uint32_t (&)[TP][kChanPerThread]) {}
};

// Nine plain weight words of one (channel, channel word) -> nine carry-save operand words.
__device__ __forceinline__ void store_w_operands(const uint32_t (&wv)[9], uint32_t *dst)
{
#pragma unroll
    for (int g = 0; g < 3; ++g) {
        const Triple t = make_triple(wv[3 * g], wv[3 * g + 1], wv[3 * g + 2]);
        dst[3 * g] = t.all;
        dst[3 * g + 1] = t.pair;
        dst[3 * g + 2] = t.first;
    }
    dst[9] = dst[10] = dst[11] = 0u;
}

// Load-time weight packing: plain [Cout][3][3][Cw] -> per channel block of 64 the exact
// shared-memory image the convolution kernel wants (operands, then per-tap sums).
__global__ void __launch_bounds__(128)
pack_weights_kernel(const uint32_t *__restrict__ w, uint32_t *__restrict__ image, int32_t Cout, int32_t Cw,
                    int32_t Cin, int32_t chan_blocks, int32_t ks)
{
    // group = (channel word, run of nine taps); taps past ks*ks are zero words
    const int taps = ks * ks, ng = groups_per_word(ks);
    const int64_t entries = (int64_t)chan_blocks * kChanPerCta * Cw * ng;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < entries;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int g = (int)(e % ng);
        const int cw = (int)((e / ng) % Cw);
        const int64_t c = e / ((int64_t)ng * Cw);  // global channel (may be >= Cout in the last block)
        const int cb = (int)(c / kChanPerCta), ch = (int)(c % kChanPerCta);
        uint32_t wv[9];
#pragma unroll
        for (int t = 0; t < 9; ++t) wv[t] = (c < Cout && 9 * g + t < taps) ? w[(c * taps + 9 * g + t) * Cw + cw] : 0u;
        uint32_t *block = image + cb * image_block_words(Cw * ng);
        store_w_operands(wv, block + w_offset(cw * ng + g, ch));
        if ((ch & 7) == 7) {  // the 4 pad words after every 8 channels
            uint32_t *pad = block + w_offset(cw * ng + g, ch) + kWRow;
            pad[0] = pad[1] = pad[2] = pad[3] = 0u;
        }
        if (cw == 0 && g == 0) {
            // sum over the true channels of one tap's weights = Cin - 2*popcount (pad bits are 0)
            int32_t *wsum = reinterpret_cast<int32_t *>(block + (int64_t)Cw * ng * kChanGroups * kWGroupStride);
            for (int t = 0; t < kMaxTaps; ++t) {
                int32_t cnt = 0;
                if (c < Cout && t < taps)
                    for (int j = 0; j < Cw; ++j) cnt += __popc(w[(c * taps + t) * Cw + j]);
                wsum[ch * kMaxTaps + t] = (c < Cout && t < taps) ? Cin - 2 * cnt : 0;
            }
        }
    }
}

// Per-channel parameters of the thread's 8 output channels for the chosen output type.
struct ChannelParams {
    float mult[kChanPerThread], bias[kChanPerThread];
    int32_t thr[kChanPerThread];
};
__device__ __forceinline__ void load_channel_params(const TiledParams &p, int chan, ChannelParams &c)
{
    if (chan + kChanPerThread <= p.Cout) {
        // all eight channels exist (every thread but those of a ragged last group): unconditional
        // loads of only what the output type needs
        if (p.out_type == LCE_OUT_BITPACKED) {
#pragma unroll
            for (int j = 0; j < kChanPerThread; ++j) {
                c.mult[j] = 0.f;
                c.bias[j] = 0.f;
                c.thr[j] = __ldg(p.thr + chan + j);
            }
        } else {
#pragma unroll
            for (int j = 0; j < kChanPerThread; ++j) {
                c.mult[j] = (p.out_type == LCE_OUT_FLOAT32) ? __ldg(p.mult + chan + j) : 0.f;
                c.bias[j] = (p.out_type == LCE_OUT_FLOAT32) ? __ldg(p.bias + chan + j) : 0.f;
                c.thr[j] = INT32_MIN;
            }
        }
    } else {
#pragma unroll
        for (int j = 0; j < kChanPerThread; ++j) {
            const bool ok = chan + j < p.Cout;
            c.mult[j] = (p.out_type == LCE_OUT_FLOAT32 && ok) ? __ldg(p.mult + chan + j) : 0.f;
            c.bias[j] = (p.out_type == LCE_OUT_FLOAT32 && ok) ? __ldg(p.bias + chan + j) : 0.f;
            c.thr[j] = (p.out_type == LCE_OUT_BITPACKED && ok) ? __ldg(p.thr + chan + j) : INT32_MIN;  // pad bits -> 0
        }
    }
}

// int32 -> fp32 without the conversion unit: for |v| < 2^22 the integer v + 0x4B400000 is the bit
// pattern of the float 12582912 + v (1.5 * 2^23, where floats are exactly one apart), so one exact
// float subtraction gives (float)v.  The kernels fold the integer addition into acc = K - 2*count
// ("biased" accumulators); the conversion then costs one FADD on the FMA pipe instead of an I2F on
// the unit the popcounts use.
constexpr int32_t kFloatBias = 0x4B400000;
constexpr int32_t kMaxBiasedK = 1 << 22;

// The thread's 8 output bits (channels 8*cg .. 8*cg+7 of the block) -> the output word they belong to:
// the 4 lanes that hold the 4 bytes of a word combine them with two shuffles, one lane stores.
__device__ __forceinline__ void store_bits_byte(const TiledParams &p, uint32_t bits, int m, bool pix_ok, int cg, int ch0)
{
    bits <<= 8 * (cg & 3);
    bits |= __shfl_xor_sync(0xffffffffu, bits, 1);
    bits |= __shfl_xor_sync(0xffffffffu, bits, 2);
    const int word = (ch0 >> 5) + (cg >> 2);
    if (pix_ok && (cg & 3) == 0 && word < p.Cow) static_cast<uint32_t *>(p.out)[(int64_t)m * p.Cow + word] = bits;
}

// Threshold compare on packed 16-bit counts without unpacking them (K < 32768).  With x the mismatch
// count, acc = K - 2x < thr  <=>  c - 2x < 0 for c = K - thr, and, c' = c | 1 being odd, <=> c' - 2x < 0
// with c' - 2x never zero.  For the pixel in the low half, (c' << 15) - (acc << 16) = 32768 (c' - 2 x_lo);
// for the pixel in the high half, (c' << 15) - acc = 32768 (c' - 2 x_hi) - x_lo, which has the sign of
// c' - 2 x_hi because that is odd and x_lo < 32768.  So the output bit is the sign bit of one
// multiply-add, and a funnel shift collects it: two instructions per output instead of five.
// The threshold is clamped to [-K-1, K+1] first (outside that range nothing changes), so c' << 15 fits.
__device__ __forceinline__ void packed_compare_operands(const int32_t (&thr)[kChanPerThread], int K, int32_t (&c15)[kChanPerThread])
{
#pragma unroll
    for (int j = 0; j < kChanPerThread; ++j) c15[j] = ((K - max(-K - 1, min(K + 1, thr[j]))) | 1) * 32768;
}
template <bool HIGH>
__device__ __forceinline__ uint32_t packed_compare_bits(const uint32_t (&acc)[kChanPerThread], const int32_t (&c15)[kChanPerThread])
{
    uint32_t bits = 0u;
#pragma unroll
    for (int j = kChanPerThread - 1; j >= 0; --j) {
        const uint32_t e = HIGH ? (uint32_t)c15[j] - acc[j] : (uint32_t)c15[j] - acc[j] * 65536u;
        bits = __funnelshift_l(e, bits, 1);  // (bits << 1) | sign(e)
    }
    return bits;
}

// The bit-packed output transform of one pixel: compare, pack the thread's 8 channels, combine the
// 4 lanes that hold the 4 bytes of one output word, store.  Every lane of the warp must call it.
__device__ __forceinline__ void store_bits(const TiledParams &p, const int32_t (&v)[kChanPerThread],
                                           const int32_t (&thr)[kChanPerThread], int m, bool pix_ok, int cg, int ch0)
{
    uint32_t bits = 0u;
#pragma unroll
    for (int j = 0; j < kChanPerThread; ++j) bits |= (v[j] < thr[j] ? 1u : 0u) << j;
    store_bits_byte(p, bits, m, pix_ok, cg, ch0);
}

// What a thread's output transform will be, decided once per kernel: the plain float cases (biased
// accumulators, all eight channels of the thread exist, 16-byte stores, no shortcut, no packed copy)
// skip every test the general form makes per pixel.
constexpr int kEpiGeneral = 0, kEpiFloat = 1, kEpiFloatRelu = 2, kEpiBits = 3;
__device__ __forceinline__ int epilogue_mode(const TiledParams &p, int chan, bool biased)
{
    if (p.out_type == LCE_OUT_BITPACKED && p.padding != LCE_PAD_SAME_ZERO) return kEpiBits;
    const bool plain = p.out_type == LCE_OUT_FLOAT32 && biased && p.residual == nullptr && p.out_packed == nullptr &&
                       p.out != nullptr && (p.Cout & 3) == 0 && chan + kChanPerThread <= p.Cout;
    return !plain ? kEpiGeneral : p.activation == LCE_ACT_RELU ? kEpiFloatRelu : kEpiFloat;
}

// Output transform of one pixel's 8 accumulators v (paper Section 3.2): float multiply-add after
// the fused activation, threshold compare + bit-pack, or the raw accumulators.  Every lane of the
// warp must call it (the bit-packed form combines 4 lanes with shuffles); pix_ok guards the store.
__device__ __forceinline__ void store_outputs(const TiledParams &p, const int32_t (&v)[kChanPerThread],
                                              const ChannelParams &c, int m, bool pix_ok, int cg, int ch0, int chan,
                                              bool biased,  // v carries + kFloatBias (float output with K < 2^22 only)
                                              int epi)      // epilogue_mode() of this thread
{
    const float (&mult)[kChanPerThread] = c.mult;
    const float (&bias)[kChanPerThread] = c.bias;
    const int32_t (&thr)[kChanPerThread] = c.thr;
    if (epi == kEpiFloat || epi == kEpiFloatRelu) {
        // the common float case with every decision already taken: one exact FADD takes the bias off the
        // accumulator, one FMA, two 16-byte stores
        float f[kChanPerThread];
        if (epi == kEpiFloat) {
#pragma unroll
            for (int j = 0; j < kChanPerThread; ++j)
                f[j] = __fmaf_rn(__fadd_rn(__int_as_float(v[j]), -12582912.0f), mult[j], bias[j]);
        } else {
#pragma unroll
            for (int j = 0; j < kChanPerThread; ++j)
                f[j] = __fmaf_rn(__fadd_rn(__int_as_float(max(v[j], kFloatBias)), -12582912.0f), mult[j], bias[j]);
        }
        if (pix_ok) {
            float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(p.out) + (int64_t)m * p.Cout + chan);
            dst[0] = make_float4(f[0], f[1], f[2], f[3]);
            dst[1] = make_float4(f[4], f[5], f[6], f[7]);
        }
        return;
    }
    if (p.out_type == LCE_OUT_BITPACKED) {
        store_bits(p, v, thr, m, pix_ok, cg, ch0);
    } else if (p.out_type == LCE_OUT_FLOAT32) {
        float f[kChanPerThread];
#pragma unroll
        for (int j = 0; j < kChanPerThread; ++j) {
            // fused ReLU on the integer: max(v, 0), or max(v + bias, bias) in the biased form
            const int32_t floor_v = p.activation == LCE_ACT_RELU ? (biased ? kFloatBias : 0) : INT32_MIN;
            const int32_t a = max(v[j], floor_v);
            const float x = biased ? __fadd_rn(__int_as_float(a), -12582912.0f) : (float)a;
            f[j] = __fmaf_rn(x, mult[j], bias[j]);
        }
        const bool vec = (p.Cout & 3) == 0 && chan + kChanPerThread <= p.Cout;
        if (p.residual != nullptr) {
            // fused shortcut: one more fp32 add, exactly as a separate add kernel would round it
            const float *r = p.residual + (int64_t)m * p.Cout + chan;
            if (pix_ok) {
                if (vec) {
                    const float4 r0 = __ldg(reinterpret_cast<const float4 *>(r));
                    const float4 r1 = __ldg(reinterpret_cast<const float4 *>(r) + 1);
                    f[0] = __fadd_rn(f[0], r0.x); f[1] = __fadd_rn(f[1], r0.y);
                    f[2] = __fadd_rn(f[2], r0.z); f[3] = __fadd_rn(f[3], r0.w);
                    f[4] = __fadd_rn(f[4], r1.x); f[5] = __fadd_rn(f[5], r1.y);
                    f[6] = __fadd_rn(f[6], r1.z); f[7] = __fadd_rn(f[7], r1.w);
                } else {
#pragma unroll
                    for (int j = 0; j < kChanPerThread; ++j)
                        if (chan + j < p.Cout) f[j] = __fadd_rn(f[j], __ldg(r + j));
                }
            }
        }
        if (pix_ok && p.out != nullptr) {
            float *dst = static_cast<float *>(p.out) + (int64_t)m * p.Cout + chan;
            if (vec) {
                reinterpret_cast<float4 *>(dst)[0] = make_float4(f[0], f[1], f[2], f[3]);
                reinterpret_cast<float4 *>(dst)[1] = make_float4(f[4], f[5], f[6], f[7]);
            } else {
#pragma unroll
                for (int j = 0; j < kChanPerThread; ++j)
                    if (chan + j < p.Cout) dst[j] = f[j];
            }
        }
        if (p.out_packed != nullptr) {
            // fused LceQuantize of the float result for the next binarized layer: bit = (y < 0)
            uint32_t bits = 0u;
#pragma unroll
            for (int j = 0; j < kChanPerThread; ++j) bits |= ((chan + j < p.Cout && f[j] < 0.0f) ? 1u : 0u) << j;
            bits <<= 8 * (cg & 3);
            bits |= __shfl_xor_sync(0xffffffffu, bits, 1);
            bits |= __shfl_xor_sync(0xffffffffu, bits, 2);
            const int word = (ch0 >> 5) + (cg >> 2);
            if (pix_ok && (cg & 3) == 0 && word < p.Cow) p.out_packed[(int64_t)m * p.Cow + word] = bits;
        }
    } else {
        if (pix_ok) {
            int32_t *dst = static_cast<int32_t *>(p.out) + (int64_t)m * p.Cout + chan;
            if ((p.Cout & 3) == 0 && chan + kChanPerThread <= p.Cout) {
                reinterpret_cast<int4 *>(dst)[0] = make_int4(v[0], v[1], v[2], v[3]);
                reinterpret_cast<int4 *>(dst)[1] = make_int4(v[4], v[5], v[6], v[7]);
            } else {
#pragma unroll
                for (int j = 0; j < kChanPerThread; ++j)
                    if (chan + j < p.Cout) dst[j] = v[j];
            }
        }
    }
}

}  // namespace
}  // namespace lce
