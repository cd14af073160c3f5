// LceBConv2d, tiled XOR/POPC kernels for 3x3 and 5x5 filters (and, further down, 1x1) (paper
// Section 3.2: im2col -> BGEMM -> output transform, here as one implicit-GEMM kernel: the im2col
// matrix is never materialised and the accumulators never leave registers before the output
// transform).
//
// Stride 1 or 2, any channel counts and image sizes:
//   * a CTA of 8 (or 4) warps owns one contiguous range of output pixels (flat (n, oh, ow) order)
//     times 64 output channels; a warp works on 4 pixels x 8 channel groups at a time (8 x 4 in a
//     channel block that has at most 32 channels), a thread on TP pixels x 8 channels, i.e. TP x 8
//     accumulators in registers.  All ranges are equal to within two pixels per thread: the last step
//     of a range runs the two-pixel form of the same code;
//   * the CTA copies the packed input rows its pixels need into shared memory, a tile of up to
//     8 x 32 x TP pixels at a time (the next tile while the current one is computed), one plane per
//     channel word, in "padded image" coordinates: rows/columns outside the image hold zero words,
//     which is exactly the paper's one-padding (a zero bit is +1.0);
//   * the weights of its 64 channels arrive as carry-save operands (csa.cuh): either copied in
//     16-byte pieces from a buffer prepared once by lce_bconv2d_pack_weights (the paper's
//     load-time "weight packing"), or derived on the fly from the plain packed weights;
//   * for every channel word nine taps of a (pixel, channel) pair form one nine-word carry-save
//     group (a 5x5 filter is three groups, the last two words zero): 16 LOP3 + 4 POPC + 4 IMAD
//     instead of 9 XOR + 9 POPC + 9 adds.  The activation-side operands of the thread's TP pixels
//     sit in registers for the whole group; the weight-side operands of one channel are read from
//     shared memory once and used for all TP pixels (shared-memory bandwidth, not issue slots, is
//     what this ordering saves);
//   * epilogue: acc = K - 2*count, then float multiply-add, threshold + bit-pack, or raw int32.
#include <stdio.h>
#include <stdlib.h>

#include <type_traits>

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
#pragma unroll
    for (int j = 0; j < kChanPerThread; ++j) {
        const bool ok = chan + j < p.Cout;
        c.mult[j] = (p.out_type == LCE_OUT_FLOAT32 && ok) ? __ldg(p.mult + chan + j) : 0.f;
        c.bias[j] = (p.out_type == LCE_OUT_FLOAT32 && ok) ? __ldg(p.bias + chan + j) : 0.f;
        c.thr[j] = (p.out_type == LCE_OUT_BITPACKED && ok) ? __ldg(p.thr + chan + j) : INT32_MIN;  // pad bits -> 0
    }
}

// Output transform of one pixel's 8 accumulators v (paper Section 3.2): float multiply-add after
// the fused activation, threshold compare + bit-pack, or the raw accumulators.  Every lane of the
// warp must call it (the bit-packed form combines 4 lanes with shuffles); pix_ok guards the store.
__device__ __forceinline__ void store_outputs(const TiledParams &p, const int32_t (&v)[kChanPerThread],
                                              const ChannelParams &c, int m, bool pix_ok, int cg, int ch0, int chan)
{
    const float (&mult)[kChanPerThread] = c.mult;
    const float (&bias)[kChanPerThread] = c.bias;
    const int32_t (&thr)[kChanPerThread] = c.thr;
    if (p.out_type == LCE_OUT_BITPACKED) {
        uint32_t bits = 0u;
#pragma unroll
        for (int j = 0; j < kChanPerThread; ++j) bits |= (v[j] < thr[j] ? 1u : 0u) << j;
        // the 4 lanes cg&~3 .. cg|3 hold the 4 bytes of one output word
        bits <<= 8 * (cg & 3);
        bits |= __shfl_xor_sync(0xffffffffu, bits, 1);
        bits |= __shfl_xor_sync(0xffffffffu, bits, 2);
        const int word = (ch0 >> 5) + (cg >> 2);
        if (pix_ok && (cg & 3) == 0 && word < p.Cow)
            static_cast<uint32_t *>(p.out)[(int64_t)m * p.Cow + word] = bits;
    } else if (p.out_type == LCE_OUT_FLOAT32) {
        float f[kChanPerThread];
#pragma unroll
        for (int j = 0; j < kChanPerThread; ++j) {
            const int32_t a = (p.activation == LCE_ACT_RELU && v[j] < 0) ? 0 : v[j];
            f[j] = __fmaf_rn((float)a, mult[j], bias[j]);
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

// 4-byte asynchronous global->shared copy (no register round trip: the copy overlaps whatever the
// thread does next).
__device__ __forceinline__ void cp_async4(uint32_t *smem_dst, const uint32_t *gmem_src)
{
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d), "l"(gmem_src) : "memory");
}

// First virtual (padded-image) row of a tile of flat pixels [m0, m_end): v = n*Hp + oh*stride.
template <int STRIDE>
__device__ __forceinline__ int tile_first_vrow(const TiledParams &p, int m0)
{
    const int r_first = m0 / p.OW;
    return (r_first / p.OH) * p.Hp + (r_first % p.OH) * STRIDE;
}

// LceQuantize fused into the loader, one image row: lane = channel within a word, one coalesced
// 128-byte load and one ballot per word (bit = 1 for a negative value), eight words in flight per
// warp; lane u keeps word u of the batch and writes it.
struct RowF32 {
    int W, Cw, Cin, plane, pl, Wp;
};
__device__ __forceinline__ void stage_row_f32(const float *src, uint32_t *dst_row, RowF32 p, int lane)
{
    const int row_words = p.W * p.Cw;
    for (int e0 = 0; e0 < row_words; e0 += 8) {
        float x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int e = e0 + u;
            const int ix = e / p.Cw, c = (e - ix * p.Cw) * 32 + lane;
            x[u] = (e < row_words && c < p.Cin) ? __ldg(src + (int64_t)ix * p.Cin + c) : 0.0f;
        }
        uint32_t mine = 0u;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t word = __ballot_sync(0xffffffffu, x[u] < 0.0f);
            if (lane == u) mine = word;
        }
        const int e = e0 + lane;
        if (lane < 8 && e < row_words) {
            const int ix = e / p.Cw, cw = e - ix * p.Cw;
            dst_row[cw * p.plane + ix + p.pl] = mine;
        }
    }
    const int edge = p.Wp - p.W;
    for (int e = lane; e < edge * p.Cw; e += 32) {
        const int cw = e / edge, k = e - cw * edge;
        dst_row[cw * p.plane + (k < p.pl ? k : p.W + k)] = 0u;
    }
}

// Copies the input rows a tile needs into shared memory: global [n][iy][ix][cw] -> [cw][v][x] in
// padded-image coordinates.  Image words travel as asynchronous copies (the caller waits for
// them); rows and columns outside the image are written as zero words (one-padding).
template <int KS, int STRIDE, int NW, bool F32>
__device__ __forceinline__ void stage_rows(const TiledParams &p, int m0, int m_end, uint32_t *sA, int warp, int lane)
{
    const int r_last = (m_end - 1) / p.OW;
    const int v_first = tile_first_vrow<STRIDE>(p, m0);
    const int v_last = (r_last / p.OH) * p.Hp + (r_last % p.OH) * STRIDE + (KS - 1);
    const int nv = v_last - v_first + 1;
    const int row_words = p.W * p.Cw;
    for (int v = warp; v < nv; v += NW) {
        const int va = v_first + v;
        const int n = va / p.Hp;
        const int iy = va - n * p.Hp - p.pt;
        uint32_t *dst_row = sA + v * p.pitch;
        if (F32 && n < p.N && iy >= 0 && iy < p.H) {
            stage_row_f32(p.in_f32 + ((int64_t)n * p.H + iy) * p.W * p.Cin, dst_row,
                          RowF32{p.W, p.Cw, p.Cin, p.plane, p.pl, p.Wp}, lane);
        } else if (n < p.N && iy >= 0 && iy < p.H) {
            const uint32_t *src = p.in + ((int64_t)n * p.H + iy) * row_words;
            for (int e = lane; e < row_words; e += 32) {
                int ix, cw;
                if (p.cw_shift >= 0) { ix = e >> p.cw_shift; cw = e & (p.Cw - 1); }
                else { ix = e / p.Cw; cw = e - ix * p.Cw; }
                cp_async4(dst_row + cw * p.plane + ix + p.pl, src + e);
            }
            const int edge = p.Wp - p.W;  // pad columns: pl on the left, the rest on the right
            for (int e = lane; e < edge * p.Cw; e += 32) {
                const int cw = e / edge, k = e - cw * edge;
                dst_row[cw * p.plane + (k < p.pl ? k : p.W + k)] = 0u;
            }
        } else {
            for (int e = lane; e < p.Wp * p.Cw; e += 32) {
                const int cw = e / p.Wp, x = e - cw * p.Wp;
                dst_row[cw * p.plane + x] = 0u;
            }
        }
    }
}

// NW warps per CTA: 4 normally; 8 when the weight operands of a channel block are so large that
// only one CTA fits an SM, so that the SM still has eight warps to hide latencies with.
template <int KS, int STRIDE, int TP, int NW, bool F32>
__global__ void __launch_bounds__(32 * NW, (TP <= 2 ? 24 : 16) / NW)
bconv3x3_kernel(const TiledParams p)
{
    constexpr int kThreads = 32 * NW;
    constexpr int kTaps = KS * KS;             // 9 or 25
    constexpr int kNG = groups_per_word(KS);   // nine-word groups per channel word: 1 or 3
    extern __shared__ __align__(16) uint32_t smem[];
    const int w_words = p.Cw * kNG * kChanGroups * kWGroupStride;
    uint32_t *sW = smem;                                           // [Cw*kNG][8 groups][kWGroupStride]
    int32_t *sWsum = reinterpret_cast<int32_t *>(smem + w_words);  // [64][9]
    uint32_t *sA0 = smem + w_words + kWsumWords;                   // 2 x [Cw][nv][pitch]

    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    // 1-D grid: ctas_full CTAs for each full channel block, then ctas_half for the half block
    // Every CTA of a channel block owns one contiguous range of flat output pixels.
    int block_y, block_x, range;
    if ((int)blockIdx.x < p.full_blocks * p.ctas_full) {
        block_y = blockIdx.x % p.full_blocks;
        block_x = blockIdx.x / p.full_blocks;
        range = p.range_full;
    } else {
        block_y = p.full_blocks;
        block_x = blockIdx.x - p.full_blocks * p.ctas_full;
        range = p.range_half;
    }
    const int r_begin = block_x * range;                 // host: (CTAs - 1) * range < M
    const int r_end = min(r_begin + range, p.M);
    const int ch0 = block_y * kChanPerCta;
    const int plane_words = p.Cw * p.plane;  // one input buffer; two of them alternate between tiles

    // ---- weights ----------------------------------------------------------------------------
    if (p.w_image != nullptr) {
        // prepared image: a plain 16-byte asynchronous copy of this channel block
        const int words = (p.padding == LCE_PAD_SAME_ZERO) ? w_words + kWsumWords : w_words;
        const uint32_t *src = p.w_image + block_y * image_block_words(p.Cw * kNG);
        for (int e = tid * 4; e < words; e += kThreads * 4) cp_async16(smem + e, src + e);
        asm volatile("cp.async.commit_group;" ::: "memory");
    } else {
        for (int e = tid; e < kChanPerCta * p.Cw * kNG; e += kThreads) {
            const int g = e % kNG;
            const int cw = (e / kNG) % p.Cw;
            const int ch = e / (kNG * p.Cw);
            uint32_t wv[9];
#pragma unroll
            for (int t = 0; t < 9; ++t)
                wv[t] = (ch0 + ch < p.Cout && 9 * g + t < kTaps)
                            ? __ldg(p.w + ((int64_t)(ch0 + ch) * kTaps + 9 * g + t) * p.Cw + cw) : 0u;
            store_w_operands(wv, sW + w_offset(cw * kNG + g, ch));
        }
        if (p.padding == LCE_PAD_SAME_ZERO) {
            for (int e = tid; e < kChanPerCta * kTaps; e += kThreads) {
                const int ch = e / kTaps, t = e - ch * kTaps;
                int32_t cnt = 0;
                if (ch0 + ch < p.Cout)
                    for (int cw = 0; cw < p.Cw; ++cw)
                        cnt += __popc(__ldg(p.w + ((int64_t)(ch0 + ch) * kTaps + t) * p.Cw + cw));
                sWsum[ch * kMaxTaps + t] = p.Cin - 2 * cnt;
            }
        }
    }

    // ---- this thread's channels --------------------------------------------------------------
    // A warp is 4 pixels x 8 channel groups; in a channel block whose upper 32 channels do not
    // exist (Cout mod 64 in 1..32) it is 8 pixels x 4 channel groups instead, so that no lane works
    // on channels that are not there.
    const int cg_bits = (block_y == p.half_block) ? 2 : 3;
    const int px = lane >> cg_bits, cg = lane & ((1 << cg_bits) - 1);
    const int pix_per_warp = 32 >> cg_bits;
    const int pix_per_step = pix_per_warp * NW;  // pixels the CTA works on at a time
    const int chan = ch0 + cg * kChanPerThread;
    const int K = kTaps * p.Cin;
    Weights124 k124;
    k124.one = p.N > 0 ? 1u : p.Cin;  // opaque to the compiler: keeps the weighted sum on multiply-adds
    k124.two = p.N > 0 ? 2u : p.Cin;
    k124.four = p.N > 0 ? 4u : p.Cin;
    asm volatile("" : "+r"(k124.one), "+r"(k124.two), "+r"(k124.four));
    const uint32_t w_saddr0 = (uint32_t)__cvta_generic_to_shared(sW + cg * kWGroupStride);

    // ---- loop over the tiles of this CTA's range; the next tile's input rows are copied into the
    // other buffer while the current tile is computed ---------------------------------------------
    if (r_begin < r_end)
        stage_rows<KS, STRIDE, NW, F32>(p, r_begin, min(r_begin + p.tile_pixels, r_end), sA0, warp, lane);
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

  for (int m0 = r_begin, buf = 0; m0 < r_end; m0 += p.tile_pixels, buf ^= 1) {
    const uint32_t *sA = sA0 + buf * plane_words;
    const int m_end = min(m0 + p.tile_pixels, r_end);
    {
        const int next = m0 + p.tile_pixels;
        if (next < r_end)
            stage_rows<KS, STRIDE, NW, F32>(p, next, min(next + p.tile_pixels, r_end), sA0 + (buf ^ 1) * plane_words, warp, lane);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    const int r_first = m0 / p.OW;
    const int v_first = tile_first_vrow<STRIDE>(p, m0);

    // running position of this lane's next pixel; the pixels of one lane are pix_per_step apart
    int m_next = m0 + warp * pix_per_warp + px;  // lanes of a warp: neighbouring pixels
    int ow, voh, oh_left;  // voh = n*Hp + oh*STRIDE: the pixel's first virtual row
    {
        const int r = m_next / p.OW;
        ow = m_next - r * p.OW;
        const int n = r / p.OH;
        const int oh = r - n * p.OH;
        voh = n * p.Hp + oh * STRIDE;
        oh_left = p.OH - 1 - oh;  // rows left in the image after this one
    }
    const int a_base_first = (m0 - r_first * p.OW) * STRIDE;  // the tile's first pixel sits in virtual row 0

    // One step: every thread works on TPX pixels x 8 channels.  TPX = TP everywhere except at the
    // end of the CTA's range, where a remainder of at most two pixels per thread takes the TPX = 2
    // form of the same code: the work of all CTAs is then equal to within 2 x pix_per_step pixels.
    auto step = [&](auto tpx_tag, const int base) {
        constexpr int TPX = decltype(tpx_tag)::value;
        int a_base[TPX];
#pragma unroll
        for (int i = 0; i < TPX; ++i) {
            // pixels past the end of the tile redo the tile's first pixel and store nothing
            a_base[i] = (m_next < m_end) ? (voh - v_first) * p.pitch + ow * STRIDE : a_base_first;
            m_next += pix_per_step;
            ow += pix_per_step;
            while (ow >= p.OW) {
                ow -= p.OW;
                if (oh_left == 0) { oh_left = p.OH - 1; voh += KS; }  // next image: Hp - (OH-1)*STRIDE = KS
                else { --oh_left; voh += STRIDE; }
            }
        }
        uint32_t acc[TPX][kChanPerThread];
#pragma unroll
        for (int i = 0; i < TPX; ++i)
#pragma unroll
            for (int j = 0; j < kChanPerThread; ++j) acc[i][j] = 0u;

        uint32_t w_saddr = w_saddr0;
        const uint32_t *plane = sA;
        for (int cw = 0; cw < p.Cw; ++cw) {
#pragma unroll
            for (int g = 0; g < kNG; ++g) {
                // activation-side operands of nine-word group g: taps 9g .. 9g+8 in (ky, kx) order;
                // taps past the filter's last one are zero words on both sides and count nothing
                Triple at[TPX][3];
#pragma unroll
                for (int i = 0; i < TPX; ++i)
#pragma unroll
                    for (int k = 0; k < 3; ++k) {
                        uint32_t v[3];
#pragma unroll
                        for (int j = 0; j < 3; ++j) {
                            const int t = 9 * g + 3 * k + j;  // compile-time after unrolling
                            v[j] = t < kTaps ? plane[a_base[i] + (t / KS) * p.pitch + (t % KS)] : 0u;
                        }
                        at[i][k] = make_triple(v[0], v[1], v[2]);
                    }
                ChannelLoop<0, TPX>::run(w_saddr, at, k124, acc);
                w_saddr += kChanGroups * kWGroupStride * 4;
            }
            plane += p.plane;
        }

        // ---- output transform -------------------------------------------------------------
        ChannelParams cp;
        load_channel_params(p, chan, cp);
#pragma unroll
        for (int i = 0; i < TPX; ++i) {
            const int m = base + i * pix_per_step + warp * pix_per_warp + px;
            const bool pix_ok = m < m_end;
            int32_t v[kChanPerThread];
#pragma unroll
            for (int j = 0; j < kChanPerThread; ++j) v[j] = K - 2 * (int32_t)acc[i][j];
            if (p.padding == LCE_PAD_SAME_ZERO) {
                // zero-padding correction: taps outside the image contributed (+1)*w; take that out
                const int mm = pix_ok ? m : m0;
                const int r = mm / p.OW;
                const int iy0 = (r % p.OH) * STRIDE - p.pt, ix0 = (mm - r * p.OW) * STRIDE - p.pl;
#pragma unroll
                for (int t = 0; t < kTaps; ++t) {
                    const int iy = iy0 + t / KS, ix = ix0 + t % KS;
                    if (iy < 0 || iy >= p.H || ix < 0 || ix >= p.W) {
#pragma unroll
                        for (int j = 0; j < kChanPerThread; ++j) v[j] -= sWsum[(cg * kChanPerThread + j) * kMaxTaps + t];
                    }
                }
            }
            store_outputs(p, v, cp, m, pix_ok, cg, ch0, chan);
        }
    };
    for (int base = m0; base < m_end;) {
        if (kTailStep && TP > 2 && m_end - base <= 2 * pix_per_step) {
            step(std::integral_constant<int, 2>{}, base);
            base += 2 * pix_per_step;
        } else {
            step(std::integral_constant<int, TP>{}, base);
            base += TP * pix_per_step;
        }
    }
    // the next tile's rows have landed, and every warp is done reading this tile's
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
  }
}

// ---- pointwise (1x1) convolution ------------------------------------------------------------
// K runs over the channel words of one pixel only, so the nine-word carry-save groups are formed
// along the channel axis: words 9g .. 9g+8 of a pixel against the same words of a channel.  What
// is left after the full groups is handled as one or two triples (4 LOP3 + 2 POPC each).  The
// words past Cw are zero on both sides and so add nothing to the count.

__host__ __device__ __forceinline__ int pointwise_groups(int n9, int rem3) { return n9 + (rem3 > 0 ? 1 : 0); }

__global__ void __launch_bounds__(128)
pack_weights_pointwise_kernel(const uint32_t *__restrict__ w, uint32_t *__restrict__ image, int32_t Cout, int32_t Cw,
                              int32_t groups, int32_t chan_blocks)
{
    const int64_t entries = (int64_t)chan_blocks * kChanPerCta * groups;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < entries;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int g = (int)(e % groups);
        const int64_t c = e / groups;
        const int cb = (int)(c / kChanPerCta), ch = (int)(c % kChanPerCta);
        uint32_t wv[9];
#pragma unroll
        for (int t = 0; t < 9; ++t) wv[t] = (c < Cout && 9 * g + t < Cw) ? w[c * Cw + 9 * g + t] : 0u;
        uint32_t *block = image + cb * image_block_words(groups);
        store_w_operands(wv, block + w_offset(g, ch));
        if ((ch & 7) == 7) {
            uint32_t *pad = block + w_offset(g, ch) + kWRow;
            pad[0] = pad[1] = pad[2] = pad[3] = 0u;
        }
        if (g == 0) {  // per-tap sums are never used by a pointwise convolution (nothing is padded)
            int32_t *wsum = reinterpret_cast<int32_t *>(block + (int64_t)groups * kChanGroups * kWGroupStride);
            for (int t = 0; t < kMaxTaps; ++t) wsum[ch * kMaxTaps + t] = 0;
        }
    }
}

template <int J, int TP, int NT>
struct TailChannelLoop {
    // leftover triples: NT (1 or 2) triples per (pixel, channel)
    __device__ __forceinline__ static void run(uint32_t w_saddr, const Triple (&at)[TP][3], const Weights124 &k,
                                               uint32_t (&acc)[TP][kChanPerThread])
    {
        Triple wt[3];
        const uint4 q0 = lds128<J * 48>(w_saddr);
        wt[0].all = q0.x; wt[0].pair = q0.y; wt[0].first = q0.z;
        if (NT > 1) {
            const uint4 q1 = lds128<J * 48 + 16>(w_saddr);
            wt[1].all = q0.w; wt[1].pair = q1.x; wt[1].first = q1.y;
        }
#pragma unroll
        for (int i = 0; i < TP; ++i)
#pragma unroll
            for (int t = 0; t < NT; ++t) popc3_mad(at[i][t], wt[t], k, acc[i][J]);
        TailChannelLoop<J + 1, TP, NT>::run(w_saddr, at, k, acc);
    }
};
template <int TP, int NT>
struct TailChannelLoop<kChanPerThread, TP, NT> {
    __device__ __forceinline__ static void run(uint32_t, const Triple (&)[TP][3], const Weights124 &,
                                               uint32_t (&)[TP][kChanPerThread]) {}
};

// Copies the packed words of a tile's input pixels into shared memory as [pixel][cwp] (cwp = Cw
// rounded up to whole triples; the extra words are zero).
__device__ __forceinline__ void stage_pixels(const TiledParams &p, int m0, int m_end, uint32_t *sA, int tid)
{
    const int count = (m_end - m0) * p.cwp;
    for (int e = tid; e < count; e += kThreads) {
        const int l = e / p.cwp, cw = e - l * p.cwp;
        if (cw < p.Cw) {
            const int m = m0 + l;
            int64_t src_pix = m;
            if (p.stride != 1 || p.OW != p.W || p.OH != p.H) {
                const int r = m / p.OW, ow = m - r * p.OW;
                const int n = r / p.OH, oh = r - n * p.OH;
                src_pix = ((int64_t)n * p.H + oh * p.stride) * p.W + ow * p.stride;
            }
            cp_async4(sA + e, p.in + src_pix * p.Cw + cw);
        } else {
            sA[e] = 0u;
        }
    }
}

template <int TP>
__global__ void __launch_bounds__(kThreads, (TP <= 2 ? 24 : 16) / kWarps)
bconv1x1_kernel(const TiledParams p)
{
    extern __shared__ __align__(16) uint32_t smem[];
    const int groups = pointwise_groups(p.n9, p.rem3);
    const int w_words = groups * kChanGroups * kWGroupStride;
    uint32_t *sW = smem;
    uint32_t *sA0 = smem + w_words + kWsumWords;  // 2 x [tile_pixels][cwp]
    const int buf_words = p.tile_pixels * p.cwp;

    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const int ch0 = blockIdx.y * kChanPerCta;

    if (p.w_image != nullptr) {
        const uint32_t *src = p.w_image + blockIdx.y * image_block_words(groups);
        for (int e = tid * 4; e < w_words; e += kThreads * 4) cp_async16(smem + e, src + e);
        asm volatile("cp.async.commit_group;" ::: "memory");
    } else {
        for (int e = tid; e < kChanPerCta * groups; e += kThreads) {
            const int ch = e / groups;
            const int g = e - ch * groups;
            uint32_t wv[9];
#pragma unroll
            for (int t = 0; t < 9; ++t)
                wv[t] = (ch0 + ch < p.Cout && 9 * g + t < p.Cw) ? __ldg(p.w + (int64_t)(ch0 + ch) * p.Cw + 9 * g + t) : 0u;
            store_w_operands(wv, sW + w_offset(g, ch));
        }
    }

    const int px = lane >> 3, cg = lane & 7;
    const int chan = ch0 + cg * kChanPerThread;
    const int K = p.Cin;
    Weights124 k124;
    k124.one = p.N > 0 ? 1u : p.Cin;
    k124.two = p.N > 0 ? 2u : p.Cin;
    k124.four = p.N > 0 ? 4u : p.Cin;
    asm volatile("" : "+r"(k124.one), "+r"(k124.two), "+r"(k124.four));
    const uint32_t w_saddr0 = (uint32_t)__cvta_generic_to_shared(sW + cg * kWGroupStride);

    int tile = blockIdx.x;
    if (tile < p.n_tiles) stage_pixels(p, tile * p.tile_pixels, min((tile + 1) * p.tile_pixels, p.M), sA0, tid);
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

    for (int buf = 0; tile < p.n_tiles; tile += gridDim.x, buf ^= 1) {
        const uint32_t *sA = sA0 + buf * buf_words;
        const int m0 = tile * p.tile_pixels;
        const int m_end = min(m0 + p.tile_pixels, p.M);
        {
            const int next = tile + gridDim.x;
            if (next < p.n_tiles)
                stage_pixels(p, next * p.tile_pixels, min((next + 1) * p.tile_pixels, p.M), sA0 + (buf ^ 1) * buf_words, tid);
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        for (int base = m0; base < m0 + p.tile_pixels; base += kPixPerStep * TP) {
            uint32_t acc[TP][kChanPerThread];
#pragma unroll
            for (int i = 0; i < TP; ++i)
#pragma unroll
                for (int j = 0; j < kChanPerThread; ++j) acc[i][j] = 0u;
            const uint32_t *apix[TP];
#pragma unroll
            for (int i = 0; i < TP; ++i) {
                const int m = base + i * kPixPerStep + warp * 4 + px;
                apix[i] = sA + (m < m_end ? (m - m0) * p.cwp : 0);  // past the end: redo pixel 0, store nothing
            }
            uint32_t w_saddr = w_saddr0;
            for (int g = 0; g < p.n9; ++g) {
                Triple at[TP][3];
#pragma unroll
                for (int i = 0; i < TP; ++i)
#pragma unroll
                    for (int t = 0; t < 3; ++t) {
                        const uint32_t *q = apix[i] + 9 * g + 3 * t;
                        at[i][t] = make_triple(q[0], q[1], q[2]);
                    }
                ChannelLoop<0, TP>::run(w_saddr, at, k124, acc);
                w_saddr += kChanGroups * kWGroupStride * 4;
            }
            if (p.rem3 > 0) {
                Triple at[TP][3];
#pragma unroll
                for (int i = 0; i < TP; ++i)
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        const uint32_t *q = apix[i] + 9 * p.n9 + 3 * (t < p.rem3 ? t : 0);
                        at[i][t] = make_triple(q[0], q[1], q[2]);
                    }
                if (p.rem3 == 1) TailChannelLoop<0, TP, 1>::run(w_saddr, at, k124, acc);
                else TailChannelLoop<0, TP, 2>::run(w_saddr, at, k124, acc);
            }
            ChannelParams cp;
            load_channel_params(p, chan, cp);
#pragma unroll
            for (int i = 0; i < TP; ++i) {
                const int m = base + i * kPixPerStep + warp * 4 + px;
                int32_t v[kChanPerThread];
#pragma unroll
                for (int j = 0; j < kChanPerThread; ++j) v[j] = K - 2 * (int32_t)acc[i][j];
                store_outputs(p, v, cp, m, m < m_end, cg, ch0, chan);
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
    }
}

template <int TP>
lce_status launch1x1(const TiledParams &p, size_t smem_bytes, dim3 grid, cudaStream_t s)
{
    auto kernel = bconv1x1_kernel<TP>;
    if (smem_bytes > 48 * 1024) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess)
            return LCE_ERR_CUDA;
    }
    kernel<<<grid, kThreads, smem_bytes, s>>>(p);
    return launch_status();
}

template <int KS, int STRIDE, int TP, int NW, bool F32 = false>
lce_status launch_kxk(const TiledParams &p, size_t smem_bytes, dim3 grid, cudaStream_t s)
{
    auto kernel = bconv3x3_kernel<KS, STRIDE, TP, NW, F32>;
    if (smem_bytes > 48 * 1024) {
        // opt in to the large dynamic shared memory carve-out
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess)
            return LCE_ERR_CUDA;
    }
    kernel<<<grid, 32 * NW, smem_bytes, s>>>(p);
    return launch_status();
}

// CTAs of 128 threads that the register file lets share an SM, per pixels-per-thread variant
// (must match the __launch_bounds__ of the kernel).
int reg_limited_ctas(int tp, int nw) { return (tp <= 2 ? 24 : 16) / nw; }

size_t smem_bytes_for(const ConvGeom &g, const TiledParams &p)
{
    return ((size_t)g.Cw * groups_per_word(g.KH) * kChanGroups * kWGroupStride + kWsumWords + 2 * (size_t)g.Cw * p.plane) * 4;
}

void set_tile(const ConvGeom &g, TiledParams *p, int tile_pixels)
{
    p->tile_pixels = tile_pixels;
    int rows_max = (tile_pixels - 1) / g.OW + 2;  // output rows a run of tile_pixels flat pixels can touch
    if (rows_max > tile_pixels) rows_max = tile_pixels;
    const int nv_max = (rows_max - 1) * g.KH + g.KH;  // consecutive output rows are at most KH virtual rows apart
    p->plane = nv_max * p->pitch;
}

bool covers3x3(const ConvGeom &g) { return g.KH == g.KW && (g.KH == 3 || g.KH == 5) && g.sh == g.sw && g.sh <= 2; }
bool covers1x1(const ConvGeom &g) { return g.KH == 1 && g.KW == 1 && g.sh == g.sw; }

bool tiled_covers(const ConvGeom &g)
{
    return (covers3x3(g) || covers1x1(g)) && g.M < (1ll << 31) - 256 &&
           (g.Cout + kChanPerCta - 1) / kChanPerCta <= 65535;
}

void pointwise_split(int Cw, int *n9, int *rem3)
{
    *n9 = Cw / 9;
    const int rem = Cw % 9;
    if (rem > 6) { ++*n9; *rem3 = 0; }
    else *rem3 = (rem + 2) / 3;
}

int image_groups(const ConvGeom &g)
{
    if (covers3x3(g)) return g.Cw * groups_per_word(g.KH);
    int n9, rem3;
    pointwise_split(g.Cw, &n9, &rem3);
    return pointwise_groups(n9, rem3);
}

#ifndef LCE_MAX_ROUNDS
#define LCE_MAX_ROUNDS 8
#endif
constexpr int kMaxRounds = LCE_MAX_ROUNDS;

struct TileChoice {
    int tp, tile, ctas_x, ctas_half, range_full, range_half;
    double cost;
};

// Pixels per thread (TP) and tile size: a tile covers 16*TP*rounds flat pixels and the grid is
// persistent (each CTA walks tiles x, x + gridDim.x, ...).  Pick the pair that balances the SMs
// best: cost = (CTAs on the busiest SM) x (tiles of the busiest CTA) x (tile work), with a
// penalty when too few warps share an SM to keep the logic pipe busy.
template <typename SmemFn>
bool choose_tile(const ConvGeom &g, int chan_blocks, SmemFn smem_for_tile, TileChoice *best, int nw = kWarps,
                 size_t smem_limit = 110 * 1024, bool has_half_block = false, bool ranged = false, bool allow_tp1 = false)
{
    int sms = 148;
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    int forced_tp = 0, forced_rounds = 0;
#ifdef LCE_TUNING
    if (const char *e = getenv("LCE_TP")) forced_tp = atoi(e);
    if (const char *e = getenv("LCE_ROUNDS")) forced_rounds = atoi(e);
#endif
    double best_cost = 0;
    best->tile = 0;
    // one pixel per thread exists for the KxK kernel with 4-warp CTAs only: the finest split of a
    // single image over the SMs (latency, not throughput)
    for (int tp = (ranged && nw == 4 && allow_tp1) ? 1 : 2; tp <= 4; ++tp) {
        if (forced_tp && tp != forced_tp) continue;
        const int unit = 4 * nw * tp;
        for (int rounds = 1; rounds <= kMaxRounds; ++rounds) {
            if (forced_rounds && rounds != forced_rounds) continue;
            // a half channel block takes two units of pixels per step
            if (has_half_block && (rounds & 1)) continue;
            const int tile = unit * rounds;
            const size_t smem = smem_for_tile(tile);
            if (smem > smem_limit) continue;
            int per_sm = (int)((220 * 1024) / (smem + 1024));
            if (per_sm < 1) per_sm = 1;
            if (per_sm > reg_limited_ctas(tp, nw)) per_sm = reg_limited_ctas(tp, nw);
            const double smem_penalty[5] = {0, 1.2, 1.06, 1.02, 1.0};  // fewer pixels per thread re-read the weight operands more often
            const int full_blocks = has_half_block ? chan_blocks - 1 : chan_blocks;
            const int64_t slots = (int64_t)sms * per_sm;
            int64_t ctas_x, ctas_half = 0, range_full = 0, range_half = 0;
            double t_cta;  // time of the busiest CTA, in pixel-steps of a full block
            if (ranged) {
                // KxK kernel: a CTA owns a contiguous range of pixels, a whole number of granules; a
                // granule is the smallest step the kernel has (2 pixels per thread when TP > 2)
                const bool tail = kTailStep && tp > 2;
                const int64_t pps = 4 * nw;                     // pixels per step and pixel-per-thread, full block
                const int64_t granule = tail ? pps : unit;      // ranges are whole numbers of granules
                // per tile: barrier bubbles and the halo rows that are staged again (measured at
                // 56x56x64: about a fifth of the time of computing those rows)
                const double tile_overhead = 4.0 + 0.2 * (g.KH - 1) * g.OW;
                auto range_for = [&](int64_t ctas, int64_t gran) { return ((g.M + ctas - 1) / ctas + gran - 1) / gran * gran; };
                auto time_of = [&](int64_t range, int pixel_scale) {  // pixel_scale 2: a half block's step covers twice the pixels
                    double t = (double)((range + tile - 1) / tile) * tile_overhead;
                    for (int64_t r = range / pixel_scale; r > 0;) {  // the kernel's own decomposition into steps
                        if (tail && r <= 2 * pps) { t += 2 * pps * smem_penalty[2]; r = 0; }
                        else { t += unit * smem_penalty[tp]; r -= unit; }
                    }
                    return t;
                };
                ctas_x = has_half_block ? (2 * slots) / (2 * full_blocks + 1) : slots / chan_blocks;
                if (ctas_x < 1) ctas_x = 1;
                t_cta = 0;
                if (full_blocks > 0) {
                    range_full = range_for(ctas_x, granule);
                    ctas_x = (g.M + range_full - 1) / range_full;
                    t_cta = time_of(range_full, 1);
                }
                if (has_half_block) {
                    ctas_half = full_blocks > 0 ? (ctas_x + 1) / 2 : (slots < 1 ? 1 : slots);
                    range_half = range_for(ctas_half, 2 * granule);
                    ctas_half = (g.M + range_half - 1) / range_half;
                    const double t_half = time_of(range_half, 2);
                    if (t_half > t_cta) t_cta = t_half;
                }
            } else {
                const int64_t n_tiles = (g.M + tile - 1) / tile;
                ctas_x = slots / chan_blocks;
                if (ctas_x < 1) ctas_x = 1;
                if (ctas_x > n_tiles) ctas_x = n_tiles;
                t_cta = (double)((n_tiles + ctas_x - 1) / ctas_x) * (tile * smem_penalty[tp] + 4.0);
            }
            const int64_t total_ctas = ctas_x * full_blocks + ctas_half;
            const int64_t ctas_on_sm = (total_ctas + sms - 1) / sms;
            const double warps = (double)total_ctas / sms * nw;
            const double eff = warps >= 16 ? 1.0 : (warps >= 8 ? 0.8 + 0.2 * (warps - 8) / 8 : 0.4 + 0.4 * warps / 8);
            const double cost = (double)ctas_on_sm * t_cta / eff;
            if (best->tile == 0 || cost < best_cost) {
                best->tile = tile; best->tp = tp; best->ctas_x = (int)ctas_x; best->ctas_half = (int)ctas_half;
                best->range_full = (int)range_full; best->range_half = (int)range_half;
                best_cost = best->cost = cost;
            }
        }
    }
    return best->tile != 0;
}

}  // namespace

size_t tiled_weight_image_bytes(const ConvGeom &g)
{
    if (!tiled_covers(g)) return 0;
    const int chan_blocks = (g.Cout + kChanPerCta - 1) / kChanPerCta;
    return (size_t)chan_blocks * image_block_words(image_groups(g)) * 4;
}

lce_status launch_pack_weights_tiled(const ConvGeom &g, const uint32_t *w, uint32_t *image, cudaStream_t s)
{
    if (!tiled_covers(g)) return LCE_ERR_UNSUPPORTED;
    const int chan_blocks = (g.Cout + kChanPerCta - 1) / kChanPerCta;
    const int groups = image_groups(g);
    const int64_t entries = (int64_t)chan_blocks * kChanPerCta * groups;
    int blocks = (int)((entries + 127) / 128);
    if (blocks > 148 * 8) blocks = 148 * 8;
    if (covers3x3(g))
        pack_weights_kernel<<<blocks, 128, 0, s>>>(w, image, g.Cout, g.Cw, g.Cin, chan_blocks, g.KH);
    else
        pack_weights_pointwise_kernel<<<blocks, 128, 0, s>>>(w, image, g.Cout, g.Cw, groups, chan_blocks);
    return launch_status();
}

// Everything the launch needs that does not depend on the buffers: geometry fields of the kernel
// parameters, the chosen variant and the launch dimensions.
struct TiledPlan {
    bool pointwise;
    int nw, tp;
    size_t smem_bytes;
    dim3 grid;
};

static lce_status plan_tiled(const ConvGeom &g, bool f32_input, TiledParams *pp, TiledPlan *plan)
{
    TiledParams &p = *pp;
    if (!tiled_covers(g)) return LCE_ERR_UNSUPPORTED;
    if (f32_input && !covers3x3(g)) return LCE_ERR_UNSUPPORTED;
    p.N = g.N; p.H = g.H; p.W = g.W; p.Cin = g.Cin; p.Cw = g.Cw; p.Cout = g.Cout; p.Cow = g.Cow;
    p.OH = g.OH; p.OW = g.OW; p.pt = g.pt; p.pl = g.pl;
    p.padding = g.padding; p.out_type = g.out_type; p.activation = g.activation;
    p.M = (int32_t)g.M;
    p.stride = g.sh;
    p.cw_shift = -1;
    p.half_block = -1;
    for (int b = 0; b < 16; ++b)
        if ((1 << b) == g.Cw) p.cw_shift = b;
    const int chan_blocks = (g.Cout + kChanPerCta - 1) / kChanPerCta;
    TileChoice c;

    if (covers1x1(g)) {
        pointwise_split(g.Cw, &p.n9, &p.rem3);
        p.cwp = 9 * p.n9 + 3 * p.rem3;
        const int groups = pointwise_groups(p.n9, p.rem3);
        auto smem_for = [&](int tile) {
            return ((size_t)groups * kChanGroups * kWGroupStride + kWsumWords + 2 * (size_t)tile * p.cwp) * 4;
        };
        if (!choose_tile(g, chan_blocks, smem_for, &c)) return LCE_ERR_UNSUPPORTED;
        p.tile_pixels = c.tile;
        p.n_tiles = (int32_t)((g.M + c.tile - 1) / c.tile);
        plan->pointwise = true;
        plan->nw = kWarps;
        plan->tp = c.tp;
        plan->grid = dim3((unsigned)c.ctas_x, (unsigned)chan_blocks, 1);
        plan->smem_bytes = smem_for(c.tile);
        return LCE_OK;
    }

    p.Hp = (g.OH - 1) * g.sh + g.KH;
    p.Wp = (g.OW - 1) * g.sh + g.KW;
    if (p.Wp < g.W + g.pl) p.Wp = g.W + g.pl;  // staging writes the whole image row; columns past the taps are unused
    p.pitch = p.Wp | 1;  // odd pitch: the 4 pixels of a warp in 4 different rows hit 4 different banks
    auto smem_for = [&](int tile) {
        set_tile(g, &p, tile);
        return smem_bytes_for(g, p);
    };
    // Candidates: CTAs of 8 or 4 warps (eight warps share one copy of the weight operands and one
    // staging buffer, which measures faster wherever whole tiles of 32*TP pixels are useful work;
    // four-warp CTAs remain for problems too small for that), with or without the half-block lane
    // mapping (which needs tiles of two units: not worth it on very small problems).
    const int tail_channels = g.Cout % kChanPerCta;
    const bool can_half = tail_channels >= 1 && tail_channels <= kChanPerCta / 2;
    int nw = 0;
    bool half = false;
    c.cost = 0;
    for (int use_half = can_half ? 1 : 0; use_half >= 0; --use_half) {
        for (int w = 8; w >= 4; w -= 4) {
            if (w == 8 && f32_input) continue;  // the float-input loader exists for four-warp CTAs only
            TileChoice t;
            bool ok = choose_tile(g, chan_blocks, smem_for, &t, w, w == 8 ? 226 * 1024 : 110 * 1024, use_half != 0, true, !f32_input);
            if (!ok && w == 4 && f32_input)
                ok = choose_tile(g, chan_blocks, smem_for, &t, 4, 226 * 1024, use_half != 0, true);
            if (ok && (nw == 0 || t.cost < c.cost)) { c = t; nw = w; half = use_half != 0; }
        }
    }
    if (nw == 0) return LCE_ERR_UNSUPPORTED;
#ifdef LCE_TUNING
    {
        const char *e_nw = getenv("LCE_NW"), *e_half = getenv("LCE_HALF");
        if (e_nw || e_half) {
            const int want_nw = e_nw ? atoi(e_nw) : nw;
            const bool want_half = e_half ? (atoi(e_half) != 0 && can_half) : half;
            TileChoice t;
            if (choose_tile(g, chan_blocks, smem_for, &t, want_nw, 226 * 1024, want_half, true, !f32_input)) { c = t; nw = want_nw; half = want_half; }
        }
    }
#endif
    set_tile(g, &p, c.tile);
    p.n_tiles = (int32_t)((g.M + c.tile - 1) / c.tile);
    p.half_block = half ? chan_blocks - 1 : -1;
    p.full_blocks = half ? chan_blocks - 1 : chan_blocks;
    p.ctas_full = c.ctas_x;
    p.ctas_half = half ? c.ctas_half : 0;
    p.range_full = c.range_full;
    p.range_half = c.range_half;
    plan->pointwise = false;
    plan->nw = nw;
    plan->tp = c.tp;
    plan->smem_bytes = smem_bytes_for(g, p);
    plan->grid = dim3((unsigned)(p.full_blocks * p.ctas_full + p.ctas_half), 1, 1);
#ifdef LCE_TUNING
    if (getenv("LCE_VERBOSE"))
        fprintf(stderr, "tiled %dx%d M=%lld Cw=%d Cout=%d: nw=%d tp=%d tile=%d grid=%dx%d+%d range=%d/%d smem=%zu cost=%.0f\n", g.KH, g.KW,
                (long long)g.M, g.Cw, g.Cout, nw, c.tp, c.tile, p.ctas_full, p.full_blocks, p.ctas_half, p.range_full, p.range_half,
                plan->smem_bytes, c.cost);
#endif
    return LCE_OK;
}

lce_status tiled_plan_info(const ConvGeom &g, TiledPlanInfo *info)
{
    TiledParams p{};
    TiledPlan plan{};
    const lce_status st = plan_tiled(g, false, &p, &plan);
    if (st != LCE_OK) return st;
    info->pointwise = plan.pointwise ? 1 : 0;
    info->warps_per_cta = plan.nw;
    info->pixels_per_thread = plan.tp;
    info->tile_pixels = p.tile_pixels;
    info->ctas = (int32_t)(plan.grid.x * plan.grid.y);
    info->ctas_half_block = plan.pointwise ? 0 : p.ctas_half;
    info->pixels_per_cta = plan.pointwise ? 0 : p.range_full;
    info->pixels_per_cta_half_block = plan.pointwise ? 0 : p.range_half;
    info->shared_bytes = (int64_t)plan.smem_bytes;
    return LCE_OK;
}

lce_status launch_bconv_tiled(const ConvGeom &g, const uint32_t *in, const uint32_t *w, const uint32_t *w_image,
                              const float *mult, const float *bias, const int32_t *thr, void *out, cudaStream_t s,
                              const float *residual, uint32_t *out_packed, const float *in_f32)
{
    // 128-bit epilogue accesses need 16-byte aligned buffers when the channel count allows them
    if ((g.Cout & 3) == 0 && g.out_type != LCE_OUT_BITPACKED && (!aligned(out, 16) || !aligned(residual, 16)))
        return LCE_ERR_UNSUPPORTED;
    if (w_image && !aligned(w_image, 16)) return LCE_ERR_ALIGNMENT;
    TiledParams p{};
    TiledPlan plan{};
    const lce_status st = plan_tiled(g, in_f32 != nullptr, &p, &plan);
    if (st != LCE_OK) return st;
    p.in = in; p.w = w; p.w_image = w_image; p.mult = mult; p.bias = bias; p.thr = thr; p.out = out;
    p.residual = residual; p.out_packed = out_packed; p.in_f32 = in_f32;
    const size_t smem_bytes = plan.smem_bytes;
    const dim3 grid = plan.grid;
    const int nw = plan.nw;
    struct { int tp; } c{plan.tp};
    if (plan.pointwise) {
        if (c.tp == 2) return launch1x1<2>(p, smem_bytes, grid, s);
        if (c.tp == 3) return launch1x1<3>(p, smem_bytes, grid, s);
        return launch1x1<4>(p, smem_bytes, grid, s);
    }
#define LCE_LAUNCH_TP(KS, ST, NW)                                                   \
    do {                                                                            \
        if (c.tp == 1) return launch_kxk<KS, ST, 1, 4>(p, smem_bytes, grid, s);     \
        if (c.tp == 2) return launch_kxk<KS, ST, 2, NW>(p, smem_bytes, grid, s);    \
        if (c.tp == 3) return launch_kxk<KS, ST, 3, NW>(p, smem_bytes, grid, s);    \
        return launch_kxk<KS, ST, 4, NW>(p, smem_bytes, grid, s);                   \
    } while (0)
    if (in_f32) {
#define LCE_LAUNCH_F32(KS, ST)                                                         \
    do {                                                                               \
        if (c.tp == 2) return launch_kxk<KS, ST, 2, 4, true>(p, smem_bytes, grid, s);  \
        if (c.tp == 3) return launch_kxk<KS, ST, 3, 4, true>(p, smem_bytes, grid, s);  \
        return launch_kxk<KS, ST, 4, 4, true>(p, smem_bytes, grid, s);                 \
    } while (0)
        if (g.KH == 3 && g.sh == 1) LCE_LAUNCH_F32(3, 1);
        if (g.KH == 3) LCE_LAUNCH_F32(3, 2);
        if (g.sh == 1) LCE_LAUNCH_F32(5, 1);
        LCE_LAUNCH_F32(5, 2);
#undef LCE_LAUNCH_F32
    }
    if (g.KH == 3 && g.sh == 1) { if (nw == 8) LCE_LAUNCH_TP(3, 1, 8); else LCE_LAUNCH_TP(3, 1, 4); }
    if (g.KH == 3) { if (nw == 8) LCE_LAUNCH_TP(3, 2, 8); else LCE_LAUNCH_TP(3, 2, 4); }
    if (g.sh == 1) { if (nw == 8) LCE_LAUNCH_TP(5, 1, 8); else LCE_LAUNCH_TP(5, 1, 4); }
    if (nw == 8) LCE_LAUNCH_TP(5, 2, 8); else LCE_LAUNCH_TP(5, 2, 4);
#undef LCE_LAUNCH_TP
}

}  // namespace lce
