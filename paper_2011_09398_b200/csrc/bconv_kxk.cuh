// The 3x3 / 5x5 tiled kernel: input-row staging (packed words, or fp32 activations binarized on
// the way in) and the kernel itself.  Included by bconv_tiled.cu after tiled_common.cuh.
#pragma once

#include <type_traits>

#include "tiled_common.cuh"

namespace lce {
namespace {

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

template <int J, int TP>
struct ChannelLoopPacked {
    __device__ __forceinline__ static void run(uint32_t w_saddr, const Triple (&at)[TP][3], const Weights124 &k, const Weights124 &khi,
                                               uint32_t (&acc)[(TP + 1) / 2][kChanPerThread])
    {
        Triple wt[3];
        load_w_triples<J>(w_saddr, wt);
        popc9_mad_pixels_packed<TP, kChanPerThread, J>(at, wt, k, khi, acc);
        ChannelLoopPacked<J + 1, TP>::run(w_saddr, at, k, khi, acc);
    }
};
template <int TP>
struct ChannelLoopPacked<kChanPerThread, TP> {
    __device__ __forceinline__ static void run(uint32_t, const Triple (&)[TP][3], const Weights124 &, const Weights124 &,
                                               uint32_t (&)[(TP + 1) / 2][kChanPerThread]) {}
};

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

    // Programmatic dependent launch: the next kernel of the stream may be scheduled from here on; this one
    // fetches its weights (constants of the model) and waits for the previous kernel only before it touches
    // the activations, the shortcut tensor or its outputs.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

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
    // float output: accumulators carry the bias that makes int -> float one exact subtraction
    const bool biased = p.out_type == LCE_OUT_FLOAT32 && K < kMaxBiasedK;
    const int Kb = biased ? K + kFloatBias : K;
    const int epi = epilogue_mode(p, chan, biased);
    Weights124 k124;
    k124.one = p.N > 0 ? 1u : p.Cin;  // opaque to the compiler: keeps the weighted sum on multiply-adds
    k124.two = p.N > 0 ? 2u : p.Cin;
    k124.four = p.N > 0 ? 4u : p.Cin;
    asm volatile("" : "+r"(k124.one), "+r"(k124.two), "+r"(k124.four));
    Weights124 khi;  // the same multipliers for the pixel kept in the high half of an accumulator
    khi.one = p.N > 0 ? (1u << 16) : p.Cin;
    khi.two = p.N > 0 ? (2u << 16) : p.Cin;
    khi.four = p.N > 0 ? (4u << 16) : p.Cin;
    asm volatile("" : "+r"(khi.one), "+r"(khi.two), "+r"(khi.four));
    const uint32_t w_saddr0 = (uint32_t)__cvta_generic_to_shared(sW + cg * kWGroupStride);

    // ---- loop over the tiles of this CTA's range; the next tile's input rows are copied into the
    // other buffer while the current tile is computed ---------------------------------------------
    asm volatile("griddepcontrol.wait;" ::: "memory");
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
        constexpr int HX = (TPX + 1) / 2;  // two pixels' 16-bit counts per accumulator register
        uint32_t acc[HX][kChanPerThread];
#pragma unroll
        for (int i = 0; i < HX; ++i)
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
                ChannelLoopPacked<0, TPX>::run(w_saddr, at, k124, khi, acc);
                w_saddr += kChanGroups * kWGroupStride * 4;
            }
            plane += p.plane;
        }

        // ---- output transform -------------------------------------------------------------
        ChannelParams cp;
        load_channel_params(p, chan, cp);
        if (epi == kEpiBits && K < 32768) {
            // bit-packed output without a padding correction: nothing to decide per pixel, and the
            // compare works on the packed counts directly
            int32_t c15[kChanPerThread];
            packed_compare_operands(cp.thr, K, c15);
#pragma unroll
            for (int i = 0; i < TPX; ++i) {
                const int m = base + i * pix_per_step + warp * pix_per_warp + px;
                const uint32_t bits = i < HX ? packed_compare_bits<false>(acc[i], c15) : packed_compare_bits<true>(acc[i - HX < 0 ? 0 : i - HX], c15);
                store_bits_byte(p, bits, m, m < m_end, cg, ch0);
            }
            return;
        }
        if (epi == kEpiBits) {
#pragma unroll
            for (int i = 0; i < TPX; ++i) {
                const int m = base + i * pix_per_step + warp * pix_per_warp + px;
                int32_t v[kChanPerThread];
#pragma unroll
                for (int j = 0; j < kChanPerThread; ++j)
                    v[j] = Kb - 2 * (int32_t)(i < HX ? (acc[i][j] & 0xFFFFu) : (acc[i - HX][j] >> 16));
                store_bits(p, v, cp.thr, m, m < m_end, cg, ch0);
            }
            return;
        }
#pragma unroll
        for (int i = 0; i < TPX; ++i) {
            const int m = base + i * pix_per_step + warp * pix_per_warp + px;
            const bool pix_ok = m < m_end;
            int32_t v[kChanPerThread];
#pragma unroll
            for (int j = 0; j < kChanPerThread; ++j)
                v[j] = Kb - 2 * (int32_t)(i < HX ? (acc[i][j] & 0xFFFFu) : (acc[i - HX][j] >> 16));
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
            store_outputs(p, v, cp, m, pix_ok, cg, ch0, chan, biased, epi);
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

}  // namespace
}  // namespace lce
