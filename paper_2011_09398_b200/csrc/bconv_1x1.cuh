// The pointwise (1x1) tiled kernel and its load-time weight packing.  Included by bconv_tiled.cu
// after tiled_common.cuh.
#pragma once

#include "tiled_common.cuh"

namespace lce {
namespace {

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

    // programmatic dependent launch, as in the KxK kernel: weights before the dependency wait, everything
    // the previous kernel may have written after it
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

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
    const bool biased = p.out_type == LCE_OUT_FLOAT32 && K < kMaxBiasedK;
    const int Kb = biased ? K + kFloatBias : K;
    const int epi = epilogue_mode(p, chan, biased);
    Weights124 k124;
    k124.one = p.N > 0 ? 1u : p.Cin;
    k124.two = p.N > 0 ? 2u : p.Cin;
    k124.four = p.N > 0 ? 4u : p.Cin;
    asm volatile("" : "+r"(k124.one), "+r"(k124.two), "+r"(k124.four));
    const uint32_t w_saddr0 = (uint32_t)__cvta_generic_to_shared(sW + cg * kWGroupStride);

    int tile = blockIdx.x;
    asm volatile("griddepcontrol.wait;" ::: "memory");
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
            if (epi == kEpiBits && K < (1 << 29)) {
                // acc < thr  <=>  c - 2*count < 0 with c = K - thr (threshold clamped to [-K-1, K+1]):
                // the output bit is the sign bit of one multiply-add, collected by a funnel shift
                int32_t c[kChanPerThread];
#pragma unroll
                for (int j = 0; j < kChanPerThread; ++j) c[j] = K - max(-K - 1, min(K + 1, cp.thr[j]));
#pragma unroll
                for (int i = 0; i < TP; ++i) {
                    const int m = base + i * kPixPerStep + warp * 4 + px;
                    uint32_t bits = 0u;
#pragma unroll
                    for (int j = kChanPerThread - 1; j >= 0; --j)
                        bits = __funnelshift_l((uint32_t)c[j] - 2u * acc[i][j], bits, 1);
                    store_bits_byte(p, bits, m, m < m_end, cg, ch0);
                }
                continue;
            }
#pragma unroll
            for (int i = 0; i < TP; ++i) {
                const int m = base + i * kPixPerStep + warp * 4 + px;
                int32_t v[kChanPerThread];
#pragma unroll
                for (int j = 0; j < kChanPerThread; ++j) v[j] = Kb - 2 * (int32_t)acc[i][j];
                store_outputs(p, v, cp, m, m < m_end, cg, ch0, chan, biased, epi);
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
    }
}

}  // namespace
}  // namespace lce
