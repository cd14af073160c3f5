// LceBConv2d for very few input channels (an RGB first layer): when KH*KW*Cin <= 32 the whole
// receptive field of an output pixel fits in ONE 32-bit word.  The paper pads the channel axis to
// a multiple of 32 (Section 3.2, LceQuantize), which for Cin = 3 spends nine word operations per
// output on 27 useful bits; here the taps' Cin bits are first gathered into a single "patch"
// word per pixel (im2col at bit granularity), the weights of a channel into a matching word, and
// the accumulator is K - 2*popcount(patch XOR weight word): one XOR + POPC per output.
// A thread owns one output pixel and walks all output channels, 32 at a time, so that it can
// write whole bit-packed output words without any cross-lane traffic.
#include "common.cuh"

namespace lce {
namespace {

constexpr int kThreads = 256;

struct PatchParams {
    const uint32_t *in;
    const uint32_t *w;
    const float *mult;
    const float *bias;
    const int32_t *thr;
    void *out;
    int32_t N, H, W, Cin, Cout, Cow, KH, KW, sh, sw, OH, OW, pt, pl;
    int32_t M, padding, out_type, activation;
};

__global__ void __launch_bounds__(kThreads)
bconv_patch_kernel(const PatchParams p)
{
    extern __shared__ __align__(16) uint32_t smem[];
    const int taps = p.KH * p.KW;
    const int cout_pad = p.Cow * 32;
    uint32_t *sWord = smem;                                             // [cout_pad] weight patch words
    int32_t *sThr = reinterpret_cast<int32_t *>(smem + cout_pad);       // [cout_pad]
    int32_t *sWsum = reinterpret_cast<int32_t *>(smem + 2 * cout_pad);  // [cout_pad][taps], zero-padding only
    // then [cout_pad] (word, popcount threshold) pairs for the bit-packed fast path
    const uint32_t mask = p.Cin >= 32 ? 0xffffffffu : ((1u << p.Cin) - 1u);

    for (int o = threadIdx.x; o < cout_pad; o += kThreads) {
        uint32_t word = 0u;
        if (o < p.Cout)
            for (int t = 0; t < taps; ++t) word |= (__ldg(p.w + (int64_t)o * taps + t) & mask) << (t * p.Cin);
        sWord[o] = word;
        sThr[o] = (o < p.Cout && p.out_type == LCE_OUT_BITPACKED) ? __ldg(p.thr + o) : INT32_MIN;  // pad bits -> 0
    }
    if (p.padding == LCE_PAD_SAME_ZERO) {
        for (int e = threadIdx.x; e < cout_pad * taps; e += kThreads) {
            const int o = e / taps, t = e - o * taps;
            // sum of one tap's weights over the true channels
            sWsum[e] = o < p.Cout ? p.Cin - 2 * __popc(__ldg(p.w + (int64_t)o * taps + t) & mask) : 0;
        }
    }
    __syncthreads();

    const int K = taps * p.Cin;

    if (p.out_type == LCE_OUT_BITPACKED && p.padding != LCE_PAD_SAME_ZERO) {
        // Bit-packed output without a zero-padding correction (the stem of a binarized network):
        // acc < thr  <=>  K - 2*popc < thr  <=>  popc > floor((K - thr) / 2), so a channel is one
        // 64-bit shared-memory read (weight word, popcount threshold), XOR, POPC, compare, OR.  Two
        // pixels per thread share that read.
        __syncthreads();  // sWord / sThr are complete; rewrite them as (word, popcount threshold) pairs
        uint2 *sPair = reinterpret_cast<uint2 *>(smem + (2 + taps) * cout_pad);
        for (int o = threadIdx.x; o < cout_pad; o += kThreads) {
            int32_t t = INT32_MAX;  // pad channels: never set
            if (o < p.Cout) t = (int32_t)(((int64_t)K - (int64_t)sThr[o]) >> 1);
            sPair[o] = make_uint2(sWord[o], (uint32_t)t);
        }
        __syncthreads();
        const int64_t stride = (int64_t)gridDim.x * kThreads;
        // (image, row, column) of the thread's two pixels, advanced by 2*stride pixels per iteration
        // with carries instead of two divisions per pixel
        const int64_t step = 2 * stride;
        const int step_ow = (int)(step % p.OW);
        const int64_t step_rows = step / p.OW;
        const int step_oh = (int)(step_rows % p.OH), step_n = (int)(step_rows / p.OH);
        int pn[2], poh[2], pow_[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int64_t m = (int64_t)blockIdx.x * kThreads + threadIdx.x + q * stride;
            const int64_t r = m / p.OW;
            pow_[q] = (int)(m - r * p.OW);
            pn[q] = (int)(r / p.OH);
            poh[q] = (int)(r - (int64_t)pn[q] * p.OH);
        }
        for (int64_t m0 = (int64_t)blockIdx.x * kThreads + threadIdx.x; m0 < p.M; m0 += step) {
            const int64_t mm[2] = {m0, m0 + stride};
            uint32_t patch[2] = {0u, 0u};
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int n = pn[q], oh = poh[q], ow = pow_[q];
                pow_[q] += step_ow;
                poh[q] += step_oh;
                pn[q] += step_n;
                if (pow_[q] >= p.OW) { pow_[q] -= p.OW; ++poh[q]; }
                if (poh[q] >= p.OH) { poh[q] -= p.OH; ++pn[q]; }
                if (mm[q] >= p.M) continue;
                const int iy0 = oh * p.sh - p.pt, ix0 = ow * p.sw - p.pl;
                const uint32_t *img = p.in + (int64_t)n * p.H * p.W;
                if (taps == 9 && p.KW == 3 && iy0 >= 0 && iy0 + 2 < p.H && ix0 >= 0 && ix0 + 2 < p.W) {
                    // 3x3 window inside the image (all but the border pixels): nine loads from three row
                    // pointers, nothing to test per tap
                    const uint32_t *r0 = img + iy0 * p.W + ix0, *r1 = r0 + p.W, *r2 = r1 + p.W;
                    uint32_t v[9];
#pragma unroll
                    for (int kx = 0; kx < 3; ++kx) {
                        v[kx] = __ldg(r0 + kx);
                        v[3 + kx] = __ldg(r1 + kx);
                        v[6 + kx] = __ldg(r2 + kx);
                    }
                    uint32_t acc_patch = 0u;
#pragma unroll
                    for (int t = 8; t >= 0; --t) acc_patch = (acc_patch << p.Cin) | (v[t] & mask);  // Horner: tap t ends at bit t*Cin
                    patch[q] = acc_patch;
                    continue;
                }
                for (int ky = 0; ky < p.KH; ++ky) {
                    const int iy = iy0 + ky;
                    for (int kx = 0; kx < p.KW; ++kx) {
                        const int ix = ix0 + kx;
                        if (iy >= 0 && iy < p.H && ix >= 0 && ix < p.W)
                            patch[q] |= (__ldg(img + iy * p.W + ix) & mask) << ((ky * p.KW + kx) * p.Cin);
                    }
                }
            }
            for (int wd = 0; wd < p.Cow; ++wd) {
                uint32_t bits0 = 0u, bits1 = 0u;
#pragma unroll
                for (int j = 31; j >= 0; --j) {
                    // popc > t  <=>  t - popc < 0: the output bit is a sign bit, shifted in from the top
                    const uint2 wt = sPair[wd * 32 + j];
                    bits0 = __funnelshift_l(wt.y - (uint32_t)__popc(patch[0] ^ wt.x), bits0, 1);
                    bits1 = __funnelshift_l(wt.y - (uint32_t)__popc(patch[1] ^ wt.x), bits1, 1);
                }
                static_cast<uint32_t *>(p.out)[mm[0] * p.Cow + wd] = bits0;
                if (mm[1] < p.M) static_cast<uint32_t *>(p.out)[mm[1] * p.Cow + wd] = bits1;
            }
        }
        return;
    }

    for (int m = blockIdx.x * kThreads + threadIdx.x; m < p.M; m += gridDim.x * kThreads) {
        const int r = m / p.OW, ow = m - r * p.OW;
        const int n = r / p.OH, oh = r - n * p.OH;
        const int iy0 = oh * p.sh - p.pt, ix0 = ow * p.sw - p.pl;
        // gather the patch: tap t contributes its Cin bits at bit position t*Cin; taps outside the
        // image contribute zero bits (= +1.0, one-padding)
        uint32_t patch = 0u, oob = 0u;
        const uint32_t *img = p.in + (int64_t)n * p.H * p.W;
        for (int ky = 0; ky < p.KH; ++ky) {
            const int iy = iy0 + ky;
            for (int kx = 0; kx < p.KW; ++kx) {
                const int ix = ix0 + kx;
                const int t = ky * p.KW + kx;
                if (iy >= 0 && iy < p.H && ix >= 0 && ix < p.W)
                    patch |= (__ldg(img + iy * p.W + ix) & mask) << (t * p.Cin);
                else
                    oob |= 1u << t;
            }
        }
        const bool zero_fix = p.padding == LCE_PAD_SAME_ZERO && oob != 0u;
        for (int wd = 0; wd < p.Cow; ++wd) {
            uint32_t bits = 0u;
#pragma unroll 8
            for (int j = 0; j < 32; ++j) {
                const int o = wd * 32 + j;
                int32_t v = K - 2 * __popc(patch ^ sWord[o]);
                if (zero_fix) {
                    // zero-padding: the out-of-image taps counted as +1 * w; take them out again
                    for (int t = 0; t < taps; ++t)
                        if ((oob >> t) & 1u) v -= sWsum[o * taps + t];
                }
                if (p.out_type == LCE_OUT_BITPACKED) {
                    bits |= (v < sThr[o] ? 1u : 0u) << j;
                } else if (o < p.Cout) {
                    if (p.out_type == LCE_OUT_FLOAT32) {
                        const int32_t a = (p.activation == LCE_ACT_RELU && v < 0) ? 0 : v;
                        static_cast<float *>(p.out)[(int64_t)m * p.Cout + o] =
                            __fmaf_rn((float)a, __ldg(p.mult + o), __ldg(p.bias + o));
                    } else {
                        static_cast<int32_t *>(p.out)[(int64_t)m * p.Cout + o] = v;
                    }
                }
            }
            if (p.out_type == LCE_OUT_BITPACKED) static_cast<uint32_t *>(p.out)[(int64_t)m * p.Cow + wd] = bits;
        }
    }
}

}  // namespace

bool patch_covers(const ConvGeom &g)
{
    return g.Cw == 1 && g.KH * g.KW > 1 && g.KH * g.KW * g.Cin <= 32 && g.M < (1ll << 31) - 4096 && g.Cow <= 256;
}

lce_status launch_bconv_patch(const ConvGeom &g, const uint32_t *in, const uint32_t *w, const float *mult,
                              const float *bias, const int32_t *thr, void *out, cudaStream_t s)
{
    if (!patch_covers(g)) return LCE_ERR_UNSUPPORTED;
    PatchParams p{};
    p.in = in; p.w = w; p.mult = mult; p.bias = bias; p.thr = thr; p.out = out;
    p.N = g.N; p.H = g.H; p.W = g.W; p.Cin = g.Cin; p.Cout = g.Cout; p.Cow = g.Cow;
    p.KH = g.KH; p.KW = g.KW; p.sh = g.sh; p.sw = g.sw; p.OH = g.OH; p.OW = g.OW; p.pt = g.pt; p.pl = g.pl;
    p.M = (int32_t)g.M; p.padding = g.padding; p.out_type = g.out_type; p.activation = g.activation;
    const size_t smem = (size_t)g.Cow * 32 * (4 + g.KH * g.KW) * 4;
    if (smem > 48 * 1024) return LCE_ERR_UNSUPPORTED;
    // one wave of resident blocks (8 x 256 threads per SM), grid-stride beyond that: every block pays
    // for building the weight words in shared memory, so fewer, longer-lived blocks are cheaper
    int64_t blocks = (g.M + kThreads - 1) / kThreads;
    if (blocks > 148 * 8) blocks = 148 * 8;
    bconv_patch_kernel<<<(unsigned)blocks, kThreads, smem, s>>>(p);
    return launch_status();
}

}  // namespace lce
