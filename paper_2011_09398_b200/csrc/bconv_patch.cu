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
    const size_t smem = (size_t)g.Cow * 32 * (2 + g.KH * g.KW) * 4;
    if (smem > 48 * 1024) return LCE_ERR_UNSUPPORTED;
    int64_t blocks = (g.M + kThreads - 1) / kThreads;
    if (blocks > 148 * 8 * 8) blocks = 148 * 8 * 8;  // grid-stride beyond 8 waves of 8 blocks per SM
    bconv_patch_kernel<<<(unsigned)blocks, kThreads, smem, s>>>(p);
    return launch_status();
}

}  // namespace lce
