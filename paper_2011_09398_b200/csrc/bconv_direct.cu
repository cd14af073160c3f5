// LceBConv2d, direct form: one thread per output value walks the taps and the packed channel
// words straight from global memory.  It covers every shape, stride, padding mode and output
// type and is the fallback for shapes the tiled kernel does not take; it is not fast.
//   acc = K_eff - 2 * sum popcount(a XOR w)            (paper Section 2 and Section 3.2)
// where out-of-image taps read a zero word (+1, one-padding) or, for zero-padding, are left
// out of both the sum and K_eff.
#include "common.cuh"

namespace lce {
namespace {

constexpr int kThreads = 256;

template <int OUT_TYPE>
__global__ void __launch_bounds__(kThreads)
bconv_direct_kernel(ConvGeom g, const uint32_t *__restrict__ in, const uint32_t *__restrict__ wts,
                    const float *__restrict__ mult, const float *__restrict__ bias,
                    const int32_t *__restrict__ thr, void *__restrict__ out)
{
    const int32_t Cpad = g.Cow * 32;  // lanes of a warp = 32 consecutive output channels of one pixel
    const int64_t total = g.M * Cpad;
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kThreads) {
        const int32_t o = (int32_t)(i % Cpad);
        int64_t p = i / Cpad;  // flat output pixel
        const int64_t pix = p;
        const int32_t ow = (int32_t)(p % g.OW);
        p /= g.OW;
        const int32_t oh = (int32_t)(p % g.OH);
        const int32_t n = (int32_t)(p / g.OH);
        int32_t acc = 0;
        if (o < g.Cout) {
            int32_t cnt = 0, taps_in = 0;
            for (int32_t ky = 0; ky < g.KH; ++ky) {
                const int32_t iy = oh * g.sh - g.pt + ky;
                for (int32_t kx = 0; kx < g.KW; ++kx) {
                    const int32_t ix = ow * g.sw - g.pl + kx;
                    const bool inside = iy >= 0 && iy < g.H && ix >= 0 && ix < g.W;
                    const uint32_t *wp = wts + (((int64_t)o * g.KH + ky) * g.KW + kx) * g.Cw;
                    if (inside) {
                        const uint32_t *ap = in + (((int64_t)n * g.H + iy) * g.W + ix) * g.Cw;
                        for (int32_t j = 0; j < g.Cw; ++j) cnt += __popc(__ldg(ap + j) ^ __ldg(wp + j));
                        ++taps_in;
                    } else if (g.padding == LCE_PAD_SAME_ONE) {
                        for (int32_t j = 0; j < g.Cw; ++j) cnt += __popc(__ldg(wp + j));  // a = zero word
                        ++taps_in;
                    }
                }
            }
            acc = taps_in * g.Cin - 2 * cnt;
        }
        if (OUT_TYPE == LCE_OUT_INT32) {
            if (o < g.Cout) static_cast<int32_t *>(out)[pix * g.Cout + o] = acc;
        } else if (OUT_TYPE == LCE_OUT_FLOAT32) {
            if (o < g.Cout) {
                const int32_t v = (g.activation == LCE_ACT_RELU && acc < 0) ? 0 : acc;
                static_cast<float *>(out)[pix * g.Cout + o] = __fmaf_rn((float)v, __ldg(mult + o), __ldg(bias + o));
            }
        } else {
            const bool bit = (o < g.Cout) && (acc < __ldg(thr + (o < g.Cout ? o : 0)));
            const uint32_t word = __ballot_sync(0xffffffffu, bit);
            if ((threadIdx.x & 31) == 0) static_cast<uint32_t *>(out)[pix * g.Cow + (o >> 5)] = word;
        }
    }
}

}  // namespace

lce_status launch_bconv_direct(const ConvGeom &g, const uint32_t *in, const uint32_t *w, const float *mult,
                               const float *bias, const int32_t *thr, void *out, cudaStream_t s)
{
    const int64_t total = g.M * g.Cow * 32;
    int64_t blocks = (total + kThreads - 1) / kThreads;
    if (blocks > 148 * 64) blocks = 148 * 64;
    // total is a multiple of 32 and so is the grid stride, so whole warps enter and leave the
    // loop together: the ballot of the bit-packed epilogue always has all 32 lanes present.
    if (g.out_type == LCE_OUT_INT32)
        bconv_direct_kernel<LCE_OUT_INT32><<<(int)blocks, kThreads, 0, s>>>(g, in, w, mult, bias, thr, out);
    else if (g.out_type == LCE_OUT_FLOAT32)
        bconv_direct_kernel<LCE_OUT_FLOAT32><<<(int)blocks, kThreads, 0, s>>>(g, in, w, mult, bias, thr, out);
    else
        bconv_direct_kernel<LCE_OUT_BITPACKED><<<(int)blocks, kThreads, 0, s>>>(g, in, w, mult, bias, thr, out);
    return launch_status();
}

}  // namespace lce
