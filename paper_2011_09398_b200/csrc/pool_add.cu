// LceBMaxPool2d (paper Section 3.2: max-pool on packed bits is the bitwise AND of the window,
// because a 0 bit is +1 and max(sign X) = sign(max X)) and the fp32 residual add that the
// shortcut pattern of Section 5.3 places between a float-output conv and the next LceQuantize.
#include "common.cuh"

namespace lce {
namespace {

constexpr int kThreads = 256;

// A block walks output rows (n, oh); its threads walk the row's words, VEC words at a time (VEC = 4:
// 128-bit loads and stores, when the word count per pixel allows), so that the only division left
// per output is a 32-bit one by the words per pixel.  Out-of-image taps are skipped (AND identity
// = all ones); channel-pad bits stay 0 because they are 0 in every input word.
template <int VEC>
__global__ void __launch_bounds__(kThreads)
bmaxpool_kernel(const uint32_t *__restrict__ in, uint32_t *__restrict__ out, int32_t N, int32_t H, int32_t W,
                int32_t Cw, int32_t OH, int32_t OW, int32_t PH, int32_t PW, int32_t sh, int32_t sw, int32_t pt,
                int32_t pl)
{
    const int32_t cv = Cw / VEC;            // vectors per pixel
    const int32_t row_vecs = OW * cv;       // vectors per output row
    const int32_t rows = N * OH;  // < 2^31: checked on the host
    for (int32_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const int32_t n = row / OH, oh = row - n * OH;
        const int32_t iy0 = oh * sh - pt;
        const uint32_t *img = in + (int64_t)n * H * W * Cw;
        uint32_t *orow = out + (int64_t)row * OW * Cw;
        for (int32_t e = threadIdx.x; e < row_vecs; e += kThreads) {
            const int32_t ow = e / cv, j = (e - ow * cv) * VEC;
            const int32_t ix0 = ow * sw - pl;
            uint32_t acc[VEC];
            if (PH == 2 && PW == 2 && iy0 >= 0 && iy0 + 1 < H && ix0 >= 0 && ix0 + 1 < W) {
                // the usual 2x2 window, inside the image: four independent loads in flight, three ANDs
                const uint32_t *s0 = img + ((int64_t)iy0 * W + ix0) * Cw + j, *s1 = s0 + (int64_t)W * Cw;
                if (VEC == 4) {
                    const uint4 a = __ldcs(reinterpret_cast<const uint4 *>(s0)), b = __ldcs(reinterpret_cast<const uint4 *>(s0 + Cw));
                    const uint4 c = __ldcs(reinterpret_cast<const uint4 *>(s1)), d = __ldcs(reinterpret_cast<const uint4 *>(s1 + Cw));
                    __stcs(reinterpret_cast<uint4 *>(orow + (int64_t)ow * Cw + j),
                           make_uint4(a.x & b.x & c.x & d.x, a.y & b.y & c.y & d.y, a.z & b.z & c.z & d.z, a.w & b.w & c.w & d.w));
                } else {
                    orow[(int64_t)ow * Cw + j] = __ldcs(s0) & __ldcs(s0 + Cw) & __ldcs(s1) & __ldcs(s1 + Cw);
                }
                continue;
            }
#pragma unroll
            for (int v = 0; v < VEC; ++v) acc[v] = 0xffffffffu;
            for (int32_t ky = 0; ky < PH; ++ky) {
                const int32_t iy = iy0 + ky;
                if (iy < 0 || iy >= H) continue;
                for (int32_t kx = 0; kx < PW; ++kx) {
                    const int32_t ix = ix0 + kx;
                    if (ix < 0 || ix >= W) continue;
                    const uint32_t *src = img + ((int64_t)iy * W + ix) * Cw + j;
                    if (VEC == 4) {
                        const uint4 q = __ldg(reinterpret_cast<const uint4 *>(src));
                        acc[0] &= q.x; acc[1] &= q.y; acc[2] &= q.z; acc[3] &= q.w;
                    } else {
                        acc[0] &= __ldg(src);
                    }
                }
            }
            if (VEC == 4) *reinterpret_cast<uint4 *>(orow + (int64_t)ow * Cw + j) = make_uint4(acc[0], acc[1], acc[2], acc[3]);
            else orow[(int64_t)ow * Cw + j] = acc[0];
        }
    }
}

__global__ void __launch_bounds__(kThreads)
add_f32_vec4_kernel(const float4 *a, const float4 *b, float4 *out, int64_t n4)
{
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n4; i += (int64_t)gridDim.x * kThreads) {
        const float4 u = __ldcs(a + i), v = __ldcs(b + i);
        out[i] = make_float4(__fadd_rn(u.x, v.x), __fadd_rn(u.y, v.y), __fadd_rn(u.z, v.z), __fadd_rn(u.w, v.w));
    }
}

__global__ void __launch_bounds__(kThreads)
add_f32_scalar_kernel(const float *a, const float *b, float *out, int64_t begin, int64_t n)
{
    for (int64_t i = begin + (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kThreads)
        out[i] = __fadd_rn(a[i], b[i]);
}

int grid_for(int64_t items, int max_blocks)
{
    int64_t b = (items + kThreads - 1) / kThreads;
    if (b < 1) b = 1;
    if (b > max_blocks) b = max_blocks;
    return (int)b;
}

}  // namespace
}  // namespace lce

extern "C" lce_status lce_bmaxpool(const uint32_t *in, uint32_t *out, int32_t batch, int32_t in_h, int32_t in_w,
                                   int32_t channels, int32_t pool_h, int32_t pool_w, int32_t stride_h,
                                   int32_t stride_w, int32_t padding, void *stream)
{
    using namespace lce;
    if (!in || !out) return LCE_ERR_INVALID_ARG;
    if (batch <= 0 || in_h <= 0 || in_w <= 0 || channels <= 0 || pool_h <= 0 || pool_w <= 0 || stride_h <= 0 ||
        stride_w <= 0)
        return LCE_ERR_INVALID_ARG;
    if (padding != LCE_PAD_VALID && padding != LCE_PAD_SAME_ONE) return LCE_ERR_INVALID_ARG;
    if (!aligned(in, 4) || !aligned(out, 4)) return LCE_ERR_ALIGNMENT;
    const Axis ah = axis_geometry(in_h, pool_h, stride_h, padding);
    const Axis aw = axis_geometry(in_w, pool_w, stride_w, padding);
    if (ah.out <= 0 || aw.out <= 0) return LCE_ERR_INVALID_ARG;
    const int32_t Cw = (channels + 31) / 32;
    const int64_t total = (int64_t)batch * ah.out * aw.out * Cw;
    (void)total;
    if ((int64_t)batch * ah.out >= (1ll << 31)) return LCE_ERR_UNSUPPORTED;
    int64_t blocks = (int64_t)batch * ah.out;  // one block per output row, grid-stride beyond 8 waves of 8 blocks per SM
    if (blocks > 148 * 8 * 8) blocks = 148 * 8 * 8;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (Cw % 4 == 0 && aligned(in, 16) && aligned(out, 16))
        bmaxpool_kernel<4><<<(unsigned)blocks, kThreads, 0, s>>>(in, out, batch, in_h, in_w, Cw, ah.out, aw.out, pool_h, pool_w,
                                                                stride_h, stride_w, ah.pad_before, aw.pad_before);
    else
        bmaxpool_kernel<1><<<(unsigned)blocks, kThreads, 0, s>>>(in, out, batch, in_h, in_w, Cw, ah.out, aw.out, pool_h, pool_w,
                                                                stride_h, stride_w, ah.pad_before, aw.pad_before);
    return launch_status();
}

extern "C" lce_status lce_add_f32(const float *a, const float *b, float *out, int64_t n, void *stream)
{
    using namespace lce;
    if (n < 0) return LCE_ERR_INVALID_ARG;
    if (n == 0) return LCE_OK;
    if (!a || !b || !out) return LCE_ERR_INVALID_ARG;
    if (!aligned(a, 4) || !aligned(b, 4) || !aligned(out, 4)) return LCE_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int64_t done = 0;
    if (aligned(a, 16) && aligned(b, 16) && aligned(out, 16) && n >= 4) {
        const int64_t n4 = n / 4;
        add_f32_vec4_kernel<<<grid_for(n4, 148 * 8), kThreads, 0, s>>>(
            reinterpret_cast<const float4 *>(a), reinterpret_cast<const float4 *>(b), reinterpret_cast<float4 *>(out), n4);
        done = n4 * 4;
    }
    if (done < n) add_f32_scalar_kernel<<<grid_for(n - done, 148 * 8), kThreads, 0, s>>>(a, b, out, done, n);
    return launch_status();
}
