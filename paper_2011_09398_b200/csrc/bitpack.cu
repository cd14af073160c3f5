// LceQuantize / LceDequantize (paper Section 3.2): sign-binarize and pack 32 channels per
// word, and the inverse.  Both are single-pass HBM streaming kernels.
#include "common.cuh"

namespace lce {
namespace {

constexpr int kPackThreads = 256;
constexpr int kWordsPerWarpPass = 32;  // one warp turns 32x32 floats (4 KB) into 32 words per pass

// channels % 32 == 0: the flat float array is a sequence of 32-float groups, each giving one
// word.  A warp reads group g with one coalesced 128-byte load (lane = channel within the
// group); __ballot_sync(x < 0) is the packed word (lane order = bit order, LSB = lowest
// channel).  All 32 loads of a pass are in flight before the first ballot; the 32 ballots are
// handed out four per lane to lanes 0..7, which write them with one 128-bit store each (128
// contiguous bytes per warp).  Passes are small so that even a 100K-word tensor gives every SM
// several warps of work: the kernel is latency-bound otherwise.
__global__ void __launch_bounds__(kPackThreads)
bitpack_aligned_kernel(const float *__restrict__ x, uint32_t *__restrict__ out, int64_t n_words)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * kPackThreads + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * kPackThreads) >> 5;
    for (int64_t w0 = warp * kWordsPerWarpPass; w0 < n_words; w0 += n_warps * kWordsPerWarpPass) {
        if (w0 + kWordsPerWarpPass <= n_words) {
            float v[kWordsPerWarpPass];
#pragma unroll
            for (int u = 0; u < kWordsPerWarpPass; ++u) v[u] = __ldcs(x + (w0 + u) * 32 + lane);
            uint32_t mine[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int u = 0; u < kWordsPerWarpPass; ++u) {
                const uint32_t word = __ballot_sync(0xffffffffu, v[u] < 0.0f);
                if ((u >> 2) == lane) mine[u & 3] = word;
            }
            // out + w0 is 16-byte aligned: w0 is a multiple of 32 words and out is checked on the host
            if (lane < kWordsPerWarpPass / 4)
                reinterpret_cast<uint4 *>(out + w0)[lane] = make_uint4(mine[0], mine[1], mine[2], mine[3]);
        } else {  // ragged last pass of the tensor
            for (int64_t w = w0; w < n_words; ++w) {
                const uint32_t word = __ballot_sync(0xffffffffu, x[w * 32 + lane] < 0.0f);
                if (lane == 0) out[w] = word;
            }
        }
    }
}

// Any channel count: one thread builds one output word from its (up to 32) channels.  For a
// small channel count (3-channel images: one word per pixel) neighbouring threads read
// neighbouring pixels, so the loads of a warp still cover one contiguous span.
__global__ void __launch_bounds__(kPackThreads)
bitpack_generic_kernel(const float *__restrict__ x, uint32_t *__restrict__ out, int64_t rows, int32_t channels,
                       int32_t words)
{
    const int64_t total = rows * words;
    for (int64_t i = (int64_t)blockIdx.x * kPackThreads + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * kPackThreads) {
        const int64_t r = i / words;
        const int32_t j = (int32_t)(i - r * words);
        const int32_t c0 = j * 32;
        const int32_t nc = min(32, channels - c0);
        const float *p = x + r * channels + c0;
        uint32_t word = 0u;
        for (int32_t c = 0; c < nc; ++c) word |= (p[c] < 0.0f ? 1u : 0u) << c;
        out[i] = word;  // pad bits stay 0
    }
}

// Very few channels (an RGB image: C = 3): one word per pixel.  A thread takes four consecutive
// pixels = 4*C floats = C aligned 128-bit loads, all in flight together, and writes its four words
// with one 128-bit store.  Rows past the last whole group of four go through the generic kernel.
template <int C>
__global__ void __launch_bounds__(kPackThreads)
bitpack_few_channels_kernel(const float4 *__restrict__ x, uint4 *__restrict__ out, int64_t groups)
{
    for (int64_t i = (int64_t)blockIdx.x * kPackThreads + threadIdx.x; i < groups;
         i += (int64_t)gridDim.x * kPackThreads) {
        float v[4 * C];
#pragma unroll
        for (int q = 0; q < C; ++q) {
            const float4 f = __ldcs(x + i * C + q);
            v[4 * q] = f.x; v[4 * q + 1] = f.y; v[4 * q + 2] = f.z; v[4 * q + 3] = f.w;
        }
        uint32_t w[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            w[r] = 0u;
#pragma unroll
            for (int c = 0; c < C; ++c) w[r] |= (v[r * C + c] < 0.0f ? 1u : 0u) << c;
        }
        out[i] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

template <int C>
void launch_few_channels(const float *x, uint32_t *out, int64_t groups, int max_blocks, cudaStream_t s)
{
    int64_t b = (groups + kPackThreads - 1) / kPackThreads;
    if (b > max_blocks) b = max_blocks;
    bitpack_few_channels_kernel<C><<<(unsigned)b, kPackThreads, 0, s>>>(reinterpret_cast<const float4 *>(x),
                                                                       reinterpret_cast<uint4 *>(out), groups);
}

// LceDequantize: one thread per output float.
__global__ void __launch_bounds__(kPackThreads)
unpack_kernel(const uint32_t *__restrict__ in, float *__restrict__ out, int64_t rows, int32_t channels,
              int32_t words)
{
    const int64_t total = rows * channels;
    for (int64_t i = (int64_t)blockIdx.x * kPackThreads + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * kPackThreads) {
        const int64_t r = i / channels;
        const int32_t c = (int32_t)(i - r * channels);
        const uint32_t word = in[r * words + (c >> 5)];
        out[i] = ((word >> (c & 31)) & 1u) ? -1.0f : 1.0f;
    }
}

// channels % 32 == 0 and a 16-byte aligned output: thread t writes the four floats of bits
// 4*(t%8) .. +3 of word t/8 with one 128-bit store (a warp stores 512 contiguous bytes and reads four
// words); no divisions.
__global__ void __launch_bounds__(kPackThreads)
unpack_aligned_kernel(const uint32_t *__restrict__ in, float4 *__restrict__ out, int64_t n_quads)
{
    for (int64_t t = (int64_t)blockIdx.x * kPackThreads + threadIdx.x; t < n_quads; t += (int64_t)gridDim.x * kPackThreads) {
        const uint32_t nib = (__ldg(in + (t >> 3)) >> (4 * (int)(t & 7))) & 0xFu;
        __stcs(out + t, make_float4((nib & 1u) ? -1.0f : 1.0f, (nib & 2u) ? -1.0f : 1.0f, (nib & 4u) ? -1.0f : 1.0f,
                                    (nib & 8u) ? -1.0f : 1.0f));
    }
}

int grid_for(int64_t work_items, int per_block, int max_blocks)
{
    int64_t b = (work_items + per_block - 1) / per_block;
    if (b < 1) b = 1;
    if (b > max_blocks) b = max_blocks;
    return (int)b;
}

}  // namespace
}  // namespace lce

extern "C" lce_status lce_bitpack(const float *x, uint32_t *out, int64_t rows, int32_t channels, void *stream)
{
    using namespace lce;
    if (rows < 0 || channels <= 0) return LCE_ERR_INVALID_ARG;
    if (rows == 0) return LCE_OK;
    if (!x || !out) return LCE_ERR_INVALID_ARG;
    if (!aligned(x, 4) || !aligned(out, 4)) return LCE_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int32_t words = (channels + 31) / 32;
    const int64_t n_words = rows * words;
    // up to 148 SMs x 8 resident blocks of 256 threads x 4 passes in the queue; grid-stride loops cover the rest
    const int max_blocks = 148 * 8 * 4;
    if (channels % 32 == 0 && aligned(out, 16)) {
        const int64_t passes = (n_words + kWordsPerWarpPass - 1) / kWordsPerWarpPass;
        bitpack_aligned_kernel<<<grid_for(passes, kPackThreads / 32, max_blocks), kPackThreads, 0, s>>>(x, out, n_words);
    } else if (channels <= 4 && rows >= 4 && aligned(x, 16) && aligned(out, 16)) {
        const int64_t groups = rows / 4;
        if (channels == 1) launch_few_channels<1>(x, out, groups, max_blocks * 4, s);
        else if (channels == 2) launch_few_channels<2>(x, out, groups, max_blocks * 4, s);
        else if (channels == 3) launch_few_channels<3>(x, out, groups, max_blocks * 4, s);
        else launch_few_channels<4>(x, out, groups, max_blocks * 4, s);
        const int64_t done = groups * 4;
        if (rows > done)
            bitpack_generic_kernel<<<1, kPackThreads, 0, s>>>(x + done * channels, out + done, rows - done, channels, 1);
    } else {
        bitpack_generic_kernel<<<grid_for(n_words, kPackThreads, max_blocks * 4), kPackThreads, 0, s>>>(
            x, out, rows, channels, words);
    }
    return launch_status();
}

extern "C" lce_status lce_unpack(const uint32_t *in, float *out, int64_t rows, int32_t channels, void *stream)
{
    using namespace lce;
    if (rows < 0 || channels <= 0) return LCE_ERR_INVALID_ARG;
    if (rows == 0) return LCE_OK;
    if (!in || !out) return LCE_ERR_INVALID_ARG;
    if (!aligned(in, 4) || !aligned(out, 4)) return LCE_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int32_t words = (channels + 31) / 32;
    if (channels % 32 == 0 && aligned(out, 16)) {
        const int64_t n_quads = rows * channels / 4;
        unpack_aligned_kernel<<<grid_for(n_quads, kPackThreads, 148 * 32), kPackThreads, 0, s>>>(in, reinterpret_cast<float4 *>(out), n_quads);
    } else {
        unpack_kernel<<<grid_for(rows * channels, kPackThreads, 148 * 32), kPackThreads, 0, s>>>(in, out, rows, channels, words);
    }
    return launch_status();
}
