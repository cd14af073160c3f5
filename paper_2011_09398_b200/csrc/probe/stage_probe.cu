// Staging probe: how fast can a CTA bring tiles of bit-packed activations [n][y][x][cw] into shared memory?
// Three ways of doing the same copy are timed with no arithmetic behind them, on the geometry of the integer
// convolution kernel (256 threads per CTA, two CTAs per SM, a tile = a few image rows plus two halo rows,
// two buffers that alternate):
//   mode 0  one 4-byte asynchronous copy per packed word into word planes [cw][row][x]   (the layout the
//           XOR/POPC kernel computes from: a lane reads neighbouring pixels of one channel word)
//   mode 1  one 16-byte asynchronous copy per four words into [row][x][cw]
//   mode 2  one tensor-map bulk copy (cp.async.bulk.tensor, this GPU's memory, no multicast) per tile into
//           [row][x][cw]; rows outside the tensor arrive as zero words
// The tensor-map copy cannot write word planes: its innermost box extent must be 16 bytes or more of
// contiguous global memory, and the contiguous direction of the input is the channel words.
#include <cuda.h>

#include <cstring>

#include "common.cuh"
#include "lce_probe.h"
#include "mx_common.cuh"

namespace lce {
namespace {

constexpr int kStageThreads = 256;

struct StageParams {
    const uint32_t *in;
    uint32_t *sink;
    unsigned long long *first_ns;  // per CTA: kernel entry -> first tile landed
    int *error;
    int rows_total, W, Cw, rows_per_tile, n_tiles, buf_words, passes;
};

__device__ __forceinline__ void cp_async_4(uint32_t *dst, const uint32_t *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_16(uint32_t *dst, const uint32_t *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}

// rows y0 - 1 .. y0 + rows_per_tile of the flattened [n * H + y] rows (one halo row on each side)
template <int MODE>
__device__ __forceinline__ void stage_tile(const StageParams &p, const CUtensorMap *map, int tile, uint32_t *buf, uint64_t *bar, int tid)
{
    const int y0 = tile * p.rows_per_tile - 1, nrows = p.rows_per_tile + 2;
    const int row_words = p.W * p.Cw;
    if (MODE == 0) {
        const int plane = nrows * p.W;
        const int cw_shift = 31 - __clz(p.Cw);  // Cw is a power of two here
        for (int r = tid >> 5; r < nrows; r += kStageThreads / 32) {
            const int y = y0 + r;
            if (y < 0 || y >= p.rows_total) {
                for (int e = tid & 31; e < row_words; e += 32) buf[(e & (p.Cw - 1)) * plane + r * p.W + (e >> cw_shift)] = 0u;
                continue;
            }
            const uint32_t *src = p.in + (size_t)y * row_words;
            for (int e = tid & 31; e < row_words; e += 32) cp_async_4(buf + (e & (p.Cw - 1)) * plane + r * p.W + (e >> cw_shift), src + e);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    } else if (MODE == 1) {
        const int quads = row_words >> 2;
        for (int r = tid >> 5; r < nrows; r += kStageThreads / 32) {
            const int y = y0 + r;
            uint32_t *dst = buf + r * row_words;
            if (y < 0 || y >= p.rows_total) {
                for (int e = tid & 31; e < quads; e += 32) *reinterpret_cast<uint4 *>(dst + 4 * e) = make_uint4(0u, 0u, 0u, 0u);
                continue;
            }
            const uint32_t *src = p.in + (size_t)y * row_words;
            for (int e = tid & 31; e < quads; e += 32) cp_async_16(dst + 4 * e, src + 4 * e);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    } else {
        if (tid == 0) {
            mbar_expect_tx(bar, (uint32_t)(nrows * row_words * 4));
            asm volatile(
                "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
                    smem_u32(buf)),
                "l"(map), "r"(0), "r"(0), "r"(y0), "r"(smem_u32(bar))
                : "memory");
        }
    }
}

template <int MODE>
__global__ void __launch_bounds__(kStageThreads, 2) stage_probe_kernel(const StageParams p, const __grid_constant__ CUtensorMap map)
{
    extern __shared__ __align__(128) uint32_t stage_smem[];
    __shared__ __align__(8) uint64_t bars[2];
    const unsigned long long t_in = globaltimer_ns();
    const int tid = threadIdx.x;
    if (MODE == 2 && tid == 0) {
        mbar_init(&bars[0], 1);
        mbar_init(&bars[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t acc = 0u;
    uint32_t parity[2] = {0u, 0u};
    bool ok = true;
    for (int pass = 0; pass < p.passes && ok; ++pass) {
        int tile = blockIdx.x, it = 0;
        if (tile < p.n_tiles) stage_tile<MODE>(p, &map, tile, stage_smem, &bars[0], tid);
        for (; tile < p.n_tiles; tile += gridDim.x, ++it) {
            const int b = it & 1;
            uint32_t *buf = stage_smem + b * p.buf_words;
            // the tile has landed
            if (MODE == 2) {
                ok = mbar_wait_bounded(&bars[b], parity[b]);
                parity[b] ^= 1u;
                if (!ok) break;
            } else {
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                __syncthreads();
            }
            if (pass == 0 && it == 0 && tid == 0) p.first_ns[blockIdx.x] = globaltimer_ns() - t_in;
            // the next tile goes into the other buffer (everybody is done reading it: the barrier below, one
            // iteration ago)
            const int next = tile + gridDim.x;
            if (next < p.n_tiles) stage_tile<MODE>(p, &map, next, stage_smem + (b ^ 1) * p.buf_words, &bars[b ^ 1], tid);
            // a token read of the tile, so that the copies cannot be dropped
            for (int e = tid; e < p.buf_words; e += 8 * kStageThreads) acc ^= buf[e];
            __syncthreads();
        }
    }
    if (!ok) atomicExch(p.error, 1);
    if (acc == 0x12345678u) p.sink[blockIdx.x] = acc;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace
}  // namespace lce

extern "C" lce_status lce_probe_stage(int32_t mode, int32_t batch, int32_t in_h, int32_t in_w, int32_t in_words,
                                      int32_t rows_per_tile, int32_t passes, double *us_per_pass, double *first_tile_us,
                                      void *stream)
{
    using namespace lce;
    if (!us_per_pass || !first_tile_us || mode < 0 || mode > 2 || batch <= 0 || in_h <= 0 || in_w <= 0 || rows_per_tile <= 0 ||
        passes <= 0)
        return LCE_ERR_INVALID_ARG;
    if (in_words < 1 || in_words > 32 || (in_words & (in_words - 1)) != 0) return LCE_ERR_INVALID_ARG;
    if (mode != 0 && in_words < 4) return LCE_ERR_UNSUPPORTED;  // 16 bytes of contiguous words per pixel
    if (in_w > 256 || rows_per_tile + 2 > 256) return LCE_ERR_UNSUPPORTED;  // box extents of a tensor map
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LCE_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return LCE_ERR_CUDA;

    StageParams p{};
    p.rows_total = batch * in_h;
    p.W = in_w;
    p.Cw = in_words;
    p.rows_per_tile = rows_per_tile;
    p.n_tiles = (p.rows_total + rows_per_tile - 1) / rows_per_tile;
    p.buf_words = (((rows_per_tile + 2) * in_w * in_words + 31) / 32) * 32;  // 128-byte multiple
    p.passes = passes;
    const size_t smem = (size_t)2 * p.buf_words * 4;
    if (smem > 96 * 1024) return LCE_ERR_UNSUPPORTED;
    const int grid = p.n_tiles < 2 * sms ? p.n_tiles : 2 * sms;
    const size_t in_bytes = (size_t)p.rows_total * in_w * in_words * 4;

    uint32_t *in = nullptr, *sink = nullptr;
    unsigned long long *first = nullptr, *host_first = nullptr;
    int *error = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    lce_status st = LCE_ERR_CUDA;
    do {
        if (cudaMalloc(&in, in_bytes) != cudaSuccess || cudaMalloc(&sink, (size_t)grid * 4) != cudaSuccess ||
            cudaMalloc(&first, (size_t)grid * 8) != cudaSuccess || cudaMalloc(&error, 4) != cudaSuccess)
            break;
        if (cudaMemsetAsync(in, 0x5A, in_bytes, s) != cudaSuccess || cudaMemsetAsync(error, 0, 4, s) != cudaSuccess) break;
        p.in = in; p.sink = sink; p.first_ns = first; p.error = error;
        CUtensorMap map;
        memset(&map, 0, sizeof(map));
        if (mode == 2) {
            void *fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
                qres != cudaDriverEntryPointSuccess)
                break;
            const cuuint64_t dims[3] = {(cuuint64_t)in_words, (cuuint64_t)in_w, (cuuint64_t)p.rows_total};
            const cuuint64_t strides[2] = {(cuuint64_t)in_words * 4, (cuuint64_t)in_w * in_words * 4};
            const cuuint32_t box[3] = {(cuuint32_t)in_words, (cuuint32_t)in_w, (cuuint32_t)(rows_per_tile + 2)};
            const cuuint32_t elem[3] = {1, 1, 1};
            if (reinterpret_cast<EncodeTiledFn>(fn)(&map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, in, dims, strides, box, elem,
                                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                                    CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                break;
        }
        auto kernel = mode == 0 ? stage_probe_kernel<0> : mode == 1 ? stage_probe_kernel<1> : stage_probe_kernel<2>;
        if (smem > 48 * 1024 && cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) break;
        if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) break;
        for (int rep = 0; rep < 2; ++rep) {  // first repetition warms up
            if (rep == 1) cudaEventRecord(e0, s);
            kernel<<<grid, kStageThreads, smem, s>>>(p, map);
        }
        cudaEventRecord(e1, s);
        if (cudaEventSynchronize(e1) != cudaSuccess || cudaGetLastError() != cudaSuccess) break;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) break;
        int host_error = 0;
        host_first = new unsigned long long[grid];
        if (cudaMemcpy(&host_error, error, 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
            cudaMemcpy(host_first, first, (size_t)grid * 8, cudaMemcpyDeviceToHost) != cudaSuccess)
            break;
        if (host_error) { st = LCE_ERR_DEVICE_TIMEOUT; break; }
        // median over the CTAs of the time from kernel entry to the first tile in shared memory
        for (int i = 1; i < grid; ++i) {
            unsigned long long v = host_first[i];
            int j = i - 1;
            while (j >= 0 && host_first[j] > v) { host_first[j + 1] = host_first[j]; --j; }
            host_first[j + 1] = v;
        }
        *first_tile_us = (double)host_first[grid / 2] * 1e-3;
        *us_per_pass = (double)ms * 1e3 / passes;
        st = LCE_OK;
    } while (0);
    delete[] host_first;
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(in); cudaFree(sink); cudaFree(first); cudaFree(error);
    return st;
}
