// Integer-pipe probes: register-resident loops of the candidate instruction mixes of the binary
// GEMM inner loop (paper Section 3.2 and its Table 1 count instructions per binary MAC on a
// Cortex-A76; this is the same exercise on an SM).  The rates measured here are the compute
// ceilings the convolution kernel is judged against.
#include "common.cuh"
#include "csa.cuh"
#include "lce_probe.h"

namespace lce {
namespace {

constexpr int kThreads = 256;
constexpr int PX = 2;   // pixels per thread in the mix probes
constexpr int CH = 8;   // output channels per thread

template <int MIX>
__global__ void __launch_bounds__(kThreads)
probe_mix_kernel(const uint32_t *__restrict__ seed, uint32_t *__restrict__ sink, long long *__restrict__ cycles,
                 int iterations)
{
    // multipliers of the weighted popcount sum, opaque to the compiler (iterations > 0 always)
    Weights124 k124;
    k124.one = iterations > 0 ? 1u : seed[0];
    k124.two = iterations > 0 ? 2u : seed[1];
    k124.four = iterations > 0 ? 4u : seed[2];
    asm volatile("" : "+r"(k124.one), "+r"(k124.two), "+r"(k124.four));
    // Activation words come from shared memory every iteration, as in the convolution kernel
    // (per pixel nine LDS feed 8 x 9 word operations); weight-side operands stay in registers.
    __shared__ uint32_t tile[1024 + 64];
    for (int i = threadIdx.x; i < 1024 + 64; i += kThreads) tile[i] = seed[i & 1023];
    uint32_t w[CH][9];
    uint32_t acc[PX][CH];
#pragma unroll
    for (int j = 0; j < CH; ++j)
#pragma unroll
        for (int t = 0; t < 9; ++t) w[j][t] = seed[(threadIdx.x * 17 + j * 9 + t + 512) & 1023];
#pragma unroll
    for (int p = 0; p < PX; ++p)
#pragma unroll
        for (int j = 0; j < CH; ++j) acc[p][j] = 0;
    Triple wt[CH][3];
#pragma unroll
    for (int j = 0; j < CH; ++j)
#pragma unroll
        for (int g = 0; g < 3; ++g) wt[j][g] = make_triple(w[j][3 * g], w[j][3 * g + 1], w[j][3 * g + 2]);

    __syncthreads();
    const int base = (threadIdx.x >> 3) * 2;  // lanes that share a pixel read the same words (broadcast)
    const long long t0 = clock64();
    for (int it = 0; it < iterations; ++it) {
        const uint32_t *row = tile + ((base + it * 11) & 1023);
#pragma unroll
        for (int p = 0; p < PX; ++p) {
            uint32_t a[9];
#pragma unroll
            for (int t = 0; t < 9; ++t) a[t] = row[p * 9 + t];
            if (MIX == 0) {
#pragma unroll
                for (int j = 0; j < CH; ++j)
#pragma unroll
                    for (int t = 0; t < 9; ++t) acc[p][j] += __popc(a[t] ^ w[j][t]);
            } else {
                Triple at[3];
#pragma unroll
                for (int g = 0; g < 3; ++g) at[g] = make_triple(a[3 * g], a[3 * g + 1], a[3 * g + 2]);
#pragma unroll
                for (int j = 0; j < CH; ++j) {
                    if (MIX == 1) {
#pragma unroll
                        for (int g = 0; g < 3; ++g) acc[p][j] += popc3(at[g], wt[j][g]);
                    } else if (MIX == 2) {
                        acc[p][j] += popc9(at, wt[j]);
                    } else {
                        popc9_mad(at, wt[j], k124, acc[p][j]);
                    }
                }
            }
        }
    }
    const long long t1 = clock64();
    uint32_t x = 0;
#pragma unroll
    for (int p = 0; p < PX; ++p)
#pragma unroll
        for (int j = 0; j < CH; ++j) x ^= acc[p][j];
    sink[(size_t)blockIdx.x * kThreads + threadIdx.x] = x;
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

// Single-instruction chains, 16 independent values per thread, each new value depending on
// three different old ones so that consecutive operations cannot be merged.
template <int KIND>
__global__ void __launch_bounds__(kThreads)
probe_unit_kernel(const uint32_t *__restrict__ seed, uint32_t *__restrict__ sink, long long *__restrict__ cycles,
                  int iterations)
{
    uint32_t v[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = seed[(threadIdx.x + i * 37) & 1023];
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iterations; ++it) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const uint32_t b = v[(i + 5) & 15], c = v[(i + 11) & 15];
                if (KIND == 10) v[i] = lop3<0x3A>(v[i], b, c);
                if (KIND == 11) v[i] = __popc(v[i]);
                if (KIND == 12) asm volatile("add.u32 %0, %0, %1;\n\tadd.u32 %0, %0, %2;" : "+r"(v[i]) : "r"(b), "r"(c));
                if (KIND == 13) asm volatile("mad.lo.u32 %0, %1, %2, %0;" : "+r"(v[i]) : "r"(b), "r"(c));
                if (KIND == 14) {  // alternate logic and multiply-add: do the two pipes overlap?
                    if (i & 1) asm volatile("mad.lo.u32 %0, %1, %2, %0;" : "+r"(v[i]) : "r"(b), "r"(c));
                    else v[i] = lop3<0x3A>(v[i], b, c);
                }
                if (KIND == 15) {  // logic, multiply-add and popcount interleaved 4:1:1
                    if ((i & 7) == 3) v[i] = __popc(v[i]) + b;
                    else if ((i & 7) == 7) asm volatile("mad.lo.u32 %0, %1, %2, %0;" : "+r"(v[i]) : "r"(b), "r"(c));
                    else v[i] = lop3<0x3A>(v[i], b, c);
                }
            }
        }
    }
    const long long t1 = clock64();
    uint32_t x = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) x ^= v[i];
    sink[(size_t)blockIdx.x * kThreads + threadIdx.x] = x;
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

// Legacy warp-level 1-bit MMA: m16n8k256, s32 accumulate, XOR+POPC or AND+POPC.
template <bool USE_AND>
__global__ void __launch_bounds__(kThreads)
probe_mma_b1_kernel(const uint32_t *__restrict__ seed, uint32_t *__restrict__ sink, long long *__restrict__ cycles,
                    int iterations)
{
    uint32_t a[4], b[2];
    int32_t d[8][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) a[i] = seed[(threadIdx.x * 4 + i) & 1023];
#pragma unroll
    for (int i = 0; i < 2; ++i) b[i] = seed[(threadIdx.x * 2 + i + 300) & 1023];
#pragma unroll
    for (int t = 0; t < 8; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) d[t][i] = 0;
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iterations; ++it) {
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            if (USE_AND)
                asm volatile(
                    "mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                    "{%0,%1,%2,%3};"
                    : "+r"(d[t][0]), "+r"(d[t][1]), "+r"(d[t][2]), "+r"(d[t][3])
                    : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
            else
                asm volatile(
                    "mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.xor.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                    "{%0,%1,%2,%3};"
                    : "+r"(d[t][0]), "+r"(d[t][1]), "+r"(d[t][2]), "+r"(d[t][3])
                    : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        }
    }
    const long long t1 = clock64();
    uint32_t x = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) x ^= (uint32_t)d[t][i];
    sink[(size_t)blockIdx.x * kThreads + threadIdx.x] = x;
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

// Do the integer pipes and the legacy 1-bit warp MMA run side by side?  Even warps run the
// nine-word carry-save loop (mix 3), odd warps the AND+POPC MMA loop (mix 21), in the same CTA at
// the same time; each group times itself.  cycles[2*block] = logic group, [2*block+1] = MMA group.
template <int MODE>  // 0: both groups, 1: the logic group alone (odd warps idle), 2: the MMA group alone
__global__ void __launch_bounds__(kThreads, 2)
probe_combined_kernel(const uint32_t *__restrict__ seed, uint32_t *__restrict__ sink, long long *__restrict__ cycles,
                      int iterations)
{
    __shared__ __align__(16) uint32_t tile[1024 + 64];
    for (int i = threadIdx.x; i < 1024 + 64; i += kThreads) tile[i] = seed[i & 1023];
    __syncthreads();
    const int warp = threadIdx.x >> 5;
    uint32_t x = 0;
    if ((warp & 1) == 0 && MODE != 2) {
        // as in the convolution kernel: 4 pixels x 8 channels per thread, activation operands in
        // registers, each channel's weight operands read from shared memory once per group
        constexpr int TPX = 4;
        Weights124 k124;
        k124.one = iterations > 0 ? 1u : seed[0];
        k124.two = iterations > 0 ? 2u : seed[1];
        k124.four = iterations > 0 ? 4u : seed[2];
        asm volatile("" : "+r"(k124.one), "+r"(k124.two), "+r"(k124.four));
        uint32_t acc[TPX][CH];
#pragma unroll
        for (int p = 0; p < TPX; ++p)
#pragma unroll
            for (int j = 0; j < CH; ++j) acc[p][j] = 0;
        const int base = (threadIdx.x >> 3) * 2;
        const uint32_t *wrow = tile + (threadIdx.x & 7) * 100;  // 8 channels x 12 words, as the kernel's layout
        const int its = iterations * 115 / 100;  // 288 word operations per iteration against the MMA group's 256 pairs
        const long long t0 = clock64();
        for (int it = 0; it < its; ++it) {
            const uint32_t *row = tile + ((base + it * 11) & 1023);
            Triple at[TPX][3];
#pragma unroll
            for (int p = 0; p < TPX; ++p)
#pragma unroll
                for (int g = 0; g < 3; ++g) at[p][g] = make_triple(row[p * 9 + 3 * g], row[p * 9 + 3 * g + 1], row[p * 9 + 3 * g + 2]);
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                const uint4 q0 = *reinterpret_cast<const uint4 *>(wrow + j * 12);
                const uint4 q1 = *reinterpret_cast<const uint4 *>(wrow + j * 12 + 4);
                const uint32_t q2 = wrow[j * 12 + 8];
                Triple wt[3];
                wt[0].all = q0.x; wt[0].pair = q0.y; wt[0].first = q0.z;
                wt[1].all = q0.w; wt[1].pair = q1.x; wt[1].first = q1.y;
                wt[2].all = q1.z; wt[2].pair = q1.w; wt[2].first = q2;
                if (j == 0) popc9_mad_pixels<TPX, CH, 0>(at, wt, k124, acc);
                if (j == 1) popc9_mad_pixels<TPX, CH, 1>(at, wt, k124, acc);
                if (j == 2) popc9_mad_pixels<TPX, CH, 2>(at, wt, k124, acc);
                if (j == 3) popc9_mad_pixels<TPX, CH, 3>(at, wt, k124, acc);
                if (j == 4) popc9_mad_pixels<TPX, CH, 4>(at, wt, k124, acc);
                if (j == 5) popc9_mad_pixels<TPX, CH, 5>(at, wt, k124, acc);
                if (j == 6) popc9_mad_pixels<TPX, CH, 6>(at, wt, k124, acc);
                if (j == 7) popc9_mad_pixels<TPX, CH, 7>(at, wt, k124, acc);
            }
        }
        const long long t1 = clock64();
#pragma unroll
        for (int p = 0; p < TPX; ++p)
#pragma unroll
            for (int j = 0; j < CH; ++j) x ^= acc[p][j];
        if (threadIdx.x == 0) cycles[2 * blockIdx.x] = t1 - t0;
    } else if ((warp & 1) == 1 && MODE != 1) {
        uint32_t a[4], b[2];
        int32_t d[8][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = seed[(threadIdx.x * 4 + i) & 1023];
#pragma unroll
        for (int i = 0; i < 2; ++i) b[i] = seed[(threadIdx.x * 2 + i + 300) & 1023];
#pragma unroll
        for (int t = 0; t < 8; ++t)
#pragma unroll
            for (int i = 0; i < 4; ++i) d[t][i] = 0;
        const long long t0 = clock64();
        for (int it = 0; it < iterations; ++it) {
#pragma unroll
            for (int t = 0; t < 8; ++t)
                asm volatile(
                    "mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                    "{%0,%1,%2,%3};"
                    : "+r"(d[t][0]), "+r"(d[t][1]), "+r"(d[t][2]), "+r"(d[t][3])
                    : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        }
        const long long t1 = clock64();
#pragma unroll
        for (int t = 0; t < 8; ++t)
#pragma unroll
            for (int i = 0; i < 4; ++i) x ^= (uint32_t)d[t][i];
        if (threadIdx.x == 32) cycles[2 * blockIdx.x + 1] = t1 - t0;
    }
    sink[(size_t)blockIdx.x * kThreads + threadIdx.x] = x;
}

}  // namespace
}  // namespace lce

extern "C" lce_status lce_probe_pipe(int32_t mix, int32_t iterations, double *ops_per_second,
                                     double *ops_per_clock_per_sm, void *stream)
{
    using namespace lce;
    if (!ops_per_second || !ops_per_clock_per_sm || iterations <= 0) return LCE_ERR_INVALID_ARG;
    double ops_per_thread_iter;
    switch (mix) {
        case 0: case 1: case 2: case 3: ops_per_thread_iter = PX * CH * 9; break;
        case 10: case 11: case 13: case 14: case 15: ops_per_thread_iter = 64; break;
        case 12: ops_per_thread_iter = 128; break;            // two adds per step
        case 20: case 21: ops_per_thread_iter = 8 * 1024.0 / 32; break;  // 8 MMAs x 16*8*256/32 word pairs per warp
        case 30: case 32: ops_per_thread_iter = 4 * CH * 9 * 1.15; break;  // logic group of the combined probe (half the warps)
        case 31: case 33: ops_per_thread_iter = 8 * 1024.0 / 32; break;    // MMA group of the combined probe (half the warps)
        default: return LCE_ERR_INVALID_ARG;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LCE_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return LCE_ERR_CUDA;
    typedef void (*probe_fn)(const uint32_t *, uint32_t *, long long *, int);
    probe_fn fn = nullptr;
    switch (mix) {
        case 0: fn = probe_mix_kernel<0>; break;
        case 1: fn = probe_mix_kernel<1>; break;
        case 2: fn = probe_mix_kernel<2>; break;
        case 3: fn = probe_mix_kernel<3>; break;
        case 10: fn = probe_unit_kernel<10>; break;
        case 11: fn = probe_unit_kernel<11>; break;
        case 12: fn = probe_unit_kernel<12>; break;
        case 13: fn = probe_unit_kernel<13>; break;
        case 14: fn = probe_unit_kernel<14>; break;
        case 15: fn = probe_unit_kernel<15>; break;
        case 20: fn = probe_mma_b1_kernel<false>; break;
        case 30: case 31: fn = probe_combined_kernel<0>; break;
        case 32: fn = probe_combined_kernel<1>; break;
        case 33: fn = probe_combined_kernel<2>; break;
        default: fn = probe_mma_b1_kernel<true>; break;
    }
    // one wave exactly: as many blocks per SM as the kernel's registers let be resident
    int blocks_per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, fn, kThreads, 0) != cudaSuccess ||
        blocks_per_sm < 1)
        return LCE_ERR_CUDA;
    const int blocks = sms * blocks_per_sm;
    uint32_t *seed = nullptr, *sink = nullptr;
    long long *cycles = nullptr;
    lce_status st = LCE_ERR_CUDA;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    uint32_t host_seed[1024];
    uint32_t lcg = 2011093980u;
    for (int i = 0; i < 1024; ++i) { lcg = lcg * 1664525u + 1013904223u; host_seed[i] = lcg ^ (lcg >> 13); }
    long long *host_cycles = nullptr;
    do {
        if (cudaMalloc(&seed, sizeof(host_seed)) != cudaSuccess) break;
        if (cudaMalloc(&sink, (size_t)blocks * kThreads * 4) != cudaSuccess) break;
        if (cudaMalloc(&cycles, (size_t)blocks * 16) != cudaSuccess) break;
        if (cudaMemcpyAsync(seed, host_seed, sizeof(host_seed), cudaMemcpyHostToDevice, s) != cudaSuccess) break;
        if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) break;
        for (int rep = 0; rep < 2; ++rep) {  // first repetition warms up
            if (rep == 1) cudaEventRecord(e0, s);
            fn<<<blocks, kThreads, 0, s>>>(seed, sink, cycles, iterations);
        }
        cudaEventRecord(e1, s);
        if (cudaEventSynchronize(e1) != cudaSuccess) break;
        if (cudaGetLastError() != cudaSuccess) break;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess || ms <= 0.f) break;
        host_cycles = new long long[2 * blocks];
        if (cudaMemcpy(host_cycles, cycles, (size_t)blocks * 16, cudaMemcpyDeviceToHost) != cudaSuccess) break;
        const bool combined = mix >= 30;
        double mean_cycles = 0;
        for (int i = 0; i < blocks; ++i) mean_cycles += (double)host_cycles[combined ? 2 * i + ((mix - 30) & 1) : i];
        mean_cycles /= blocks;
        const double per_thread = ops_per_thread_iter * (double)iterations;
        // combined probe: the group is half the threads, and its rate per second is taken from its own
        // cycle count at the clock the whole launch ran at (the groups need not end together)
        const double threads = combined ? kThreads / 2 : kThreads;
        const double total = per_thread * (double)blocks * threads;
        *ops_per_clock_per_sm = per_thread * threads * blocks_per_sm / mean_cycles;
        if (combined) {
            int khz = 0;
            if (cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev) != cudaSuccess) break;
            *ops_per_second = *ops_per_clock_per_sm * sms * (double)khz * 1e3;  // at the maximum SM clock
        } else {
            *ops_per_second = total / (ms * 1e-3);
        }
        st = LCE_OK;
    } while (0);
    delete[] host_cycles;
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(seed); cudaFree(sink); cudaFree(cycles);
    return st;
}
