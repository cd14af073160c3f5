// LceBConv2d on the 5th-generation tensor cores with 4-bit operands (tcgen05 kind::mxf4, accumulators
// in TMEM).  The +-1 multiply-accumulate of the paper's binary GEMM (Section 2: dot = K - 2 popcount(a
// XOR w); Section 3.2, LceBConv2d) is an exact contraction in any number format that holds +1, -1 and
// 0: e2m1 holds all three in four bits, block scales of 1.0 change nothing, and the fp32 accumulator
// is exact for |sum| < 2^24.  One instruction multiplies 128 x N x 64 values, twice the depth of an
// 8-bit instruction for the same operand bytes, and a zero operand gives the paper's zero-padding
// variant and the channel padding without any correction term.
//
// The packed bits stay the storage and transfer format (32x smaller, Section 3.2).  A 32-bit word
// of activations or weights becomes one 16-byte row chunk of 32 e2m1 values in shared memory:
// nibble = 0x2 (+1.0) | bit << 3 (sign), four shift-and-mask operations per word; pad channels of
// the weights and, for zero-padding, pad pixels are the nibble 0 (0.0).
//
// Implicit GEMM, D[channel][position] = W[channel][k] * X[position][k]^T, M = 128 output channels (TMEM
// lanes), N = a tile of up to 224 grid positions (TMEM columns), K = 64 per instruction:
//   * positions: the images are stacked into one grid of row pitch Wg and Hg rows per image.  For
//     stride 1 the pixel (y, x) sits at (y + pad_top, x + pad_left) and rows / images share their pad
//     positions (the right pad of a row is the left pad of the next); output (oh, ow) is the
//     position of its window's top-left corner and tap (ky, kx) reads position + ky * Wg + kx.  For
//     stride 2 the padded image is split into four phase grids (row parity x column parity), in
//     which tap (ky, kx) of output (oh, ow) is position + (ky / 2) * Wg + kx / 2 of phase
//     (ky % 2, kx % 2).  Positions that are no output (pad columns, pad rows) are computed and dropped.
//   * shared memory holds, per phase, [channel word][position][16 bytes]: the B operand of a tap is
//     the same buffer shifted by the tap's position offset (K-major, no swizzle, rows 16 bytes
//     apart), so every staged position is expanded once for all taps.  T consecutive tiles share one
//     buffer of T * Nt + halo rows, so the halo a tile reads beyond its own positions is staged once
//     per T tiles; there are two to four such buffers (as many as shared memory has room for, up to what
//     lets the loaders run four tiles ahead).
//   * the weights were expanded when the model was loaded (lce_bconv2d_pack_weights) into the exact
//     operand image [channel block][tap][channel word][128 channels][16 bytes] (for out_c <= 64 the
//     channel block is repeated down the 128 rows, so that every TMEM lane quarter holds values a
//     finisher warp can work on); the bulk-copy engine brings taps into a ring of shared-memory stages
//     (cp.async.bulk + mbarrier transaction count).  If every tap fits they are fetched once per CTA,
//     all counted on one barrier; otherwise they stream past once per tile, in groups of taps that
//     alternate between two stages (one copy, one wait and one commit per group).
//   * roles: 8 loader warps (prefetch the packed words of the next chunk with cp.async, expand the
//     current one), one warp that issues the MMAs (all lanes run the same code, the elected lane
//     issues), one warp that feeds the weight ring and, once the weights are resident, issues the MMAs
//     of every other tile, 16 finisher warps (tcgen05.ld, output transform, stores).  Two accumulator
//     buffers: the MMAs of tile t and the output transform of tile t-1 overlap, and the loaders run up
//     to four tiles ahead of the finished MMAs (rings of four barriers).  The roles meet only through
//     mbarriers; every wait is bounded by time, after which the kernel records a status, waits (bounded)
//     for what it has in flight, frees its TMEM and returns.
//   * output transform (Section 3.2): a TMEM lane is a channel and a column a position.  Bit-packed
//     output: the sign of (accumulator - threshold) of 32 positions per lane, then a 32 x 32 bit
//     transpose across the warp gives each lane the finished word of one pixel.  Float / int32 output
//     is written straight from the registers: per position a warp stores its 32 consecutive channels as
//     one 128-byte line.
//   * launched with programmatic stream serialization, dependents released at kernel entry: set-up and
//     the weight copies may overlap the tail of the previous kernel of the stream; activations, shortcut
//     and outputs are touched only after griddepcontrol.wait.
#include <atomic>
#include <math.h>
#include <mutex>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "mx_common.cuh"

namespace lce {
namespace {

constexpr int kLoaders = 256;                                // warps 0-7
constexpr int kFinishers = 512;                              // warps 8-23 (warp % 4 = TMEM lane quarter, four column groups)
constexpr int kMxThreads = kLoaders + kFinishers + 64;       // + MMA issuer warp + weight producer warp
constexpr int kIssuerWarp = (kLoaders + kFinishers) / 32;
constexpr int kProducerTid = (kIssuerWarp + 1) * 32;
constexpr int kColGroups = kFinishers / 128;                 // finisher warps per TMEM lane quarter
constexpr int kMaxNt = 224;                                  // tile width (positions); two accumulators + scales fit 512 columns
constexpr uint32_t kD1Col = 240;                             // TMEM column of the second accumulator buffer
constexpr uint32_t kSfaCol = 480, kSfbCol = 496;             // block scales (all 1.0) of the A / B operand
constexpr int kMaxTaps = 64;
constexpr int kMaxStages = 32;
constexpr int kPixSlots = 8;                                 // see the note at kOffPix

// shared-memory map (bytes)
constexpr int kOffBars = 0;          // full_x[4] tile_done[4] full_d[2] empty_d[2] done[2] scales full_w[32] empty_w[32]
constexpr int kOffSlot = 1000;       // TMEM base address; 1004 fills issued, 1008 fills consumed
// int32[8][224]: output pixel of a column, or -1.  A ring of eight tiles: the finishers hand an
// accumulator back before they have stored its values, so the loaders can be up to four tiles ahead
// of a finisher that still reads its tile's slot (tile t + 5 cannot be staged before finisher t is done).
constexpr int kOffPix = 1024;
constexpr int kOffTbl = 8192;        // uint2[1024]: operand offsets (A, B; 16-byte units) of the MMAs of a tile
constexpr int kOffDyn = 16384;      // raw words, weight ring, position buffers
constexpr int kMaxTblMmas = kMaxTaps * 16;                   // 64 taps x 16 K steps (in_c <= 1024): every shape the kernel covers

enum { BAR_FULL_X0 = 0, BAR_FULL_X3 = 3, BAR_TILE_DONE0, BAR_TILE_DONE3 = BAR_TILE_DONE0 + 3, BAR_FULL_D0, BAR_FULL_D1, BAR_EMPTY_D0, BAR_EMPTY_D1, BAR_DONE, BAR_DONE_B,
       BAR_SCALES, BAR_FULL_W0,
       BAR_EMPTY_W0 = BAR_FULL_W0 + kMaxStages, BAR_COUNT = BAR_EMPTY_W0 + kMaxStages };
static_assert(BAR_COUNT * 8 <= kOffSlot, "barriers overlap the TMEM slot");


// ---- what a wait that gave up leaves behind --------------------------------------------------------------
// A device word (read by lce_device_status) and, once it has been set up, a word in mapped host memory
// that the host reads without synchronising: the next call on that device reports LCE_ERR_DEVICE_TIMEOUT.
__device__ int g_mx_status = 0;

__device__ __forceinline__ void mx_report_timeout(int *host_flag)
{
    g_mx_status = 1;
    if (host_flag) {
        *reinterpret_cast<volatile int *>(host_flag) = 1;
        __threadfence_system();
    }
}

constexpr int kFlagDevices = 64;
std::mutex g_flag_mutex;
std::atomic<int *> g_flag_host{nullptr};   // int[kFlagDevices] in mapped, portable host memory
std::atomic<int *> g_flag_dev{nullptr};    // the same array as the devices see it

// Sets the flag array up on first use.  Not a stream operation: must not run while a stream is capturing.
int *mx_flag_array(bool device_view)
{
    int *h = g_flag_host.load(std::memory_order_acquire);
    if (!h) {
        std::lock_guard<std::mutex> lock(g_flag_mutex);
        h = g_flag_host.load(std::memory_order_acquire);
        if (!h) {
            void *mem = nullptr, *dev = nullptr;
            if (cudaHostAlloc(&mem, kFlagDevices * sizeof(int), cudaHostAllocPortable | cudaHostAllocMapped) != cudaSuccess) {
                cudaGetLastError();
                return nullptr;
            }
            memset(mem, 0, kFlagDevices * sizeof(int));
            if (cudaHostGetDevicePointer(&dev, mem, 0) != cudaSuccess) {
                cudaGetLastError();
                cudaFreeHost(mem);
                return nullptr;
            }
            g_flag_dev.store(static_cast<int *>(dev), std::memory_order_release);
            g_flag_host.store(static_cast<int *>(mem), std::memory_order_release);
            h = static_cast<int *>(mem);
        }
    }
    return device_view ? g_flag_dev.load(std::memory_order_acquire) : h;
}

int current_device_index()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kFlagDevices) return -1;
    return dev;
}

// the current device's flag as a kernel argument; null while it cannot be set up (a capturing stream)
int *mx_flag_for_launch(cudaStream_t s)
{
    const int dev = current_device_index();
    if (dev < 0) return nullptr;
    if (!g_flag_host.load(std::memory_order_acquire)) {
        cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(s, &st) != cudaSuccess || st != cudaStreamCaptureStatusNone) {
            cudaGetLastError();
            return nullptr;
        }
    }
    int *arr = mx_flag_array(true);
    return arr ? arr + dev : nullptr;
}

struct MxParams {
    const uint32_t *in;
    const uint8_t *wimg;
    const float *mult;
    const float *bias;
    const int32_t *thr;
    void *out;
    const float *residual;   // fused shortcut (float output), or null
    uint32_t *out_packed;    // fused LceQuantize of the float result, or null
    int *host_flag;          // host-mapped word set when a wait gives up, or null
    int32_t N, H, W, Cw, Cw2, Cout, Cow;
    int32_t OH, OW, KH, KW, stride, pt, pl, K;
    int32_t Wg, Hg, n_phase;
    uint32_t Wg_mul, Wg_sh, Hg_mul, Hg_sh;                // divisions by Wg, Hg as multiply + shift
    uint32_t c0_mul, c0_sh, c1_mul, c1_sh;                // ... by the items per phase of a first / later chunk
    int32_t Nt, P;           // tile width; rows of a position buffer per phase and channel word = T * Nt + halo
    int32_t T, halo;         // tiles that share a position buffer; positions a tile reads beyond its own
    int32_t n_tiles, n_super, total_q;
    int32_t taps, ksteps, stages, resident;
    int32_t group_taps, groups;  // streamed weights: taps per ring stage, stages' worth of taps per tile = ceil(taps / group_taps)
    int32_t tap_bytes, raw_words, x_bytes;
    int32_t n_xbuf, ahead;   // position buffers (2..4); tiles the loaders may be ahead of the finished MMAs (2..4)
    int32_t off_w, off_x;    // byte offsets in shared memory
    int32_t cp_words;        // words per cp.async: 4, 2 or 1
    int32_t pad_zero, out_type, activation, write_float;
    int32_t dup_log2;        // log2 of the copies of the channel block in the 128 rows: 1 for out_c <= 64, 2 for out_c <= 32, else 0
};

// n / d for 0 <= n < 2^31 with (mul, sh) from the host: floor(n * mul / 2^sh), exact
__device__ __forceinline__ int fast_div(int n, uint32_t mul, uint32_t sh) { return (int)(((uint64_t)(uint32_t)n * mul) >> sh); }

// what the loaders need of the geometry, in registers (kernel parameters read inside their loops cost
// more than the arithmetic)
struct MxGeo {
    int N, H, W, Cw, Cw2, Wg, Hg, P, n_phase, stride, pt, pl, pad_zero, cp_words;
    uint32_t Wg_mul, Wg_sh, Hg_mul, Hg_sh;
    const uint32_t *in;
};

// A chunk of a position buffer: rows lo .. lo + count - 1 (of every phase), which hold the grid positions
// q0 + lo ..; (mul, sh) divide by count.
struct MxChunk {
    int q0, lo, count;
    uint32_t mul, sh;
};

// What the loader threads keep in registers for the whole kernel (read from the kernel parameters once).
struct MxLoad {
    MxGeo geo;
    int Nt, T, halo, n_tiles, n_super, OH, OW, raw_words, fast_words, n_xbuf, ahead;
    uint32_t c0_mul, c0_sh, c1_mul, c1_sh;
};

// the chunk of tile k of the super-tile that starts at position q0: the first tile brings the halo
__device__ __forceinline__ MxChunk mx_chunk_of(const MxLoad &l, int q0, int k)
{
    MxChunk c;
    c.q0 = q0;
    c.lo = k ? k * l.Nt + l.halo : 0;
    c.count = k ? l.Nt : l.Nt + l.halo;
    c.mul = k ? l.c1_mul : l.c0_mul;
    c.sh = k ? l.c1_sh : l.c0_sh;
    return c;
}

// position j of the tile that starts at q0, phase ph -> inside the image? and the pixel's word offset
__device__ __forceinline__ bool mx_locate(const MxGeo &p, int q0, int ph, int j, int64_t *word_offset)
{
    const int f = q0 + j;
    const int r = fast_div(f, p.Wg_mul, p.Wg_sh), c = f - r * p.Wg;
    const int n = fast_div(r, p.Hg_mul, p.Hg_sh), rr = r - n * p.Hg;
    const int py = p.stride == 2 ? (ph >> 1) : 0, px = p.stride == 2 ? (ph & 1) : 0;
    const int y = rr * p.stride + py - p.pt, x = c * p.stride + px - p.pl;
    const bool ok = n < p.N && (unsigned)y < (unsigned)p.H && (unsigned)x < (unsigned)p.W;
    *word_offset = ok ? (((int64_t)n * p.H + y) * p.W + x) * p.Cw : 0;
    return ok;
}

// packed words of the chunk's positions -> raw[item][Cw] (pad positions: zero words), asynchronously
__device__ __forceinline__ void mx_prefetch(const MxGeo &p, const MxChunk &c, uint32_t *raw, int ltid)
{
    const int items = p.n_phase * c.count;
    for (int i = ltid; i < items; i += kLoaders) {
        const int ph = p.n_phase == 1 ? 0 : fast_div(i, c.mul, c.sh), j = i - ph * c.count;
        int64_t off;
        const bool ok = mx_locate(p, c.q0 + c.lo, ph, j, &off);
        const uint32_t *src = p.in + off;
        uint32_t *dst = raw + (size_t)i * p.Cw;
        if (p.cp_words == 4) {
            for (int cw = 0; cw < p.Cw; cw += 4) cp_async_zfill<16>(dst + cw, src + cw, ok);
        } else if (p.cp_words == 2) {
            for (int cw = 0; cw < p.Cw; cw += 2) cp_async_zfill<8>(dst + cw, src + cw, ok);
        } else {
            for (int cw = 0; cw < p.Cw; ++cw) cp_async_zfill<4>(dst + cw, src + cw, ok);
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// every thread expands the words it prefetched itself (same item mapping): waiting for its own copies is enough
__device__ __forceinline__ void mx_expand(const MxGeo &p, const MxChunk &c, const uint32_t *raw, uint8_t *X, int ltid)
{
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    const int items = p.n_phase * c.count;
    for (int i = ltid; i < items; i += kLoaders) {
        const int ph = p.n_phase == 1 ? 0 : fast_div(i, c.mul, c.sh), j = i - ph * c.count;
        bool zero = false;
        if (p.pad_zero) {
            int64_t off;
            zero = !mx_locate(p, c.q0 + c.lo, ph, j, &off);
        }
        const uint32_t *src = raw + (size_t)i * p.Cw;
        uint4 *dst = reinterpret_cast<uint4 *>(X) + (size_t)ph * p.Cw2 * p.P + c.lo + j;
        for (int cw = 0; cw < p.Cw; ++cw) {
            uint4 v = mx_expand_word(src[cw]);
            if (zero) v = make_uint4(0u, 0u, 0u, 0u);
            dst[(size_t)cw * p.P] = v;
        }
    }
}

// The common cases (no zero-padding, aligned input; stride 1 with 2 / 4 / 8 / 16 channel words, stride 2 with
// 1 / 2 / 4 / 8) with everything about the words and the phases known at compile time: one asynchronous copy of
// 4 or 8 bytes or CW / 4 of 16 bytes per position, vector reads of the staged words, no loop or branch per
// word, the phase of an item by comparison instead of division.
template <int CW, int NPH>
__device__ __forceinline__ void mx_fast_item(const MxChunk &c, int i, int *ph, int *j)
{
    if (NPH == 1) {
        *ph = 0;
        *j = i;
    } else {
        const int h = i >= 2 * c.count ? 2 : 0;
        const int r = i - h * c.count;
        const int q = r >= c.count ? 1 : 0;
        *ph = h + q;
        *j = r - q * c.count;
    }
}

template <int CW, int NPH>
__device__ __forceinline__ void mx_prefetch_fast(const MxGeo &p, const MxChunk &c, uint32_t *raw, int ltid)
{
    const int items = NPH * c.count;
    for (int i = ltid; i < items; i += kLoaders) {
        int ph, j;
        mx_fast_item<CW, NPH>(c, i, &ph, &j);
        int64_t off;
        const bool ok = mx_locate(p, c.q0 + c.lo, ph, j, &off);
        const uint32_t *src = p.in + off;
        uint32_t *dst = raw + i * CW;
        if (CW == 1) {
            cp_async_zfill<4>(dst, src, ok);
        } else if (CW == 2) {
            cp_async_zfill<8>(dst, src, ok);
        } else {
#pragma unroll
            for (int w = 0; w < CW; w += 4) cp_async_zfill<16>(dst + w, src + w, ok);
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

template <int CW, int NPH>
__device__ __forceinline__ void mx_expand_fast(const MxGeo &p, const MxChunk &c, const uint32_t *raw, uint8_t *X, int ltid)
{
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    const int items = NPH * c.count;
    for (int i = ltid; i < items; i += kLoaders) {
        int ph, j;
        mx_fast_item<CW, NPH>(c, i, &ph, &j);
        uint32_t w[CW];
        if (CW == 1) {
            w[0] = raw[i];
        } else if (CW == 2) {
            const uint2 q = *reinterpret_cast<const uint2 *>(raw + i * 2);
            w[0] = q.x; w[1] = q.y;
        } else {
#pragma unroll
            for (int k = 0; k < CW; k += 4) {
                const uint4 q = *reinterpret_cast<const uint4 *>(raw + i * CW + k);
                w[k] = q.x; w[k + 1] = q.y; w[k + 2] = q.z; w[k + 3] = q.w;
            }
        }
        uint4 *dst = reinterpret_cast<uint4 *>(X) + (size_t)ph * p.Cw2 * p.P + c.lo + j;
#pragma unroll
        for (int k = 0; k < CW; ++k) dst[(size_t)k * p.P] = mx_expand_word(w[k]);
    }
}

// Stride 2 with an even image width and an even left pad: the pixels of the column phases 0 and 1 of a grid
// position are neighbours in memory, so one item is a row phase and a position, one copy of 2 CW words brings
// both column phases, and the address arithmetic is done once for the two.
template <int CW>
__device__ __forceinline__ void mx_prefetch_pair(const MxGeo &p, const MxChunk &c, uint32_t *raw, int ltid)
{
    const int items = 2 * c.count;
    for (int i = ltid; i < items; i += kLoaders) {
        const int py = i >= c.count ? 1 : 0, j = i - py * c.count;
        int64_t off;
        const bool ok = mx_locate(p, c.q0 + c.lo, 2 * py, j, &off);  // column phase 0; phase 1 is the next pixel, inside with it
        const uint32_t *src = p.in + off;
        uint32_t *dst = raw + i * 2 * CW;
        if (CW == 1) {
            cp_async_zfill<8>(dst, src, ok);
        } else {
#pragma unroll
            for (int w = 0; w < 2 * CW; w += 4) cp_async_zfill<16>(dst + w, src + w, ok);
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

template <int CW>
__device__ __forceinline__ void mx_expand_pair(const MxGeo &p, const MxChunk &c, const uint32_t *raw, uint8_t *X, int ltid)
{
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    const int items = 2 * c.count;
    for (int i = ltid; i < items; i += kLoaders) {
        const int py = i >= c.count ? 1 : 0, j = i - py * c.count;
        uint32_t w[2 * CW];
        if (CW == 1) {
            const uint2 q = *reinterpret_cast<const uint2 *>(raw + i * 2);
            w[0] = q.x; w[1] = q.y;
        } else {
#pragma unroll
            for (int k = 0; k < 2 * CW; k += 4) {
                const uint4 q = *reinterpret_cast<const uint4 *>(raw + i * 2 * CW + k);
                w[k] = q.x; w[k + 1] = q.y; w[k + 2] = q.z; w[k + 3] = q.w;
            }
        }
        uint4 *dst0 = reinterpret_cast<uint4 *>(X) + (size_t)(2 * py) * p.Cw2 * p.P + c.lo + j;  // column phase 0
        uint4 *dst1 = dst0 + (size_t)p.Cw2 * p.P;                                                 // column phase 1
#pragma unroll
        for (int k = 0; k < CW; ++k) {
            dst0[(size_t)k * p.P] = mx_expand_word(w[k]);
            dst1[(size_t)k * p.P] = mx_expand_word(w[CW + k]);
        }
    }
}

// which form the loaders use: 0 the general one, else channel words (+ 32 for the stride-2 form, + 64 for the
// stride-2 form that copies the two column phases together)
__device__ __forceinline__ int mx_fast_words(const MxGeo &p)
{
    const bool words_ok = (p.Cw == 1) || (p.Cw == 2 && p.cp_words >= 2) || ((p.Cw == 4 || p.Cw == 8 || p.Cw == 16) && p.cp_words == 4);
    if (p.pad_zero || !words_ok) return 0;
    if (p.n_phase == 1) return p.Cw >= 2 ? p.Cw : 0;
    const bool pairs = (p.W & 1) == 0 && (p.pl & 1) == 0 && (reinterpret_cast<uintptr_t>(p.in) & 15) == 0 && p.Cw <= 4;
    return pairs ? 64 + p.Cw : p.Cw == 8 ? 40 : 0;
}

__device__ __forceinline__ void mx_prefetch_any(int fw, const MxGeo &p, const MxChunk &c, uint32_t *raw, int ltid)
{
    if (fw == 2) mx_prefetch_fast<2, 1>(p, c, raw, ltid);
    else if (fw == 4) mx_prefetch_fast<4, 1>(p, c, raw, ltid);
    else if (fw == 8) mx_prefetch_fast<8, 1>(p, c, raw, ltid);
    else if (fw == 16) mx_prefetch_fast<16, 1>(p, c, raw, ltid);
    else if (fw == 40) mx_prefetch_fast<8, 4>(p, c, raw, ltid);
    else if (fw == 65) mx_prefetch_pair<1>(p, c, raw, ltid);
    else if (fw == 66) mx_prefetch_pair<2>(p, c, raw, ltid);
    else if (fw == 68) mx_prefetch_pair<4>(p, c, raw, ltid);
    else mx_prefetch(p, c, raw, ltid);
}

__device__ __forceinline__ void mx_expand_any(int fw, const MxGeo &p, const MxChunk &c, const uint32_t *raw, uint8_t *X, int ltid)
{
    if (fw == 2) mx_expand_fast<2, 1>(p, c, raw, X, ltid);
    else if (fw == 4) mx_expand_fast<4, 1>(p, c, raw, X, ltid);
    else if (fw == 8) mx_expand_fast<8, 1>(p, c, raw, X, ltid);
    else if (fw == 16) mx_expand_fast<16, 1>(p, c, raw, X, ltid);
    else if (fw == 40) mx_expand_fast<8, 4>(p, c, raw, X, ltid);
    else if (fw == 65) mx_expand_pair<1>(p, c, raw, X, ltid);
    else if (fw == 66) mx_expand_pair<2>(p, c, raw, X, ltid);
    else if (fw == 68) mx_expand_pair<4>(p, c, raw, X, ltid);
    else mx_expand(p, c, raw, X, ltid);
}

// B operand of tap (ky, kx): its phase buffer (stride 2) shifted by the tap's position offset, in 16-byte units
__device__ __forceinline__ uint32_t tap_b_offset(const MxParams &p, int ky, int kx)
{
    if (p.stride == 2) return (uint32_t)((((ky & 1) * 2 + (kx & 1)) * p.Cw2) * p.P + (ky >> 1) * p.Wg + (kx >> 1));
    return (uint32_t)(ky * p.Wg + kx);
}

// One lane of the converged warp, the same one every time
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
    return pred != 0;
}

// N MMAs straight from a table of operand offsets, back to back in one block of code: the loads of the
// block are independent, and between two MMAs there is nothing but the next descriptor's move.  The
// issuing warp pays about 100 clocks per tcgen05.mma in its instruction stream, whether the instruction
// is predicated off or not (measured), so blocks come in exact sizes (8, 4, 2, 1) instead of one
// predicated block of eight.  The whole issuer warp runs this; only the elected lane issues.
template <int N>
__device__ __forceinline__ void mx_issue_block(uint32_t tmem_d, const uint2 *tbl, uint32_t a_base, uint32_t b_base, uint32_t desc_hi,
                                               uint32_t idesc, uint32_t sfa, uint32_t sfb, uint32_t accumulate);
template <>
__device__ __forceinline__ void mx_issue_block<8>(uint32_t tmem_d, const uint2 *tbl, uint32_t a_base, uint32_t b_base, uint32_t desc_hi,
                                                  uint32_t idesc, uint32_t sfa, uint32_t sfb, uint32_t accumulate)
{
    uint32_t a[8], b[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const uint2 o = tbl[k];
        a[k] = a_base + o.x;
        b[k] = b_base + o.y;
    }
    if (elect_one()) {
        asm volatile(
            "{\n\t.reg .pred pa, pt;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 pa, %21, 0;\n\t"
            "setp.eq.b32 pt, 0, 0;\n\t"
            "mov.b64 da, {%1, %17};\n\t mov.b64 db, {%9, %17};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %18, [%19], [%20], pa;\n\t"
            "mov.b64 da, {%2, %17};\n\t mov.b64 db, {%10, %17};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %18, [%19], [%20], pt;\n\t"
            "mov.b64 da, {%3, %17};\n\t mov.b64 db, {%11, %17};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %18, [%19], [%20], pt;\n\t"
            "mov.b64 da, {%4, %17};\n\t mov.b64 db, {%12, %17};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %18, [%19], [%20], pt;\n\t"
            "mov.b64 da, {%5, %17};\n\t mov.b64 db, {%13, %17};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %18, [%19], [%20], pt;\n\t"
            "mov.b64 da, {%6, %17};\n\t mov.b64 db, {%14, %17};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %18, [%19], [%20], pt;\n\t"
            "mov.b64 da, {%7, %17};\n\t mov.b64 db, {%15, %17};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %18, [%19], [%20], pt;\n\t"
            "mov.b64 da, {%8, %17};\n\t mov.b64 db, {%16, %17};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %18, [%19], [%20], pt;\n\t"
            "}"
            :
            : "r"(tmem_d), "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(a[4]), "r"(a[5]), "r"(a[6]), "r"(a[7]), "r"(b[0]), "r"(b[1]), "r"(b[2]), "r"(b[3]), "r"(b[4]), "r"(b[5]), "r"(b[6]), "r"(b[7]), "r"(desc_hi), "r"(idesc), "r"(sfa), "r"(sfb), "r"(accumulate)
            : "memory");
    }
}
template <>
__device__ __forceinline__ void mx_issue_block<4>(uint32_t tmem_d, const uint2 *tbl, uint32_t a_base, uint32_t b_base, uint32_t desc_hi,
                                                  uint32_t idesc, uint32_t sfa, uint32_t sfb, uint32_t accumulate)
{
    uint32_t a[4], b[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint2 o = tbl[k];
        a[k] = a_base + o.x;
        b[k] = b_base + o.y;
    }
    if (elect_one()) {
        asm volatile(
            "{\n\t.reg .pred pa, pt;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 pa, %13, 0;\n\t"
            "setp.eq.b32 pt, 0, 0;\n\t"
            "mov.b64 da, {%1, %9};\n\t mov.b64 db, {%5, %9};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %10, [%11], [%12], pa;\n\t"
            "mov.b64 da, {%2, %9};\n\t mov.b64 db, {%6, %9};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %10, [%11], [%12], pt;\n\t"
            "mov.b64 da, {%3, %9};\n\t mov.b64 db, {%7, %9};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %10, [%11], [%12], pt;\n\t"
            "mov.b64 da, {%4, %9};\n\t mov.b64 db, {%8, %9};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %10, [%11], [%12], pt;\n\t"
            "}"
            :
            : "r"(tmem_d), "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]), "r"(b[2]), "r"(b[3]), "r"(desc_hi), "r"(idesc), "r"(sfa), "r"(sfb), "r"(accumulate)
            : "memory");
    }
}
template <>
__device__ __forceinline__ void mx_issue_block<2>(uint32_t tmem_d, const uint2 *tbl, uint32_t a_base, uint32_t b_base, uint32_t desc_hi,
                                                  uint32_t idesc, uint32_t sfa, uint32_t sfb, uint32_t accumulate)
{
    uint32_t a[2], b[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const uint2 o = tbl[k];
        a[k] = a_base + o.x;
        b[k] = b_base + o.y;
    }
    if (elect_one()) {
        asm volatile(
            "{\n\t.reg .pred pa, pt;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 pa, %9, 0;\n\t"
            "setp.eq.b32 pt, 0, 0;\n\t"
            "mov.b64 da, {%1, %5};\n\t mov.b64 db, {%3, %5};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %6, [%7], [%8], pa;\n\t"
            "mov.b64 da, {%2, %5};\n\t mov.b64 db, {%4, %5};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %6, [%7], [%8], pt;\n\t"
            "}"
            :
            : "r"(tmem_d), "r"(a[0]), "r"(a[1]), "r"(b[0]), "r"(b[1]), "r"(desc_hi), "r"(idesc), "r"(sfa), "r"(sfb), "r"(accumulate)
            : "memory");
    }
}
template <>
__device__ __forceinline__ void mx_issue_block<1>(uint32_t tmem_d, const uint2 *tbl, uint32_t a_base, uint32_t b_base, uint32_t desc_hi,
                                                  uint32_t idesc, uint32_t sfa, uint32_t sfb, uint32_t accumulate)
{
    uint32_t a[1], b[1];
#pragma unroll
    for (int k = 0; k < 1; ++k) {
        const uint2 o = tbl[k];
        a[k] = a_base + o.x;
        b[k] = b_base + o.y;
    }
    if (elect_one()) {
        asm volatile(
            "{\n\t.reg .pred pa, pt;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 pa, %7, 0;\n\t"
            "setp.eq.b32 pt, 0, 0;\n\t"
            "mov.b64 da, {%1, %3};\n\t mov.b64 db, {%2, %3};\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %4, [%5], [%6], pa;\n\t"
            "}"
            :
            : "r"(tmem_d), "r"(a[0]), "r"(b[0]), "r"(desc_hi), "r"(idesc), "r"(sfa), "r"(sfb), "r"(accumulate)
            : "memory");
    }
}

__device__ __forceinline__ void mx_issue_table(uint32_t tmem_d, const uint2 *tbl, int count, uint32_t a_base, uint32_t b_base, uint32_t desc_hi,
                                               uint32_t idesc, uint32_t sfa, uint32_t sfb, uint32_t &accumulate)
{
    int i = 0;
    for (; i + 8 <= count; i += 8) {
        mx_issue_block<8>(tmem_d, tbl + i, a_base, b_base, desc_hi, idesc, sfa, sfb, accumulate);
        accumulate = 1;
    }
    if (count & 4) {
        mx_issue_block<4>(tmem_d, tbl + i, a_base, b_base, desc_hi, idesc, sfa, sfb, accumulate);
        accumulate = 1;
        i += 4;
    }
    if (count & 2) {
        mx_issue_block<2>(tmem_d, tbl + i, a_base, b_base, desc_hi, idesc, sfa, sfb, accumulate);
        accumulate = 1;
        i += 2;
    }
    if (count & 1) {
        mx_issue_block<1>(tmem_d, tbl + i, a_base, b_base, desc_hi, idesc, sfa, sfb, accumulate);
        accumulate = 1;
    }
}

// 32 x 32 bit transpose across the warp: in: lane = row, bit j = column j; out: lane j holds column j.
// Five butterfly steps; in step k a lane keeps the bits under its mask and takes the others from its
// partner's word rotated by k towards them (the bits that wrap around fall under the kept mask).  The
// per-lane masks and rotation counts are worked out once per warp: a step is one shuffle, one funnel shift
// and one three-input logic operation.
struct Transpose32 {
    uint32_t keep[5];   // bits this lane keeps in the steps k = 16, 8, 4, 2, 1
    uint32_t rot[5];    // left-rotation of the partner's word
};

__device__ __forceinline__ Transpose32 transpose32_setup(int lane)
{
    Transpose32 t;
#pragma unroll
    for (int i = 0; i < 5; ++i) {
        const int k = 16 >> i;
        const uint32_t low = k == 16 ? 0x0000FFFFu : k == 8 ? 0x00FF00FFu : k == 4 ? 0x0F0F0F0Fu : k == 2 ? 0x33333333u : 0x55555555u;
        // a lane without bit k keeps its low halves and takes the partner's low halves moved up by k;
        // a lane with bit k keeps its high halves and takes the partner's high halves moved down by k
        t.keep[i] = (lane & k) ? ~low : low;
        t.rot[i] = (lane & k) ? 32u - (uint32_t)k : (uint32_t)k;
    }
    return t;
}

__device__ __forceinline__ uint32_t warp_transpose32(uint32_t m, const Transpose32 &t)
{
#pragma unroll
    for (int i = 0; i < 5; ++i) {
        const uint32_t y = __shfl_xor_sync(0xffffffffu, m, 16 >> i);
        const uint32_t moved = __funnelshift_l(y, y, t.rot[i]);
        m = (m & t.keep[i]) | (moved & ~t.keep[i]);
    }
    return m;
}

// What a finisher warp needs for every tile, worked out once before its tile loop (divisions and
// kernel-parameter reads per tile cost a third of the warp's instructions when they sat in the epilogue).
// TMEM lane quarter of the warp = warp % 4; with few output channels the 128 rows hold `dup` copies of
// the channel block, and the warps of copy `sub` take other columns than those of copy 0, so that no
// finisher warp is idle.
struct MxFin {
    int Nt, n_chunks;        // tile width; 32-column chunks of a tile
    int group, n_groups;     // this warp takes chunks group, group + n_groups, ...
    int last_chunk;          // its last one (-1: none: nothing to read for this warp)
    uint32_t lane_off;       // TMEM lane offset of its quarter
    bool ch_ok;              // this lane's channel exists
    float thr, mult, bias;   // this lane's channel: threshold (-inf if it does not exist), multiplier, bias
    int64_t cout, cow;
    uint32_t *out_words;     // bit-packed output, at this warp's channel word
    float *outp;             // float / int32 output, at this lane's channel
    const float *resp;       // shortcut tensor at this lane's channel, or null
    uint32_t *packp;         // re-quantised copy at this warp's channel word, or null
    bool relu, write_float;
    Transpose32 tr;          // bit-packed output: the transpose's per-lane constants
};

__device__ __forceinline__ MxFin mx_fin_context(const MxParams &p, int fw, int lane, int ch0)
{
    MxFin f;
    const int quarter = fw & 3, dl = p.dup_log2;                    // dup = 1 << dl copies of the channel block
    const int cq = quarter & ((4 >> dl) - 1), sub = quarter >> (2 - dl);
    const int channel = ch0 + cq * 32 + lane;
    f.Nt = p.Nt;
    f.n_chunks = (p.Nt + 31) >> 5;
    f.group = ((fw >> 2) << dl) + sub;
    f.n_groups = kColGroups << dl;                                   // 4, 8 or 16
    const bool real = ch0 + cq * 32 < p.Cout && f.group < f.n_chunks;
    f.last_chunk = real ? f.group + ((f.n_chunks - 1 - f.group) & ~(f.n_groups - 1)) : -1;
    f.lane_off = (uint32_t)(quarter * 32) << 16;
    f.ch_ok = channel < p.Cout;
    // this lane's constants straight from global memory (constants of the model, never the previous kernel's
    // output): their latency passes while the first tile is being staged
    f.thr = -INFINITY;
    if (f.ch_ok && p.out_type == LCE_OUT_BITPACKED) {
        // acc < thr is unchanged by clamping thr to [-K-1, K+1] (|acc| <= K), and then thr is exact in fp32
        f.thr = (float)max(-p.K - 1, min(p.K + 1, __ldg(p.thr + channel)));
    }
    f.mult = (f.ch_ok && p.out_type == LCE_OUT_FLOAT32) ? __ldg(p.mult + channel) : 0.f;
    f.bias = (f.ch_ok && p.out_type == LCE_OUT_FLOAT32) ? __ldg(p.bias + channel) : 0.f;
    f.cout = p.Cout;
    f.cow = p.Cow;
    f.out_words = static_cast<uint32_t *>(p.out) + (ch0 >> 5) + cq;
    f.outp = static_cast<float *>(p.out) + channel;
    f.resp = p.residual ? p.residual + channel : nullptr;
    f.packp = p.out_packed ? p.out_packed + (ch0 >> 5) + cq : nullptr;
    f.relu = p.activation == LCE_ACT_RELU;
    f.write_float = p.write_float != 0;
    f.tr = transpose32_setup(lane);
    return f;
}

// Bit-packed output of one tile (Section 3.2: accumulator compared with the per-channel threshold).
// Lane = channel; per 32-column chunk the sign of (accumulator - threshold) of 32 positions, then a 32 x 32
// bit transpose across the warp gives every lane the finished word of one pixel.
__device__ __forceinline__ void mx_epilogue_bits(const MxFin &f, uint32_t tmem_d, const int32_t *sPix, int lane, uint64_t *empty_d)
{
    for (int ck = f.group; ck <= f.last_chunk; ck += f.n_groups) {
        const int c0 = ck * 32;
        float v[32];
        const bool full = c0 + 32 <= f.Nt;
        if (full) tmem_ld32(tmem_d + f.lane_off + (uint32_t)c0, v);
        else tmem_ld16(tmem_d + f.lane_off + (uint32_t)c0, v);
        if (ck == f.last_chunk) {  // last read of the accumulator by this warp: hand it back before the arithmetic
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(empty_d);
        }
        // bit j = (acc_j < thr): the sign of acc - thr (both are small integers held exactly);
        // four short chains instead of one long one
        uint32_t m0 = 0u, m1 = 0u, m2 = 0u, m3 = 0u;
#pragma unroll
        for (int j = 7; j >= 0; --j) {
            m0 = __funnelshift_l(__float_as_uint(v[j] - f.thr), m0, 1);
            m1 = __funnelshift_l(__float_as_uint(v[8 + j] - f.thr), m1, 1);
            m2 = __funnelshift_l(__float_as_uint(v[16 + j] - f.thr), m2, 1);
            m3 = __funnelshift_l(__float_as_uint(v[24 + j] - f.thr), m3, 1);
        }
        uint32_t m = m0 | (m1 << 8);
        if (full) m |= (m2 << 16) | (m3 << 24);
        const uint32_t word = warp_transpose32(m, f.tr);
        const int pix = (c0 + lane < f.Nt) ? sPix[c0 + lane] : -1;
        if (pix >= 0) f.out_words[pix * f.cow] = word;
    }
    if (f.last_chunk < 0) {  // nothing to read for this warp
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        mbar_arrive(empty_d);
    }
}

// Float / int32 output of one tile (Section 3.2: int -> float, fused activation, one multiply-add;
// Section 5.3: optional shortcut add and re-quantisation).  A lane holds one channel of 32 positions:
// for every position the warp writes its 32 consecutive channels as one 128-byte store, so a value
// costs one multiply-add and one store instruction and nothing is staged.  The re-quantised copy is a
// warp ballot of the signs: the finished word of the pixel.  Everything the loops need sits in
// registers before they start (kernel parameters read inside them cost more than the arithmetic).
enum { EPI_FLOAT = 0, EPI_FLOAT_FUSED = 1, EPI_INT32 = 2, EPI_BITS = 3, EPI_PLAIN = 4 };

template <int MODE>
__device__ __forceinline__ void mx_store_chunk(const float (&v)[32], int cols, const int32_t *sPixChunk, int64_t cout, float *outp,
                                               bool ch_ok, float mult, float bias)
{
    // straight-line code: every store is predicated, nothing branches, so the 32 positions' address
    // arithmetic, multiply-adds and stores overlap instead of running one position after the other
#pragma unroll
    for (int j4 = 0; j4 < 32; j4 += 4) {
        const int4 pix4 = *reinterpret_cast<const int4 *>(sPixChunk + j4);  // the same for every lane (slots past the tile: never stored)
        const int pix[4] = {pix4.x, pix4.y, pix4.z, pix4.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const bool st = ch_ok && pix[u] >= 0 && j4 + u < cols;
            const int64_t o = pix[u] * cout;
            if (MODE != EPI_INT32) {
                const float y = __fmaf_rn(v[j4 + u], mult, bias);
                if (st) outp[o] = y;
            } else {
                const int32_t y = __float2int_rn(v[j4 + u]);
                if (st) reinterpret_cast<int32_t *>(outp)[o] = y;
            }
        }
    }
}

template <int MODE>
__device__ __forceinline__ void mx_epilogue_values(const MxFin &f, uint32_t tmem_d, const int32_t *sPix, int lane, uint64_t *empty_d)
{
    for (int ck = f.group; ck <= f.last_chunk; ck += f.n_groups) {
        const int c0 = ck * 32;
        const int cols = min(32, f.Nt - c0);
        float v[32];
        if (cols == 32) tmem_ld32(tmem_d + f.lane_off + (uint32_t)c0, v);
        else tmem_ld16(tmem_d + f.lane_off + (uint32_t)c0, v);
        if (ck == f.last_chunk) {  // last read of the accumulator by this warp
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(empty_d);
        }
        mx_store_chunk<MODE>(v, cols, sPix + c0, f.cout, f.outp, f.ch_ok, f.mult, f.bias);
    }
    if (f.last_chunk < 0) {  // nothing to read for this warp
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        mbar_arrive(empty_d);
    }
}

// Float output with the shortcut add and the re-quantised copy fused in (Section 5.3).  Per 32-column chunk
// the warp first asks for the shortcut values of all 32 positions (they do not depend on the accumulator:
// 32 independent 128-byte loads in flight per warp; with eight the memory latency set the pace), then reads
// the accumulators 16 columns at a time, and per position does the multiply-add, the add, the 128-byte store
// and the ballot whose result is the pixel's finished word.
template <bool RES, bool PACK, bool WRITE_FLOAT>
__device__ __forceinline__ void mx_epilogue_fused_as(const MxFin &f, uint32_t tmem_d, const int32_t *sPix, int lane, uint64_t *empty_d)
{
    // which of the three parts (shortcut add, re-quantised copy, float output) a launch has is a template
    // argument: a test of a pointer per position turns the unrolled block below into branchy code that
    // runs at a third of the speed (measured on the plain float transform, and again here)
    const float floor_v = f.relu ? 0.f : -INFINITY;
    for (int ck = f.group; ck <= f.last_chunk; ck += f.n_groups) {
        const int c0 = ck * 32;
        const int cols = min(32, f.Nt - c0);  // 32, or 16 in a tile's last chunk
        const int32_t *pixc = sPix + c0;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            if (half * 16 < cols) {
                // the shortcut values of the half's 16 positions first (they do not depend on the accumulator: 16
                // independent 128-byte loads in flight per warp), then the accumulators
                float r[16];
                if (RES) {
#pragma unroll
                    for (int j4 = 0; j4 < 16; j4 += 4) {
                        const int4 p4 = *reinterpret_cast<const int4 *>(pixc + half * 16 + j4);  // the same for every lane
                        const int pix[4] = {p4.x, p4.y, p4.z, p4.w};
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const bool ld = f.ch_ok && pix[u] >= 0 && half * 16 + j4 + u < cols;
                            r[j4 + u] = ld ? __ldg(f.resp + (ld ? pix[u] : 0) * f.cout) : 0.f;
                        }
                    }
                }
                float v[16];
                tmem_ld16x(tmem_d + f.lane_off + (uint32_t)(c0 + half * 16), v);
                if (ck == f.last_chunk && (half + 1) * 16 >= cols) {  // last read of the accumulator by this warp
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    mbar_arrive(empty_d);
                }
                uint32_t my_word = 0u;  // lane u keeps the re-quantised word of the half's position u: one store for the 16
#pragma unroll
                for (int j4 = 0; j4 < 16; j4 += 4) {
                    const int4 p4 = *reinterpret_cast<const int4 *>(pixc + half * 16 + j4);
                    const int pix[4] = {p4.x, p4.y, p4.z, p4.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const bool pos_ok = pix[u] >= 0 && half * 16 + j4 + u < cols;  // the same for every lane
                        float y = __fmaf_rn(fmaxf(v[j4 + u], floor_v), f.mult, f.bias);
                        if (RES) y = __fadd_rn(y, r[j4 + u]);
                        if (WRITE_FLOAT) {
                            if (f.ch_ok && pos_ok) f.outp[pix[u] * f.cout] = y;
                        }
                        if (PACK) {
                            const uint32_t word = __ballot_sync(0xffffffffu, f.ch_ok && y < 0.f);
                            if (lane == j4 + u) my_word = word;
                        }
                    }
                }
                if (PACK) {
                    const int my_pos = half * 16 + (lane & 15);
                    const int my_pix = pixc[my_pos];
                    if (lane < 16 && my_pix >= 0 && my_pos < cols) f.packp[my_pix * f.cow] = my_word;
                }
            }
        }
    }
    if (f.last_chunk < 0) {  // nothing to read for this warp
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        mbar_arrive(empty_d);
    }
}

__device__ __forceinline__ void mx_epilogue_fused(const MxFin &f, uint32_t tmem_d, const int32_t *sPix, int lane, uint64_t *empty_d)
{
    const int form = (f.resp != nullptr ? 4 : 0) | (f.packp != nullptr ? 2 : 0) | (f.write_float ? 1 : 0);
    switch (form) {
        case 1: mx_epilogue_fused_as<false, false, true>(f, tmem_d, sPix, lane, empty_d); break;
        case 2: mx_epilogue_fused_as<false, true, false>(f, tmem_d, sPix, lane, empty_d); break;
        case 3: mx_epilogue_fused_as<false, true, true>(f, tmem_d, sPix, lane, empty_d); break;
        case 5: mx_epilogue_fused_as<true, false, true>(f, tmem_d, sPix, lane, empty_d); break;
        case 6: mx_epilogue_fused_as<true, true, false>(f, tmem_d, sPix, lane, empty_d); break;
        case 7: mx_epilogue_fused_as<true, true, true>(f, tmem_d, sPix, lane, empty_d); break;
        default: mx_epilogue_fused_as<false, false, false>(f, tmem_d, sPix, lane, empty_d); break;  // nothing to write: only hands the accumulator back
    }
}

// EPI: EPI_PLAIN carries the three plain output transforms (bit-packed, float, int32; chosen per launch by the
// output type), EPI_FLOAT_FUSED the float transform with the shortcut add, the activation and the re-quantised
// copy.  One instantiation for the plain forms matters more than their few KB of code: a network alternates
// bit-packed and float layers, and two kernels of 160 KB alternating evict each other from the SMs' instruction
// caches at every launch (config 2 as one flushed step: 103 us with a kernel per form, 87 us with one for all
// three); the fused form stays apart because its register needs spoil the float form's code when they share one.
template <int EPI>
__global__ void __launch_bounds__(kMxThreads, 1) bconv_mx_kernel(const __grid_constant__ MxParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kOffBars);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + kOffSlot);
    int32_t *fills = reinterpret_cast<int32_t *>(smem + kOffSlot + 4);  // [0] issued by the producer, [1] consumed by the issuer
    int32_t *sPix = reinterpret_cast<int32_t *>(smem + kOffPix);
    uint2 *tbl = reinterpret_cast<uint2 *>(smem + kOffTbl);
    uint32_t *raw0 = reinterpret_cast<uint32_t *>(smem + kOffDyn);
    uint8_t *sW = smem + p.off_w;
    uint8_t *sX0 = smem + p.off_x;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ch0 = blockIdx.y * 128;
    const int first_tile = blockIdx.x, tile_step = gridDim.x;

    // the next kernel of the stream may start setting itself up as soon as every CTA of this one has got here
    if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- set-up, its parts side by side: the issuer warp allocates TMEM, the producer warp initialises the
    // barriers and starts the weight copies, the finisher warps fill the table of operand offsets, the
    // loaders fetch the first chunk of activations ---------------------------------------------------------
    const int n_mma = p.taps * p.ksteps;
    // the weight producer's progress (one thread): fills issued, ring stage and (tile-local) tap group of the next one
    int prod_g = 0, prod_total = 0, prod_stage = 0, prod_tap = 0;
    uint32_t prod_parity = 1;  // the first pass over the ring waits for nothing
    if (warp == kIssuerWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else if (warp == kIssuerWarp + 1) {
        for (int b = lane; b < BAR_COUNT; b += 32) {
            const uint32_t count = b <= BAR_FULL_X3 ? kLoaders : (b == BAR_EMPTY_D0 || b == BAR_EMPTY_D1) ? kFinishers : b == BAR_SCALES ? 4 : 1;
            mbar_init(&bars[b], count);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        __syncwarp();
        // The weights are constants of the model: their copies start at once, whatever the previous kernel of
        // the stream is still doing, one lane per copy.  Resident: all taps, every copy counted on the same
        // barrier; streamed: the first pass over the ring (stage = fill number; at most 32 stages).
        const uint8_t *src = p.wimg + (size_t)blockIdx.y * p.taps * p.tap_bytes;
        if (p.resident) {
            if (lane == 0) mbar_expect_tx(&bars[BAR_FULL_W0], (uint32_t)(p.taps * p.tap_bytes));
            __syncwarp();
            for (int tap = lane; tap < p.taps; tap += 32)
                bulk_copy_g2s(sW + (size_t)tap * p.tap_bytes, src + (size_t)tap * p.tap_bytes, (uint32_t)p.tap_bytes, &bars[BAR_FULL_W0]);
            prod_g = 1;
        } else {
            int my_tiles = 0;
            for (int st = first_tile; st < p.n_super; st += tile_step) my_tiles += min(p.T, p.n_tiles - st * p.T);
            // a fill = one group of up to group_taps consecutive taps (one copy: they are contiguous in the image)
            prod_total = my_tiles * p.groups;
            prod_g = min(p.stages, prod_total);
            if (lane < prod_g) {
                const int first = (lane % p.groups) * p.group_taps;
                const uint32_t bytes = (uint32_t)(min(p.group_taps, p.taps - first) * p.tap_bytes);
                mbar_expect_tx(&bars[BAR_FULL_W0 + lane], bytes);
                bulk_copy_g2s(sW + (size_t)lane * p.group_taps * p.tap_bytes, src + (size_t)first * p.tap_bytes, bytes, &bars[BAR_FULL_W0 + lane]);
            }
            prod_tap = prod_g % p.groups;   // the next fill's group within its tile
            if (prod_g == p.stages) prod_parity ^= 1u; else prod_stage = prod_g;
        }
        __syncwarp();
        if (lane == 0) {
            fills[0] = prod_g;
            fills[1] = 0;
        }
    } else if (tid >= kLoaders) {
        for (int e = tid - kLoaders; e < n_mma; e += kFinishers) {
            const int tap = e / p.ksteps, kk = e - tap * p.ksteps;
            const int ky = tap / p.KW, kx = tap - ky * p.KW;
            // A: K step (+ the tap's ring stage when all taps are resident: stage = tap); B: the tap's offset + K step
            const uint32_t b_off = tap_b_offset(p, ky, kx);
            tbl[e] = make_uint2((p.resident ? (uint32_t)tap * ((uint32_t)p.tap_bytes >> 4) : 0u) + 256u * kk, b_off + 2u * (uint32_t)p.P * kk);
        }
    }
    // The loaders' first prefetch goes out before the CTA-wide barrier of the set-up: it needs the previous
    // kernel's output (hence the dependency wait) and plain shared memory, nothing that is set up above.
    MxLoad ld;
    if (tid < kLoaders) {
        MxGeo &geo = ld.geo;
        geo.N = p.N; geo.H = p.H; geo.W = p.W; geo.Cw = p.Cw; geo.Cw2 = p.Cw2; geo.Wg = p.Wg; geo.Hg = p.Hg; geo.P = p.P;
        geo.n_phase = p.n_phase; geo.stride = p.stride; geo.pt = p.pt; geo.pl = p.pl; geo.pad_zero = p.pad_zero; geo.cp_words = p.cp_words;
        geo.Wg_mul = p.Wg_mul; geo.Wg_sh = p.Wg_sh; geo.Hg_mul = p.Hg_mul; geo.Hg_sh = p.Hg_sh;
        geo.in = p.in;
        ld.Nt = p.Nt; ld.T = p.T; ld.halo = p.halo; ld.n_tiles = p.n_tiles; ld.n_super = p.n_super; ld.OH = p.OH; ld.OW = p.OW;
        ld.raw_words = p.raw_words; ld.n_xbuf = p.n_xbuf; ld.ahead = p.ahead;
        ld.c0_mul = p.c0_mul; ld.c0_sh = p.c0_sh; ld.c1_mul = p.c1_mul; ld.c1_sh = p.c1_sh;
        ld.fast_words = mx_fast_words(geo);
        asm volatile("griddepcontrol.wait;" ::: "memory");  // the activations may come from the previous kernel
        if (first_tile < ld.n_super) {
            // through the general form where its staging layout is the fast form's too (all but the paired stride-2
            // form): one more inlined copy of every fast form costs more in code size than it saves here
            const MxChunk c0 = mx_chunk_of(ld, first_tile * ld.T * ld.Nt, 0);
            if (ld.fast_words >= 64) mx_prefetch_any(ld.fast_words, geo, c0, raw0, tid);
            else mx_prefetch(geo, c0, raw0, tid);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    if (warp >= kLoaders / 32 && warp < kLoaders / 32 + 4) {
        // block scales: every byte 0x7F = 2^0 (ue8m0), for all 128 lanes of the 32 scale columns, written by the
        // first four finisher warps (one per lane quarter; they have nothing else to do yet); the issuer
        // waits for the four arrivals before its first MMA
        const uint32_t one = 0x7F7F7F7Fu;
        const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + kSfaCol;
#pragma unroll
        for (int c = 0; c < 32; c += 8)
            asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1};" ::"r"(taddr + c), "r"(one) : "memory");
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars[BAR_SCALES]);
    }

    bool ok = true;
    if (tid < kLoaders) {
        // ======================= loaders ==============================================================
        const MxGeo &geo = ld.geo;
        const int Nt = ld.Nt, T = ld.T, n_tiles = ld.n_tiles, n_super = ld.n_super, OH = ld.OH, OW = ld.OW, raw_words = ld.raw_words;
        const size_t x_bytes = (size_t)p.x_bytes;
        auto chunk_of = [&](int q0, int k) { return mx_chunk_of(ld, q0, k); };
        const int n_xbuf = ld.n_xbuf, ahead = ld.ahead;
        int it = 0, xbuf = 0;
        for (int st = first_tile; st < n_super && ok; st += tile_step, xbuf = xbuf + 1 == n_xbuf ? 0 : xbuf + 1) {
            const int q0 = st * T * Nt;
            uint8_t *X = sX0 + xbuf * x_bytes;
            for (int k = 0; k < T && st * T + k < n_tiles; ++k, ++it) {
                if (it >= ahead) {
                    // At most `ahead` tiles in front of the finished MMAs: those of tile it - ahead are done (a
                    // ring of four barriers, one commit per tile).  That keeps the arrivals on the four full_x
                    // barriers within one phase of what the issuer has seen, and (the MMAs finish in order; ahead
                    // <= (n_xbuf - 1) * T + 1) it means that the super-tile whose position buffer this chunk
                    // overwrites has been read completely.
                    const int done = it - ahead;
                    ok = mbar_wait_bounded(&bars[BAR_TILE_DONE0 + (done & 3)], (uint32_t)(done >> 2) & 1u);
                    if (!ok) break;
                }
                mx_expand_any(ld.fast_words, geo, chunk_of(q0, k), raw0 + (it & 1) * raw_words, X, tid);
                if (tid < Nt) {
                    const int f = q0 + k * Nt + tid;
                    const int r = fast_div(f, geo.Wg_mul, geo.Wg_sh), c = f - r * geo.Wg;
                    const int n = fast_div(r, geo.Hg_mul, geo.Hg_sh), rr = r - n * geo.Hg;
                    const bool col_ok = n < geo.N && rr < OH && c < OW;
                    sPix[(it & (kPixSlots - 1)) * kMaxNt + tid] = col_ok ? (n * OH + rr) * OW + c : -1;
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(&bars[BAR_FULL_X0 + (it & 3)]);
                // only now the words of the next chunk: the MMAs of this tile must not wait for loads they do not need
                const bool more_here = k + 1 < T && st * T + k + 1 < n_tiles;
                if (more_here || st + tile_step < n_super)
                    mx_prefetch_any(ld.fast_words, geo, more_here ? chunk_of(q0, k + 1) : chunk_of((st + tile_step) * T * Nt, 0),
                                    raw0 + ((it + 1) & 1) * raw_words, tid);
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else if (tid < kLoaders + kFinishers) {
        // ======================= finishers ============================================================
        const int fw = warp - kLoaders / 32;  // 0..15: lane quarter fw & 3 (= warp & 3), column group fw >> 2
        const MxFin fin = mx_fin_context(p, fw, lane, ch0);
        asm volatile("griddepcontrol.wait;" ::: "memory");  // outputs and the shortcut tensor: only after the previous kernel
        const int T = p.T, n_tiles = p.n_tiles, n_super = p.n_super, out_type = p.out_type;
        uint32_t par_full_d[2] = {0, 0};
        int it = 0;
        for (int st = first_tile; st < n_super && ok; st += tile_step) {
            for (int k = 0; k < T && st * T + k < n_tiles; ++k, ++it) {
                const int buf = it & 1;
                ok = mbar_wait_bounded(&bars[BAR_FULL_D0 + buf], par_full_d[buf]);
                par_full_d[buf] ^= 1u;
                ok = __all_sync(0xffffffffu, ok);  // the warp goes on together (its epilogue uses warp-wide shuffles and ballots)
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmem_d = tmem_base + (buf ? kD1Col : 0u);
                const int32_t *pix = sPix + (it & (kPixSlots - 1)) * kMaxNt;
                if (EPI == EPI_FLOAT_FUSED) mx_epilogue_fused(fin, tmem_d, pix, lane, &bars[BAR_EMPTY_D0 + buf]);
                else if (out_type == LCE_OUT_BITPACKED) mx_epilogue_bits(fin, tmem_d, pix, lane, &bars[BAR_EMPTY_D0 + buf]);
                else if (out_type == LCE_OUT_INT32) mx_epilogue_values<EPI_INT32>(fin, tmem_d, pix, lane, &bars[BAR_EMPTY_D0 + buf]);
                else mx_epilogue_values<EPI_FLOAT>(fin, tmem_d, pix, lane, &bars[BAR_EMPTY_D0 + buf]);
            }
        }
    } else if (warp == kIssuerWarp || (warp == kIssuerWarp + 1 && p.resident != 0)) {
        // ======================= MMA issuer: a warp, every lane with the same values ==================
        // With the weights resident the producer warp has nothing left to do and becomes a second issuer: the
        // two take alternate tiles (one accumulator buffer each), so that one warp's per-tile bookkeeping and
        // waits run while the other's MMAs are in the pipe.
        const int my_parity = warp - kIssuerWarp;
        // instruction descriptor (block-scaled kinds): A, B = e2m1 (1), both K-major, N >> 3 at bit 17,
        // scales ue8m0 (bit 23), M >> 4 at bit 24, scale-factor ids 0
        const uint32_t idesc = (1u << 7) | (1u << 10) | ((uint32_t)(p.Nt >> 3) << 17) | (1u << 23) | ((uint32_t)(128 >> 4) << 24);
        // shared-memory descriptors (units of 16 bytes): low = start | K-chunk stride << 16; high = 8-row
        // group stride (128 bytes) | version 1 at bit 46; no swizzle
        const uint32_t desc_hi = 8u | (1u << 14);
        // everything the loops use, read from the kernel parameters once
        const int T = p.T, n_tiles = p.n_tiles, n_super = p.n_super, Nt = p.Nt, ksteps = p.ksteps, stages = p.stages, taps = p.taps, group_taps = p.group_taps;
        const bool resident = p.resident != 0;
        const uint32_t w_lo0 = ((uint32_t)p.off_w >> 4) + (smem_u32(smem) >> 4) + (128u << 16);
        const uint32_t x_lo_buf0 = ((uint32_t)p.off_x >> 4) + (smem_u32(smem) >> 4) + ((uint32_t)p.P << 16);
        const uint32_t x_units = (uint32_t)p.x_bytes >> 4, tap_units = (uint32_t)p.tap_bytes >> 4;
        const uint32_t group_units = tap_units * (uint32_t)p.group_taps;
        const uint32_t sfa = tmem_base + kSfaCol, sfb = tmem_base + kSfbCol;
        uint32_t par_empty_d[2] = {0, 0};
        const int n_xbuf = p.n_xbuf;
        ok = __all_sync(0xffffffffu, mbar_wait_bounded(&bars[BAR_SCALES], 0));  // the block scales are in TMEM
        int g = 0, stage_i = 0;
        uint32_t w_parity = 0;
        int it = 0;
        int xbuf = 0;
        for (int st = first_tile; st < n_super && ok; st += tile_step, xbuf = xbuf + 1 == n_xbuf ? 0 : xbuf + 1)
        for (int k = 0; k < T && st * T + k < n_tiles && ok; ++k, ++it) {
            const int buf = it & 1;
            if (resident && buf != my_parity) continue;
            ok = mbar_wait_bounded(&bars[BAR_FULL_X0 + (it & 3)], (uint32_t)(it >> 2) & 1u);
            if (ok && it >= 2) {  // the accumulator buffer must have been read out
                ok = mbar_wait_bounded(&bars[BAR_EMPTY_D0 + buf], par_empty_d[buf]);
                par_empty_d[buf] ^= 1u;
            }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t tmem_d = tmem_base + (buf ? kD1Col : 0u);
            // B operand: the super-tile's position buffer from this tile's first row on
            const uint32_t x_lo0 = x_lo_buf0 + (uint32_t)xbuf * x_units + (uint32_t)(k * Nt);
            uint32_t accumulate = 0;
            if (resident) {
                // every tap stays in shared memory: one wait for all of them (a single barrier counts the bytes
                // of all the copies) before the CTA's first tile, then nothing between the MMAs of a tile
                if (it < 2) {  // this warp's first tile
                    ok = __all_sync(0xffffffffu, mbar_wait_bounded(&bars[BAR_FULL_W0], 0));
                    if (!ok) break;
                    if (lane == 0) fills[1] = 1;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                }
                mx_issue_table(tmem_d, tbl, n_mma, w_lo0, x_lo0, desc_hi, idesc, sfa, sfb, accumulate);
            } else {
                // the taps stream through the ring a group at a time: wait for the group, issue its taps' MMAs,
                // hand its stage back (the wait, the commit and the bookkeeping cost this warp about 600 clocks,
                // as much as six MMAs: hence groups, not single taps)
                int tap = 0;
                while (tap < taps) {
                    ok = __all_sync(0xffffffffu, mbar_wait_bounded(&bars[BAR_FULL_W0 + stage_i], w_parity));
                    if (!ok) break;
                    ++g;
                    if (lane == 0) fills[1] = g;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    uint32_t a_tap = w_lo0 + (uint32_t)stage_i * group_units;
                    const int group_end = min(taps, tap + group_taps);
                    for (; tap < group_end; ++tap, a_tap += tap_units)
                        mx_issue_table(tmem_d, tbl + tap * ksteps, ksteps, a_tap, x_lo0, desc_hi, idesc, sfa, sfb, accumulate);
                    if (elect_one()) mma_commit(&bars[BAR_EMPTY_W0 + stage_i]);
                    if (++stage_i == stages) { stage_i = 0; w_parity ^= 1u; }
                }
            }
            if (!ok) break;
            if (elect_one()) {
                mma_commit(&bars[BAR_FULL_D0 + buf]);         // to the finishers: the accumulator is complete
                mma_commit(&bars[BAR_TILE_DONE0 + (it & 3)]);  // to the loaders: the tile's operands have been read
            }
        }
    } else if (tid == kProducerTid) {
        // ======================= weight producer: one thread, the rest of the streamed taps ===========
        const uint8_t *src = p.wimg + (size_t)blockIdx.y * p.taps * p.tap_bytes;
        for (; !p.resident && prod_g < prod_total; ++prod_g) {
            ok = mbar_wait_bounded(&bars[BAR_EMPTY_W0 + prod_stage], prod_parity);
            if (!ok) break;
            const int first = prod_tap * p.group_taps;
            const uint32_t bytes = (uint32_t)(min(p.group_taps, p.taps - first) * p.tap_bytes);
            mbar_expect_tx(&bars[BAR_FULL_W0 + prod_stage], bytes);
            bulk_copy_g2s(sW + (size_t)prod_stage * p.group_taps * p.tap_bytes, src + (size_t)first * p.tap_bytes, bytes, &bars[BAR_FULL_W0 + prod_stage]);
            fills[0] = prod_g + 1;
            if (++prod_tap == p.groups) prod_tap = 0;
            if (++prod_stage == p.stages) { prod_stage = 0; prod_parity ^= 1u; }
        }
    }
    if (!ok) mx_report_timeout(p.host_flag);

    // ---- tear-down: nothing of this CTA may still be in flight when its TMEM and shared memory go ----
    // When no wait gave up, the finishers have waited for the MMAs of every tile and the issuer for every
    // weight copy; otherwise the lane that issued the MMAs waits for what is still under way.
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    const bool all_ok = __syncthreads_and(ok) != 0;
    if (!all_ok || fills[0] != fills[1]) {
        if ((warp == kIssuerWarp || (warp == kIssuerWarp + 1 && p.resident != 0)) && elect_one()) {
            uint64_t *done = &bars[warp == kIssuerWarp ? BAR_DONE : BAR_DONE_B];
            mma_commit(done);                                  // arrives when every MMA this lane issued has finished
            bool drained = mbar_wait_bounded(done, 0);
            // weight copies that were started but never consumed
            const int issued = fills[0], consumed = fills[1];
            for (int g = consumed; warp == kIssuerWarp && g < issued && drained; ++g)
                drained = mbar_wait_bounded(&bars[BAR_FULL_W0 + g % p.stages], (uint32_t)(g / p.stages) & 1u);
            if (!drained) mx_report_timeout(p.host_flag);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == kIssuerWarp) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
}

// ---- load-time weight image -----------------------------------------------------------------------------
// plain packed words [Cout][taps][Cw] -> e2m1 operand image [channel block][tap][Cw2][128 channels][16 bytes];
// channels past Cout, the pad channel word of an odd Cw and channels past Cin inside a word are 0.0; with out_c
// <= 64 (<= 32) the rows hold two (four) copies of the channels, so that every TMEM lane quarter has work for a
// finisher warp
__global__ void mx_pack_weights_kernel(const uint32_t *w, uint4 *image, int Cout, int Cin, int Cw, int Cw2, int taps, int n_blocks, int dup)
{
    const int64_t total = (int64_t)n_blocks * taps * Cw2 * 128;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int row = (int)(e & 127);
        int64_t t = e >> 7;
        const int cw = (int)(t % Cw2);
        t /= Cw2;
        const int tap = (int)(t % taps);
        const int blk = (int)(t / taps);
        const int o = blk * 128 + (row & (128 / dup - 1));  // few output channels: the block is repeated down the 128 rows
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (o < Cout && cw < Cw) {
            v = mx_expand_word(w[((int64_t)o * taps + tap) * Cw + cw]);
            const int valid = Cin - cw * 32;  // channels of this word that exist
            if (valid < 32) {
                // value (register j, nibble i) is channel 4 i + j of the word
                uint32_t m[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    m[j] = 0u;
                    for (int i = 0; i < 8; ++i)
                        if (4 * i + j < valid) m[j] |= 0xFu << (4 * i);
                }
                v.x &= m[0]; v.y &= m[1]; v.z &= m[2]; v.w &= m[3];
            }
        }
        image[e] = v;
    }
}

struct MxPlan {
    int Nt, P, T, stages, resident, group_taps, groups, n_blocks, ctas_x, n_tiles, n_super, total_q, Wg, Hg, n_phase, Cw2, taps, halo, n_xbuf, ahead;
    size_t raw_words, x_bytes, tap_bytes, off_w, off_x, smem;
};

constexpr size_t kSmemLimit = 227 * 1024;

bool mx_plan_uncached(const ConvGeom &g, int sms, MxPlan *pl);

// The plan depends on the geometry alone, and a network repeats few geometries: the last few plans of
// each host thread are kept (the search below walks about a hundred candidates otherwise).
bool mx_plan(const ConvGeom &g, int sms, MxPlan *pl)
{
    struct Entry {
        ConvGeom g;
        int sms;
        bool valid, found;
        MxPlan plan;
    };
    constexpr int kEntries = 16;
    static thread_local Entry cache[kEntries];
    static thread_local int next = 0;
    for (int i = 0; i < kEntries; ++i) {
        const Entry &e = cache[i];
        if (e.valid && e.sms == sms && memcmp(&e.g, &g, sizeof(ConvGeom)) == 0) {
            *pl = e.plan;
            return e.found;
        }
    }
    Entry &e = cache[next];
    next = (next + 1) % kEntries;
    memset(&e.g, 0, sizeof(ConvGeom));
    e.g = g;
    e.sms = sms;
    e.found = mx_plan_uncached(g, sms, &e.plan);
    e.valid = true;
    *pl = e.plan;
    return e.found;
}

bool mx_plan_uncached(const ConvGeom &g, int sms, MxPlan *pl)
{
    if (g.sh != g.sw || (g.sh != 1 && g.sh != 2)) return false;
    if (g.Cw > 32) return false;
    const int taps = g.KH * g.KW;
    if (taps > kMaxTaps) return false;
    const int s = g.sh;
    int Wg, Hg, halo;
    if (s == 1) {
        const int pr = max(0, (g.OW - 1) + g.KW - g.W - g.pl), pb = max(0, (g.OH - 1) + g.KH - g.H - g.pt);
        Wg = g.W + max(g.pl, pr);
        Hg = g.H + max(g.pt, pb);
        halo = (g.KH - 1) * Wg + (g.KW - 1);
    } else {
        Wg = g.OW + (g.KW - 1) / 2;
        Hg = g.OH + (g.KH - 1) / 2;
        halo = ((g.KH - 1) / 2) * Wg + (g.KW - 1) / 2;
    }
    const int64_t total_q = (int64_t)g.N * Hg * Wg;
    if (total_q >= (1ll << 31) - 4096 || g.M >= (1ll << 31)) return false;
    pl->Wg = Wg; pl->Hg = Hg; pl->halo = halo; pl->total_q = (int)total_q;
    pl->n_phase = s * s;
    pl->Cw2 = g.Cw + (g.Cw & 1);
    pl->taps = taps;
    pl->tap_bytes = (size_t)pl->Cw2 * 2048;
    pl->n_blocks = (g.Cout + 127) / 128;
    const int ctas_max = max(1, sms / pl->n_blocks);
    const int ksteps = pl->Cw2 / 2;
    double best = 1e30;
    bool found = false;
    for (int nt = 16; nt <= kMaxNt; nt += 16) {
        const int n_tiles = (int)((total_q + nt - 1) / nt);
        for (int T = 1; T <= 8; ++T) {
            // T tiles share one position buffer of T * nt + halo rows: the halo is staged once per T tiles
            const int P = T * nt + halo;
            if (P > 16383) break;  // descriptor strides are 14-bit counts of 16 bytes
            if (T > 1 && (T - 1) * ctas_max >= n_tiles) break;   // no CTA would have that many tiles
            const size_t raw_words = (((size_t)pl->n_phase * (nt + halo) * g.Cw + 3) / 4) * 4;
            const size_t x_bytes = (size_t)pl->n_phase * pl->Cw2 * P * 16;
            const size_t fixed = kOffDyn + 2 * raw_words * 4;
            const size_t off_w = (fixed + 127) / 128 * 128;
            const size_t rest = 2 * x_bytes + 256;
            if (off_w + rest + (taps > 1 ? 2 : 1) * pl->tap_bytes > kSmemLimit) break;
            // taps that fit beside the position buffers: all of them -> resident (one stage per tap, one barrier);
            // otherwise a ring of two stages of half the fitting taps each (a group costs the issuer one wait and
            // one commit, whatever its size: two large groups measured better than three or four smaller ones)
            const int slots = (int)((kSmemLimit - off_w - rest) / pl->tap_bytes);
            const bool resident = slots >= taps;
            int stages, group_taps, groups;
            if (resident) {
                stages = taps; group_taps = 1; groups = taps;
            } else {
                group_taps = slots >= 4 ? slots / 2 : 1;
                groups = (taps + group_taps - 1) / group_taps;
                group_taps = (taps + groups - 1) / groups;  // even groups
                stages = min(kMaxStages, slots / group_taps);
            }
            const int n_super = (n_tiles + T - 1) / T;
            const int ctas_x = min(ctas_max, n_super);
            const int per_cta = ((n_super + ctas_x - 1) / ctas_x) * T;
            // clocks per MMA: 43 + N/2, at least 100 (measured); the loaders need about 400 + 8 clocks per staged
            // position and tile
            const double mma1 = fmax(100.0, 43.0 + nt / 2.0);
            const double mma = (double)taps * ksteps * mma1;
            // a streamed tap: its bytes from L2 (every SM streams at once: the L2 gives each about 19 bytes per clock,
            // 5.5 TB/s in all), or its share of a copy's latency, or what the single issuer needs
            // per tap (wait for the stage, issue, hand the stage back: about 600 clocks on top of the MMAs;
            // measured on a nine-tap, one-MMA-per-tap layer: 6000 clocks per tile whether 2 or 4 stages)
            const double stream = resident ? 0.0 : (double)groups * fmax(fmax(group_taps * pl->tap_bytes / 19.0, 1300.0 / stages), 600.0 + group_taps * ksteps * mma1);
            // stride 2: four phases per position, staged two at a time where the geometry allows (mx_prefetch_pair)
            const double per_position = s == 1 ? 1.0 : ((g.W & 1) == 0 && (g.pl & 1) == 0 && g.Cw <= 4) ? 2.0 : 3.0;
            const double load = 400.0 + 8.0 * per_position * (nt + (double)halo / T);
            const double cost = per_cta * (fmax(fmax(mma, stream), load) + 150.0);
            if (cost < best) {
                best = cost;
                found = true;
                pl->Nt = nt; pl->P = P; pl->T = T; pl->stages = stages; pl->resident = resident ? 1 : 0; pl->group_taps = group_taps; pl->groups = groups;
                pl->n_tiles = n_tiles; pl->n_super = n_super; pl->ctas_x = ctas_x;
                pl->raw_words = raw_words; pl->x_bytes = x_bytes;
                pl->off_w = off_w;
                pl->off_x = (off_w + (size_t)stages * group_taps * pl->tap_bytes + 127) / 128 * 128;
                // More position buffers where shared memory is left over (thin layers): the loaders may then be
                // up to four tiles ahead, ahead <= (n_xbuf - 1) * T + 1, and the hand-overs between the roles
                // (a few hundred clocks each) drop out of the per-tile cycle.
                int n_xbuf = 2;
                while (n_xbuf < 4 && (n_xbuf - 1) * T + 1 < 4 && pl->off_x + (size_t)(n_xbuf + 1) * x_bytes <= kSmemLimit) ++n_xbuf;
                pl->n_xbuf = n_xbuf;
                pl->ahead = min(4, (n_xbuf - 1) * T + 1);
                pl->smem = pl->off_x + (size_t)n_xbuf * x_bytes;
            }
        }
    }
    return found;
}

// floor(n / d) = (n * mul) >> sh for every 0 <= n < 2^31: sh = 31 + ceil(log2 d), mul = floor(2^sh / d) + 1
// (the excess mul * d - 2^sh is at most d <= 2^(sh - 31), so n * excess < 2^sh)
void fast_div_constants(uint32_t d, uint32_t *mul, uint32_t *sh)
{
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;
    *sh = 31 + l;
    *mul = (uint32_t)(((1ull << (31 + l)) / d) + 1);
}

template <int EPI>
lce_status launch_mx(const MxParams &p, dim3 grid, size_t smem, cudaStream_t s)
{
    static SmemOptIn opted;
    if (!opted.ensure(bconv_mx_kernel<EPI>, smem)) return LCE_ERR_CUDA;
    // Programmatic dependent launch: the CTAs of this grid may be scheduled while the previous kernel of the
    // stream is still draining; they set themselves up and fetch their weights (constants of the model),
    // and wait for the previous kernel's completion (griddepcontrol.wait) before they touch anything it may
    // have written or may still read: the activations, the shortcut tensor, the outputs.
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kMxThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, bconv_mx_kernel<EPI>, p) != cudaSuccess) {
        cudaGetLastError();
        return LCE_ERR_CUDA;
    }
    return LCE_OK;
}

int mx_dup(const ConvGeom &g) { return g.Cout <= 32 ? 4 : g.Cout <= 64 ? 2 : 1; }

int device_sms()
{
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms > 0 ? sms : 148;
}

}  // namespace

bool tensor_covers(const ConvGeom &g)
{
    MxPlan pl;
    return mx_plan(g, 148, &pl);
}

size_t tensor_weight_image_bytes(const ConvGeom &g)
{
    MxPlan pl;
    if (!mx_plan(g, 148, &pl)) return 0;
    return (size_t)pl.n_blocks * pl.taps * pl.tap_bytes;
}

lce_status launch_pack_weights_tensor(const ConvGeom &g, const uint32_t *w, void *image, cudaStream_t s)
{
    MxPlan pl;
    if (!mx_plan(g, 148, &pl)) return LCE_ERR_UNSUPPORTED;
    const int64_t total = (int64_t)pl.n_blocks * pl.taps * pl.Cw2 * 128;
    const int64_t want = (total + 255) / 256;
    const int blocks = (int)(want < 4096 ? want : 4096);
    mx_pack_weights_kernel<<<blocks, 256, 0, s>>>(w, static_cast<uint4 *>(image), g.Cout, g.Cin, g.Cw, pl.Cw2, pl.taps, pl.n_blocks, mx_dup(g));
    mx_flag_array(false);  // load time is the moment to set up the host-visible status word (it cannot be done under stream capture)
    return launch_status();
}

lce_status tensor_plan_info(const ConvGeom &g, TensorPlanInfo *info)
{
    MxPlan pl;
    if (!mx_plan(g, device_sms(), &pl)) return LCE_ERR_UNSUPPORTED;
    info->tile_positions = pl.Nt;
    info->ctas = pl.ctas_x * pl.n_blocks;
    info->weight_stages = pl.stages;
    info->weights_resident = pl.resident;
    info->shared_bytes = (int64_t)pl.smem;
    return LCE_OK;
}

lce_status launch_bconv_tensor(const ConvGeom &g, const uint32_t *in, const void *w_image, const float *mult, const float *bias,
                               const int32_t *thr, void *out, cudaStream_t s, const float *residual, uint32_t *out_packed)
{
    MxPlan pl;
    if (!w_image || !mx_plan(g, device_sms(), &pl)) return LCE_ERR_UNSUPPORTED;
    MxParams p{};
    p.in = in; p.wimg = static_cast<const uint8_t *>(w_image); p.mult = mult; p.bias = bias; p.thr = thr; p.out = out;
    p.residual = residual; p.out_packed = out_packed;
    p.host_flag = mx_flag_for_launch(s);
    p.N = g.N; p.H = g.H; p.W = g.W; p.Cw = g.Cw; p.Cw2 = pl.Cw2; p.Cout = g.Cout; p.Cow = g.Cow;
    p.OH = g.OH; p.OW = g.OW; p.KH = g.KH; p.KW = g.KW; p.stride = g.sh; p.pt = g.pt; p.pl = g.pl;
    p.K = g.KH * g.KW * g.Cin;
    p.Wg = pl.Wg; p.Hg = pl.Hg; p.n_phase = pl.n_phase;
    fast_div_constants((uint32_t)pl.Wg, &p.Wg_mul, &p.Wg_sh);
    fast_div_constants((uint32_t)pl.Hg, &p.Hg_mul, &p.Hg_sh);
    fast_div_constants((uint32_t)(pl.Nt + pl.halo), &p.c0_mul, &p.c0_sh);
    fast_div_constants((uint32_t)pl.Nt, &p.c1_mul, &p.c1_sh);
    p.Nt = pl.Nt; p.P = pl.P; p.T = pl.T; p.halo = pl.halo; p.n_tiles = pl.n_tiles; p.n_super = pl.n_super; p.total_q = pl.total_q;
    p.taps = pl.taps; p.ksteps = pl.Cw2 / 2; p.stages = pl.stages; p.resident = pl.resident; p.group_taps = pl.group_taps; p.groups = pl.groups;
    p.tap_bytes = (int32_t)pl.tap_bytes; p.raw_words = (int32_t)pl.raw_words; p.x_bytes = (int32_t)pl.x_bytes;
    p.n_xbuf = pl.n_xbuf; p.ahead = pl.ahead;
    p.off_w = (int32_t)pl.off_w; p.off_x = (int32_t)pl.off_x;
    p.cp_words = (g.Cw % 4 == 0 && aligned(in, 16)) ? 4 : (g.Cw % 2 == 0 && aligned(in, 8)) ? 2 : 1;
    p.pad_zero = g.padding == LCE_PAD_SAME_ZERO;
    p.out_type = g.out_type; p.activation = g.activation;
    p.write_float = out != nullptr;
    p.dup_log2 = mx_dup(g) == 4 ? 2 : mx_dup(g) == 2 ? 1 : 0;
    if (!aligned(w_image, 16)) return LCE_ERR_ALIGNMENT;
    const dim3 grid((unsigned)pl.ctas_x, (unsigned)pl.n_blocks);
    if (g.out_type == LCE_OUT_FLOAT32 && (residual || out_packed || !out || g.activation != LCE_ACT_NONE))
        return launch_mx<EPI_FLOAT_FUSED>(p, grid, pl.smem, s);
    return launch_mx<EPI_PLAIN>(p, grid, pl.smem, s);
}


// ---- status of the bounded waits ----------------------------------------------------------------------
namespace {
// One CTA waits, with the kernels' own helper and the given limit, on a barrier that nobody arrives
// at, and reports the expiry the way the convolution kernels do.  Touches no tensor-core state.
__global__ void mx_wait_probe_kernel(uint64_t limit_ns, int *host_flag)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait_bounded(&bar, 0, limit_ns)) mx_report_timeout(host_flag);
    }
}
}  // namespace

lce_status tensor_wait_probe(uint64_t limit_ns, cudaStream_t s)
{
    mx_wait_probe_kernel<<<1, 32, 0, s>>>(limit_ns, mx_flag_for_launch(s));
    return launch_status();
}

// 0 = no bounded wait has given up on the current device since the library was loaded (or since the reset).
lce_status tensor_device_status(int *status)
{
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_mx_status, sizeof(int)) != cudaSuccess) return LCE_ERR_CUDA;
    *status = v;
    return LCE_OK;
}

lce_status tensor_device_status_reset()
{
    const int zero = 0;
    if (cudaMemcpyToSymbol(g_mx_status, &zero, sizeof(int)) != cudaSuccess) return LCE_ERR_CUDA;
    const int dev = current_device_index();
    int *arr = g_flag_host.load(std::memory_order_acquire);
    if (arr && dev >= 0) *reinterpret_cast<volatile int *>(arr + dev) = 0;
    return LCE_OK;
}

// Host-side look at the mapped word: no synchronisation, no CUDA call beyond cudaGetDevice.
bool tensor_timeout_flagged()
{
    int *arr = g_flag_host.load(std::memory_order_acquire);
    if (!arr) return false;
    const int dev = current_device_index();
    return dev >= 0 && *reinterpret_cast<volatile int *>(arr + dev) != 0;
}

}  // namespace lce
