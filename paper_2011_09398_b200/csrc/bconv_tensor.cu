// LceBConv2d on the 5th-generation tensor cores (tcgen05 kind::i8, accumulators in TMEM): the
// +-1 multiply-accumulate of the paper's binary GEMM (Section 2; Section 3.2) is an exact int8
// contraction once every bit is expanded to the byte +1 / -1.  The packed bits stay the storage
// and transfer format (32x smaller, as in the paper); the expansion happens in shared memory.
//
// 3x3, stride 1, one-padding, as an implicit GEMM with the "shifted window" trick:
//   * the images of the batch are stacked into one tall padded grid with ONE shared pad row
//     between images and ONE shared pad column per row (row pitch Wp = W+1): the right pad of a
//     row is the left pad of the next, the bottom pad of an image the top pad of the next.  Pad
//     positions hold +1 bytes, which is exactly the paper's one-padding.
//   * GEMM row q = flat index of the window's top-left corner in that grid; tap (ky,kx) of row q
//     is grid position q + ky*Wp + kx.  So in shared memory, laid out as
//     [16-channel chunk][grid position][16 bytes], the A operand of a tap is the SAME buffer
//     shifted by (ky*Wp + kx) * 16 bytes: every staged pixel is expanded once and used by all nine
//     taps.  Rows whose window starts on a pad column / pad row are computed and thrown away
//     ((H+1)(W+1)/(HW) of the work: 4 % at 56x56, 31 % at 7x7).
//   * operand descriptors: K-major, no swizzle, 8-row groups 128 bytes apart (so rows are
//     uniformly 16 bytes apart), the two 16-byte K chunks of one K=32 instruction one whole
//     plane apart.
//   * one CTA = 128 GEMM rows (TMEM lanes) x a block of output channels (TMEM columns), persistent
//     over row tiles.  The packed input words of the next tile are prefetched with cp.async.
//     Two schedules:
//       - RESIDENT (small K*N): the block's weights are expanded once and stay in shared memory;
//         per tile one thread issues all 9*Cw MMAs, and while they run all threads expand the
//         next tile's input into the other A buffer;
//       - STREAMING (large K*N): the weights of one tap at a time are expanded into one of two
//         B buffers while the previous tap's MMAs run.
//   * tcgen05.commit signals MMA completion on mbarriers; every wait on them is bounded; on expiry
//     the kernel records a status word, abandons its work, frees its TMEM and returns.
#include <stdio.h>
#include <stdlib.h>

#include "common.cuh"

namespace lce {
namespace {

constexpr int kWorkers = 256;  // 8 worker warps: warps w and w+4 share TMEM lanes 32*(w%4).. and split the columns
constexpr int kThreads = kWorkers + 32;  // + one warp that only issues MMAs
constexpr int kTileM = 128;
constexpr uint32_t kSpinLimit = 1u << 22;  // bounded wait: about a second at worst, far above any real tile

__device__ int g_tensor_status = 0;  // 0 ok, 1 = an mbarrier wait expired
#ifdef LCE_TUNING
__device__ long long g_dbg[256];
#define DBG_T(slot) do { if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0 && it < 6) g_dbg[it * 8 + (slot)] = clock64(); } while (0)
#else
#define DBG_T(slot) do {} while (0)
#endif

struct TensorParams {
    const uint32_t *in;
    const uint32_t *w;
    const float *mult;
    const float *bias;
    const int32_t *thr;
    void *out;
    int32_t N, H, W, Cin, Cw, Cout, Cow;
    int32_t Wp;          // grid row pitch = W + 1
    int32_t Hs;          // rows per image in the stacked grid = H + 1
    int32_t P;           // staged grid positions per tile = kTileM + 2*Wp + 2
    int32_t n_tiles;     // ceil(total grid positions / kTileM)
    int32_t total_q;     // N * Hs * Wp
    int32_t n_blk;       // output channels per CTA: 32, 64, 128 or 256
    int32_t n_blk_log2;
    int32_t tmem_cols;   // power of two >= max(32, n_blk)
    int32_t pad_corr;    // 9 * (32*Cw - Cin): what the zero pad bits (+1 * +1) add to every accumulator
    int32_t out_type, activation;
    int32_t vec_store;   // float / int32 rows may be written with 128-bit stores (2: with 256-bit stores)
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait; false when the limit was reached.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity)
{
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 4096) __nanosleep(128);  // long waits back off; short ones wake up at once
    }
    return false;
}

__device__ __forceinline__ void mma_commit(uint64_t *bar)
{
    // arrives on the barrier when every MMA issued so far has finished (operand reads included)
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, int32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, "
        "[%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

// 4-byte asynchronous global->shared copy; with valid == false a zero word is written
__device__ __forceinline__ void cp_async4_zfill(uint32_t *smem_dst, const uint32_t *gmem_src, bool valid)
{
    const int src_size = valid ? 4 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(src_size) : "memory");
}

// 32 bits -> 32 bytes (+1 where the bit is 0, -1 where it is 1), as two 16-byte chunks; the
// table maps one byte of bits to its eight bytes
__device__ __forceinline__ void expand_word(const uint2 *table, uint32_t word, uint4 *chunk_lo, uint4 *chunk_hi)
{
    const uint2 a = table[word & 0xFFu], b = table[(word >> 8) & 0xFFu];
    const uint2 c = table[(word >> 16) & 0xFFu], d = table[word >> 24];
    *chunk_lo = make_uint4(a.x, a.y, b.x, b.y);
    *chunk_hi = make_uint4(c.x, c.y, d.x, d.y);
}

// The same expansion without the table, on the integer pipes only (the streaming schedule expands
// weights while the tensor core streams both operands from shared memory, so shared-memory
// bandwidth is the scarce resource there).  For a 4-bit value n, n * 0x00204081 puts bit i at
// bit 8i (other partial products land between the byte boundaries and are masked away); then
// byte = 1 + 254*bit.
__device__ __forceinline__ uint32_t expand_nibble(uint32_t n)
{
    const uint32_t spread = (n * 0x00204081u) & 0x01010101u;
    return spread * 0xFEu + 0x01010101u;
}
__device__ __forceinline__ void expand_word_alu(uint32_t word, uint4 *chunk_lo, uint4 *chunk_hi)
{
    uint32_t r[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) r[k] = expand_nibble((word >> (4 * k)) & 0xFu);
    *chunk_lo = make_uint4(r[0], r[1], r[2], r[3]);
    *chunk_hi = make_uint4(r[4], r[5], r[6], r[7]);
}

// packed words of the grid positions q0 .. q0+P-1 -> raw[cw*P + row] (pad positions: zero word)
template <int STRIDE = kWorkers>
__device__ __forceinline__ void prefetch_raw(const TensorParams &p, int q0, uint32_t *raw, int tid)
{
    for (int row = tid; row < p.P; row += STRIDE) {
        const int f = q0 + row;
        const int rr = f / p.Wp, cc = f - rr * p.Wp;
        const int n = rr / p.Hs, ry = rr - n * p.Hs;
        const bool ok = cc != 0 && ry != 0 && n < p.N;
        const uint32_t *src = ok ? p.in + (((int64_t)n * p.H + (ry - 1)) * p.W + (cc - 1)) * p.Cw : p.in;
        for (int cw = 0; cw < p.Cw; ++cw) cp_async4_zfill(raw + cw * p.P + row, ok ? src + cw : src, ok);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// every thread expands the words it prefetched itself (same row mapping), so waiting for its own
// copies is enough
template <int STRIDE = kWorkers, bool USE_TABLE = false>
__device__ __forceinline__ void expand_a(const TensorParams &p, const uint2 *table, const uint32_t *raw, uint8_t *sA, int tid)
{
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    for (int row = tid; row < p.P; row += STRIDE) {
        for (int cw = 0; cw < p.Cw; ++cw) {
            uint4 lo, hi;
            if (USE_TABLE) expand_word(table, raw[cw * p.P + row], &lo, &hi);
            else expand_word_alu(raw[cw * p.P + row], &lo, &hi);
            uint4 *dst = reinterpret_cast<uint4 *>(sA) + (size_t)(2 * cw) * p.P + row;
            dst[0] = lo;
            dst[p.P] = hi;
        }
    }
}

// Issues MMAs first .. first+count-1 of a tile.  One thread feeds the whole tensor core, so
// its instruction stream must be short: the start offsets of both operands of every MMA of a
// tile sit in a shared-memory table (filled once per CTA), and eight MMAs at a time are issued
// back to back from one block of code.  A descriptor's high half (row-group stride, version)
// never changes; its low half = (base + offset) | plane stride << 16.
__device__ __forceinline__ void issue_mmas(uint32_t tmem, const uint2 *offs, int first, int count, uint32_t a_base_lo,
                                           uint32_t b_base_lo, uint32_t desc_hi, uint32_t idesc, uint32_t &accumulate)
{
    for (int i0 = 0; i0 < count; i0 += 8) {
        uint32_t a_lo[8], b_lo[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint2 o = offs[first + min(i0 + k, count - 1)];
            a_lo[k] = a_base_lo + o.x;
            b_lo[k] = b_base_lo + o.y;
        }
        const int n = count - i0;  // MMAs k < n of this batch are real
        asm volatile(
            "{\n\t.reg .pred pa, pt, g;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 pa, %19, 0;\n\t"
            "setp.eq.b32 pt, 0, 0;\n\t"
            "mov.b64 da, {%1, %17};\n\t mov.b64 db, {%9, %17};\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %18, {%21, %21, %21, %21}, pa;\n\t"
            "setp.gt.s32 g, %20, 1;\n\t mov.b64 da, {%2, %17};\n\t mov.b64 db, {%10, %17};\n\t"
            "@g tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %18, {%21, %21, %21, %21}, pt;\n\t"
            "setp.gt.s32 g, %20, 2;\n\t mov.b64 da, {%3, %17};\n\t mov.b64 db, {%11, %17};\n\t"
            "@g tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %18, {%21, %21, %21, %21}, pt;\n\t"
            "setp.gt.s32 g, %20, 3;\n\t mov.b64 da, {%4, %17};\n\t mov.b64 db, {%12, %17};\n\t"
            "@g tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %18, {%21, %21, %21, %21}, pt;\n\t"
            "setp.gt.s32 g, %20, 4;\n\t mov.b64 da, {%5, %17};\n\t mov.b64 db, {%13, %17};\n\t"
            "@g tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %18, {%21, %21, %21, %21}, pt;\n\t"
            "setp.gt.s32 g, %20, 5;\n\t mov.b64 da, {%6, %17};\n\t mov.b64 db, {%14, %17};\n\t"
            "@g tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %18, {%21, %21, %21, %21}, pt;\n\t"
            "setp.gt.s32 g, %20, 6;\n\t mov.b64 da, {%7, %17};\n\t mov.b64 db, {%15, %17};\n\t"
            "@g tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %18, {%21, %21, %21, %21}, pt;\n\t"
            "setp.gt.s32 g, %20, 7;\n\t mov.b64 da, {%8, %17};\n\t mov.b64 db, {%16, %17};\n\t"
            "@g tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %18, {%21, %21, %21, %21}, pt;\n\t"
            "}"
            :
            : "r"(tmem), "r"(a_lo[0]), "r"(a_lo[1]), "r"(a_lo[2]), "r"(a_lo[3]), "r"(a_lo[4]), "r"(a_lo[5]), "r"(a_lo[6]),
              "r"(a_lo[7]), "r"(b_lo[0]), "r"(b_lo[1]), "r"(b_lo[2]), "r"(b_lo[3]), "r"(b_lo[4]), "r"(b_lo[5]), "r"(b_lo[6]),
              "r"(b_lo[7]), "r"(desc_hi), "r"(idesc), "r"(accumulate), "r"(n), "r"(0u)
            : "memory");
        accumulate = 1;
    }
}

// Threshold as the pixel-row epilogue compares it: acc_raw - pad_corr < thr  <=>  acc_raw - (thr + pad_corr) < 0,
// with thr clamped to +-2^30 (|acc| <= 9 * 32 * 32, so nothing changes) and channels that do not exist
// given the lowest value, which no accumulator is below: their bits are 0.
__device__ __forceinline__ int32_t biased_threshold(const TensorParams &p, bool real_channel, int channel)
{
    const int32_t t = real_channel ? __ldg(p.thr + channel) : INT32_MIN;
    return max(-(1 << 30), min(1 << 30, t)) + p.pad_corr;
}

// Output transform of one tile: thread = TMEM lane = GEMM row; 32 channels per TMEM load.
__device__ __forceinline__ void epilogue(const TensorParams &p, uint32_t tmem_base, int q0, int ch0, const float *sMult,
                                         const float *sBias, const int32_t *sThr, int tid)
{
    const int warp = tid >> 5;
    const int row = (warp & 3) * 32 + (tid & 31);  // a warp can only read the TMEM lanes 32*(warp%4)..+31
    const int q = q0 + row;
    const int rr = q / p.Wp, c = q - rr * p.Wp;
    const int n = rr / p.Hs, oh = rr - n * p.Hs;
    const bool row_ok = q < p.total_q && n < p.N && oh < p.H && c < p.W;
    const int64_t pix = ((int64_t)n * p.H + oh) * p.W + c;
    const uint32_t lane_addr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    // warps 0-3 take the first half of the columns, warps 4-7 the second (whole warps skip together)
    const int half_cols = p.n_blk >= 64 ? p.n_blk / 2 : p.n_blk;
    const int c_begin = (warp >> 2) * half_cols;
    const int c_end = (p.n_blk >= 64 || warp < 4) ? c_begin + half_cols : c_begin;
    for (int c0 = c_begin; c0 < c_end; c0 += 32) {
        int32_t v[32];
        tmem_ld32(lane_addr + (uint32_t)c0, v);
        const int o0 = ch0 + c0;
        if (p.out_type == LCE_OUT_BITPACKED) {
            // sThr holds threshold + pad correction, clamped so that the difference cannot overflow (pad
            // channels: the lowest value, bit 0): the output bit is the sign of raw accumulator - sThr,
            // shifted in from the top; the array is read four channels at a time (c0 is a multiple of 32)
            uint32_t bits = 0u;
#pragma unroll
            for (int j = 28; j >= 0; j -= 4) {
                const int4 t4 = *reinterpret_cast<const int4 *>(sThr + c0 + j);
                bits = __funnelshift_l((uint32_t)(v[j + 3] - t4.w), bits, 1);
                bits = __funnelshift_l((uint32_t)(v[j + 2] - t4.z), bits, 1);
                bits = __funnelshift_l((uint32_t)(v[j + 1] - t4.y), bits, 1);
                bits = __funnelshift_l((uint32_t)(v[j] - t4.x), bits, 1);
            }
            if (row_ok && o0 < p.Cout) static_cast<uint32_t *>(p.out)[pix * p.Cow + (o0 >> 5)] = bits;
            continue;
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] -= p.pad_corr;
        if (p.out_type == LCE_OUT_FLOAT32) {
            float f[32];
            const int32_t floor_v = p.activation == LCE_ACT_RELU ? 0 : INT32_MIN;
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
                // c0 is a multiple of 32: the per-channel arrays are read four floats at a time
                const float4 m4 = *reinterpret_cast<const float4 *>(sMult + c0 + j), b4 = *reinterpret_cast<const float4 *>(sBias + c0 + j);
                f[j] = __fmaf_rn((float)max(v[j], floor_v), m4.x, b4.x);
                f[j + 1] = __fmaf_rn((float)max(v[j + 1], floor_v), m4.y, b4.y);
                f[j + 2] = __fmaf_rn((float)max(v[j + 2], floor_v), m4.z, b4.z);
                f[j + 3] = __fmaf_rn((float)max(v[j + 3], floor_v), m4.w, b4.w);
            }
            if (row_ok) {
                float *dst = static_cast<float *>(p.out) + pix * p.Cout + o0;
                if (p.vec_store == 2 && o0 + 32 <= p.Cout) {
                    // one whole 32-byte sector per lane and instruction
#pragma unroll
                    for (int j = 0; j < 32; j += 8)
                        asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst + j), "f"(f[j]), "f"(f[j + 1]), "f"(f[j + 2]),
                                     "f"(f[j + 3]), "f"(f[j + 4]), "f"(f[j + 5]), "f"(f[j + 6]), "f"(f[j + 7])
                                     : "memory");
                } else if (p.vec_store && o0 + 32 <= p.Cout) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4 *>(dst + j) = make_float4(f[j], f[j + 1], f[j + 2], f[j + 3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (o0 + j < p.Cout) dst[j] = f[j];
                }
            }
        } else if (row_ok) {
            int32_t *dst = static_cast<int32_t *>(p.out) + pix * p.Cout + o0;
            if (p.vec_store && o0 + 32 <= p.Cout) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) *reinterpret_cast<int4 *>(dst + j) = make_int4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (o0 + j < p.Cout) dst[j] = v[j];
            }
        }
    }
}

constexpr int kMaxWordsPerThread = 8;  // streaming schedule: packed weight words of one tap per worker thread

__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Barrier slots in shared memory
enum { BAR_FULL_A0 = 0, BAR_FULL_A1, BAR_FULL_D0, BAR_FULL_D1, BAR_EMPTY_D0, BAR_EMPTY_D1, BAR_FULL_B0, BAR_FULL_B1,
       BAR_EMPTY_B0, BAR_EMPTY_B1, BAR_COUNT };

// Warp-specialised kernel.  Warps 0-7 ("workers", 256 threads) expand operands into shared
// memory and run the output transform; warp 8 does nothing but issue MMAs (one lane).  They
// meet only through mbarriers, never through __syncthreads inside the tile loop:
//   full_a[s]  workers -> issuer : input tile expanded into A buffer s            (256 arrivals)
//   full_b[s]  workers -> issuer : one tap's weights expanded into B buffer s     (256, streaming)
//   empty_b[s] issuer  -> workers: the MMAs that read B buffer s have finished    (tcgen05.commit)
//   full_d[d]  issuer  -> workers: accumulator buffer d is complete               (tcgen05.commit)
//   empty_d[d] workers -> issuer : accumulator buffer d has been read out         (256 arrivals)
// A wait that runs out of iterations makes its thread leave the loop; the others then run out on
// their own waits, everybody reaches the final barrier, TMEM is freed.
template <bool RESIDENT>
__global__ void __launch_bounds__(kThreads, 1)
bconv3x3_tensor_kernel(const TensorParams p)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    // [table 2 KB][barriers + tmem slot, 128 B][per-channel params 3*n_blk words][MMA offsets][raw A 2x][B][A]
    uint2 *table = reinterpret_cast<uint2 *>(smem_raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + 2048);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_raw + 2048 + 96);
    float *sMult = reinterpret_cast<float *>(smem_raw + 2048 + 128);
    float *sBias = sMult + p.n_blk;
    int32_t *sThr = reinterpret_cast<int32_t *>(sBias + p.n_blk);
    uint2 *offs = reinterpret_cast<uint2 *>(sThr + p.n_blk);          // [9*Cw] operand start offsets of a tile's MMAs
    uint32_t *raw0 = reinterpret_cast<uint32_t *>(offs + ((9 * p.Cw + 1) / 2) * 2);
    const int raw_words = ((p.P * p.Cw + 3) / 4) * 4;
    uint8_t *sB = reinterpret_cast<uint8_t *>(raw0 + 2 * raw_words);
    const size_t b_tap_bytes = (size_t)2 * p.Cw * p.n_blk * 16;  // one tap: [2*Cw chunks][n_blk][16]
    uint8_t *sA0 = sB + (RESIDENT ? 9 : 2) * b_tap_bytes;
    const size_t a_bytes = (size_t)2 * p.Cw * p.P * 16;          // [2*Cw chunks][P][16]

    const int tid = threadIdx.x, warp = tid >> 5;
    const bool worker = tid < kWorkers;
    const int ch0 = blockIdx.y * p.n_blk;

    // ---- one-time set-up (all threads) ---------------------------------------------------------
    for (int e = tid; e < 256; e += kThreads) {
        uint32_t lo = 0, hi = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            lo |= (((e >> j) & 1) ? 0xFFu : 0x01u) << (8 * j);
            hi |= (((e >> (j + 4)) & 1) ? 0xFFu : 0x01u) << (8 * j);
        }
        table[e] = make_uint2(lo, hi);
    }
    for (int e = tid; e < p.n_blk; e += kThreads) {
        const bool ok = ch0 + e < p.Cout;
        sMult[e] = (ok && p.out_type == LCE_OUT_FLOAT32) ? __ldg(p.mult + ch0 + e) : 0.f;
        sBias[e] = (ok && p.out_type == LCE_OUT_FLOAT32) ? __ldg(p.bias + ch0 + e) : 0.f;
        sThr[e] = biased_threshold(p, ok && p.out_type == LCE_OUT_BITPACKED, ch0 + e);
    }
    for (int e = tid; e < 9 * p.Cw; e += kThreads) {
        const int tap = e / p.Cw, cw = e - tap * p.Cw;
        // A: window shift of the tap + K step (two planes of P rows); B: K step (two planes of
        // n_blk rows), plus the tap's block when all nine taps are resident.  Units of 16 bytes.
        const uint32_t a_off = (uint32_t)((tap / 3) * p.Wp + (tap % 3) + 2 * cw * p.P);
        const uint32_t b_off = (uint32_t)(2 * cw * p.n_blk) + (RESIDENT ? (uint32_t)(tap * 2 * p.Cw * p.n_blk) : 0u);
        offs[e] = make_uint2(a_off, b_off);
    }
    if (tid == 0) {
        mbar_init(&bars[BAR_FULL_A0], kWorkers);
        mbar_init(&bars[BAR_FULL_A1], kWorkers);
        mbar_init(&bars[BAR_FULL_D0], 1);
        mbar_init(&bars[BAR_FULL_D1], 1);
        mbar_init(&bars[BAR_EMPTY_D0], kWorkers);
        mbar_init(&bars[BAR_EMPTY_D1], kWorkers);
        mbar_init(&bars[BAR_FULL_B0], kWorkers);
        mbar_init(&bars[BAR_FULL_B1], kWorkers);
        mbar_init(&bars[BAR_EMPTY_B0], 1);
        mbar_init(&bars[BAR_EMPTY_B1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    // instruction descriptor: D = S32, A and B signed 8-bit, both K-major, N = n_blk, M = 128
    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_blk >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
    const uint32_t b_saddr = smem_u32(sB);
    // descriptor halves (units of 16 bytes): low = start | plane stride << 16; high = row-group
    // stride (8 = 128 bytes) | version 1 at bit 46
    const uint32_t desc_hi = 8u | (1u << 14);
    const int words_per_tap = p.n_blk * p.Cw;  // packed weight words of one tap of this channel block
    const int first_tile = blockIdx.x, tile_step = gridDim.x;
    bool ok = true;

    if (!worker) {
        // ======================= MMA issuer: one lane of warp 8 ===================================
        if (tid == kWorkers) {
            uint32_t par_full_a[2] = {0, 0}, par_empty_d[2] = {0, 0}, par_full_b[2] = {0, 0};
            int g = 0;  // taps issued so far (streaming: B buffer = g & 1)
            for (int tile = first_tile, it = 0; tile < p.n_tiles && ok; tile += tile_step, ++it) {
                const int ab = RESIDENT ? (it & 1) : 0;  // A buffer
                const int db = RESIDENT ? (it & 1) : 0;  // accumulator buffer
                ok = mbar_wait_bounded(&bars[BAR_FULL_A0 + ab], par_full_a[ab]);
                par_full_a[ab] ^= 1u;
                if (ok && it >= (RESIDENT ? 2 : 1)) {  // the accumulator buffer must have been read out
                    ok = mbar_wait_bounded(&bars[BAR_EMPTY_D0 + db], par_empty_d[db]);
                    par_empty_d[db] ^= 1u;
                }
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmem_d = tmem_base + (uint32_t)(db * p.n_blk);
                const uint32_t a_lo0 = (smem_u32(sA0 + ab * a_bytes) >> 4) | ((uint32_t)p.P << 16);
                uint32_t accumulate = 0;
                if (RESIDENT) {
                    issue_mmas(tmem_d, offs, 0, 9 * p.Cw, a_lo0, (b_saddr >> 4) | ((uint32_t)p.n_blk << 16), desc_hi, idesc, accumulate);
                } else {
                    for (int tap = 0; tap < 9 && ok; ++tap, ++g) {
                        const int sb = g & 1;
                        ok = mbar_wait_bounded(&bars[BAR_FULL_B0 + sb], par_full_b[sb]);
                        par_full_b[sb] ^= 1u;
                        if (!ok) break;
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        issue_mmas(tmem_d, offs, tap * p.Cw, p.Cw, a_lo0,
                                   ((b_saddr + (uint32_t)(sb * b_tap_bytes)) >> 4) | ((uint32_t)p.n_blk << 16), desc_hi, idesc, accumulate);
                        mma_commit(&bars[BAR_EMPTY_B0 + sb]);
                    }
                    if (!ok) break;
                }
                mma_commit(&bars[BAR_FULL_D0 + db]);
            }
        }
    } else {
        // ======================= workers: expansion and output transform ==========================
        uint32_t par_full_d[2] = {0, 0}, par_empty_b[2] = {0, 0};
        int tile = first_tile;
        if (tile < p.n_tiles) prefetch_raw(p, tile * kTileM, raw0, tid);

        if (RESIDENT) {
            // weights: packed [o][tap][cw] -> bytes [tap][chunk][channel][16], once
            for (int e0 = tid; e0 < 9 * words_per_tap; e0 += kWorkers * 8) {
                uint32_t wv[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int e = e0 + k * kWorkers;
                    const int ch = e & (p.n_blk - 1), tc = e >> p.n_blk_log2;  // tc = tap*Cw + cw
                    const int tap = tc / p.Cw, cw = tc - tap * p.Cw;
                    wv[k] = (e < 9 * words_per_tap && ch0 + ch < p.Cout) ? __ldg(p.w + ((int64_t)(ch0 + ch) * 9 + tap) * p.Cw + cw) : 0u;
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int e = e0 + k * kWorkers;
                    if (e < 9 * words_per_tap) {
                        const int ch = e & (p.n_blk - 1), tc = e >> p.n_blk_log2;
                        const int tap = tc / p.Cw, cw = tc - tap * p.Cw;
                        uint4 lo, hi;
                        expand_word(table, wv[k], &lo, &hi);
                        uint4 *dst = reinterpret_cast<uint4 *>(sB + tap * b_tap_bytes) + (size_t)(2 * cw) * p.n_blk + ch;
                        dst[0] = lo;
                        dst[p.n_blk] = hi;
                    }
                }
            }
            if (tile < p.n_tiles) {
                expand_a(p, table, raw0, sA0, tid);
                if (tile + tile_step < p.n_tiles) prefetch_raw(p, (tile + tile_step) * kTileM, raw0 + raw_words, tid);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(&bars[BAR_FULL_A0]);
            }
            for (int it = 0; tile < p.n_tiles && ok; tile += tile_step, ++it) {
                const int next = tile + tile_step;
                const int cur = it & 1, nxt = cur ^ 1;
                if (next < p.n_tiles) {
                    // A buffer nxt was last read by the MMAs of tile it-1, whose completion (full_d)
                    // this thread waited for in the previous iteration
                    expand_a(p, table, raw0 + nxt * raw_words, sA0 + nxt * a_bytes, tid);
                    if (next + tile_step < p.n_tiles) prefetch_raw(p, (next + tile_step) * kTileM, raw0 + cur * raw_words, tid);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    mbar_arrive(&bars[BAR_FULL_A0 + nxt]);
                }
                ok = mbar_wait_bounded(&bars[BAR_FULL_D0 + cur], par_full_d[cur]);
                par_full_d[cur] ^= 1u;
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                epilogue(p, tmem_base + (uint32_t)(cur * p.n_blk), tile * kTileM, ch0, sMult, sBias, sThr, tid);
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                mbar_arrive(&bars[BAR_EMPTY_D0 + cur]);
            }
        } else {
            // A thread expands consecutive channel words of ONE channel (kWorkers / n_blk threads share a
            // channel): its loads of a tap are then one or two whole 32-byte sectors instead of eight
            // words in eight different sectors, and its shared-memory stores stay channel-fastest.
            const int tpc = kWorkers >> p.n_blk_log2;            // threads per channel: 1, 2, 4 or 8
            const int wpt = (p.Cw + tpc - 1) / tpc;              // <= kMaxWordsPerThread (host-checked)
            const int my_ch = tid & (p.n_blk - 1), cw0 = (tid >> p.n_blk_log2) * wpt;
            const bool ch_real = ch0 + my_ch < p.Cout;
            const bool vec_w = (p.Cw & 3) == 0 && (wpt & 3) == 0 && (reinterpret_cast<uintptr_t>(p.w) & 15) == 0;
            int g = 0;  // taps produced so far
            for (int it = 0; tile < p.n_tiles && ok; tile += tile_step, ++it) {
                const int next = tile + tile_step;
                // the single A buffer was last read by the previous tile's MMAs: full_d awaited below
                expand_a(p, table, raw0 + (it & 1) * raw_words, sA0, tid);
                if (next < p.n_tiles) prefetch_raw(p, next * kTileM, raw0 + ((it + 1) & 1) * raw_words, tid);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(&bars[BAR_FULL_A0]);

                uint32_t wv[kMaxWordsPerThread];
                auto load_tap = [&](int tap) {
                    const uint32_t *src = p.w + ((int64_t)(ch0 + (ch_real ? my_ch : 0)) * 9 + tap) * p.Cw + cw0;
                    if (vec_w) {
#pragma unroll
                        for (int k = 0; k < kMaxWordsPerThread; k += 4) {
                            uint4 q = make_uint4(0u, 0u, 0u, 0u);
                            if (ch_real && k < wpt && cw0 + k < p.Cw) q = __ldg(reinterpret_cast<const uint4 *>(src + k));
                            wv[k] = q.x; wv[k + 1] = q.y; wv[k + 2] = q.z; wv[k + 3] = q.w;
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < kMaxWordsPerThread; ++k)
                            wv[k] = (ch_real && k < wpt && cw0 + k < p.Cw) ? __ldg(src + k) : 0u;
                    }
                };
                load_tap(0);
                for (int tap = 0; tap < 9 && ok; ++tap, ++g) {
                    const int sb = g & 1;
                    if (g >= 2) {  // the MMAs of two taps ago read this B buffer
                        ok = mbar_wait_bounded(&bars[BAR_EMPTY_B0 + sb], par_empty_b[sb]);
                        par_empty_b[sb] ^= 1u;
                        if (!ok) break;
                    }
                    uint8_t *dstB = sB + sb * b_tap_bytes;
#pragma unroll
                    for (int k = 0; k < kMaxWordsPerThread; ++k) {
                        if (k < wpt && cw0 + k < p.Cw) {
                            const int ch = my_ch, cw = cw0 + k;
                            uint4 lo, hi;
                            expand_word_alu(wv[k], &lo, &hi);
                            uint4 *dst = reinterpret_cast<uint4 *>(dstB) + (size_t)(2 * cw) * p.n_blk + ch;
                            dst[0] = lo;
                            dst[p.n_blk] = hi;
                        }
                    }
                    if (tap + 1 < 9) load_tap(tap + 1);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    mbar_arrive(&bars[BAR_FULL_B0 + sb]);
                }
                if (!ok) break;
                ok = mbar_wait_bounded(&bars[BAR_FULL_D0], par_full_d[0]);
                par_full_d[0] ^= 1u;
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                epilogue(p, tmem_base, tile * kTileM, ch0, sMult, sBias, sThr, tid);
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                mbar_arrive(&bars[BAR_EMPTY_D0]);
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    if (!ok) g_tensor_status = 1;

    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}


// RESIDENT schedule with the worker roles split over two warp groups, so that the expansion of
// tile t+1, the MMAs of tile t and the output transform of tile t-1 run at the same time (a kernel
// that allocates TMEM is given one CTA per SM, so the overlap has to come from inside the CTA):
// warps 0-7 "loaders" (prefetch + expand the input tile), warps 8-15 "finishers" (read the
// accumulators, output transform), warp 16 issues MMAs.  Barriers as above; full_d[s] is awaited by
// both groups (the loaders reuse A buffer s only after the MMAs that read it are done).
constexpr int kSplitThreads = 2 * kWorkers + 32;

__global__ void __launch_bounds__(kSplitThreads, 1)
bconv3x3_tensor_split_kernel(const TensorParams p)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    uint2 *table = reinterpret_cast<uint2 *>(smem_raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + 2048);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_raw + 2048 + 96);
    float *sMult = reinterpret_cast<float *>(smem_raw + 2048 + 128);
    float *sBias = sMult + p.n_blk;
    int32_t *sThr = reinterpret_cast<int32_t *>(sBias + p.n_blk);
    uint2 *offs = reinterpret_cast<uint2 *>(sThr + p.n_blk);
    uint32_t *raw0 = reinterpret_cast<uint32_t *>(offs + ((9 * p.Cw + 1) / 2) * 2);
    const int raw_words = ((p.P * p.Cw + 3) / 4) * 4;
    uint8_t *sB = reinterpret_cast<uint8_t *>(raw0 + 2 * raw_words);
    const size_t b_tap_bytes = (size_t)2 * p.Cw * p.n_blk * 16;
    uint8_t *sA0 = sB + 9 * b_tap_bytes;
    const size_t a_bytes = (size_t)2 * p.Cw * p.P * 16;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int ch0 = blockIdx.y * p.n_blk;

    for (int e = tid; e < 256; e += kSplitThreads) {
        uint32_t lo = 0, hi = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            lo |= (((e >> j) & 1) ? 0xFFu : 0x01u) << (8 * j);
            hi |= (((e >> (j + 4)) & 1) ? 0xFFu : 0x01u) << (8 * j);
        }
        table[e] = make_uint2(lo, hi);
    }
    for (int e = tid; e < p.n_blk; e += kSplitThreads) {
        const bool ok = ch0 + e < p.Cout;
        sMult[e] = (ok && p.out_type == LCE_OUT_FLOAT32) ? __ldg(p.mult + ch0 + e) : 0.f;
        sBias[e] = (ok && p.out_type == LCE_OUT_FLOAT32) ? __ldg(p.bias + ch0 + e) : 0.f;
        sThr[e] = biased_threshold(p, ok && p.out_type == LCE_OUT_BITPACKED, ch0 + e);
    }
    for (int e = tid; e < 9 * p.Cw; e += kSplitThreads) {
        const int tap = e / p.Cw, cw = e - tap * p.Cw;
        const uint32_t a_off = (uint32_t)((tap / 3) * p.Wp + (tap % 3) + 2 * cw * p.P);
        const uint32_t b_off = (uint32_t)(2 * cw * p.n_blk) + (uint32_t)(tap * 2 * p.Cw * p.n_blk);
        offs[e] = make_uint2(a_off, b_off);
    }
    if (tid == 0) {
        mbar_init(&bars[BAR_FULL_A0], kWorkers);
        mbar_init(&bars[BAR_FULL_A1], kWorkers);
        mbar_init(&bars[BAR_FULL_D0], 1);
        mbar_init(&bars[BAR_FULL_D1], 1);
        mbar_init(&bars[BAR_EMPTY_D0], kWorkers);
        mbar_init(&bars[BAR_EMPTY_D1], kWorkers);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_blk >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
    const uint32_t b_saddr = smem_u32(sB);
    const uint32_t desc_hi = 8u | (1u << 14);
    const int words_per_tap = p.n_blk * p.Cw;
    const int first_tile = blockIdx.x, tile_step = gridDim.x;
    bool ok = true;

    if (tid >= 2 * kWorkers) {
        // ---- MMA issuer: one lane -------------------------------------------------------------
        if (tid == 2 * kWorkers) {
            uint32_t par_full_a[2] = {0, 0}, par_empty_d[2] = {0, 0};
            for (int tile = first_tile, it = 0; tile < p.n_tiles && ok; tile += tile_step, ++it) {
                const int sbuf = it & 1;
                ok = mbar_wait_bounded(&bars[BAR_FULL_A0 + sbuf], par_full_a[sbuf]);
                par_full_a[sbuf] ^= 1u;
                if (ok && it >= 2) {  // the accumulator buffer must have been read out
                    ok = mbar_wait_bounded(&bars[BAR_EMPTY_D0 + sbuf], par_empty_d[sbuf]);
                    par_empty_d[sbuf] ^= 1u;
                }
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmem_d = tmem_base + (uint32_t)(sbuf * p.n_blk);
                const uint32_t a_lo0 = (smem_u32(sA0 + sbuf * a_bytes) >> 4) | ((uint32_t)p.P << 16);
                uint32_t accumulate = 0;
                issue_mmas(tmem_d, offs, 0, 9 * p.Cw, a_lo0, (b_saddr >> 4) | ((uint32_t)p.n_blk << 16), desc_hi, idesc, accumulate);
                mma_commit(&bars[BAR_FULL_D0 + sbuf]);
            }
        }
    } else {
        // ---- both worker groups expand the resident weights, then part ways ----------------------
        if (tid < kWorkers && first_tile < p.n_tiles) prefetch_raw(p, first_tile * kTileM, raw0, tid);
        const bool quads = (p.Cw & 3) == 0 && (reinterpret_cast<uintptr_t>(p.w) & 15) == 0;
        if (quads) {
            // Four consecutive channel words of one channel per 128-bit load (channel-fastest over the
            // lanes, so the shared-memory stores stay conflict-free): a quarter of the load requests of
            // the word-by-word form, which kept the load unit busy for most of the set-up time.  Half of
            // the words go through the look-up table and half through the integer pipes, which work
            // side by side.
            const int units = 9 * words_per_tap / 4;  // (channel, quad) pairs; a quad lies inside one tap
            for (int u0 = tid; u0 < units; u0 += 2 * kWorkers * 2) {
                uint4 q[2];
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const int u = u0 + k * 2 * kWorkers;
                    const int ch = u & (p.n_blk - 1), tc = (u >> p.n_blk_log2) * 4;
                    q[k] = (u < units && ch0 + ch < p.Cout) ? __ldg(reinterpret_cast<const uint4 *>(p.w + (int64_t)(ch0 + ch) * 9 * p.Cw + tc))
                                                            : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const int u = u0 + k * 2 * kWorkers;
                    if (u < units) {
                        const int ch = u & (p.n_blk - 1), tc = (u >> p.n_blk_log2) * 4;
                        const int tap = tc / p.Cw, cw = tc - tap * p.Cw;
                        const uint32_t wq[4] = {q[k].x, q[k].y, q[k].z, q[k].w};
                        uint4 *dst = reinterpret_cast<uint4 *>(sB + tap * b_tap_bytes) + (size_t)(2 * cw) * p.n_blk + ch;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint4 lo, hi;
                            if (i & 1) expand_word(table, wq[i], &lo, &hi);
                            else expand_word_alu(wq[i], &lo, &hi);
                            dst[(size_t)(2 * i) * p.n_blk] = lo;
                            dst[(size_t)(2 * i + 1) * p.n_blk] = hi;
                        }
                    }
                }
            }
        }
        for (int e0 = tid; !quads && e0 < 9 * words_per_tap; e0 += 2 * kWorkers * 8) {
            uint32_t wv[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int e = e0 + k * 2 * kWorkers;
                const int ch = e & (p.n_blk - 1), tc = e >> p.n_blk_log2;  // tc = tap*Cw + cw
                const int tap = tc / p.Cw, cw = tc - tap * p.Cw;
                wv[k] = (e < 9 * words_per_tap && ch0 + ch < p.Cout) ? __ldg(p.w + ((int64_t)(ch0 + ch) * 9 + tap) * p.Cw + cw) : 0u;
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int e = e0 + k * 2 * kWorkers;
                if (e < 9 * words_per_tap) {
                    const int ch = e & (p.n_blk - 1), tc = e >> p.n_blk_log2;
                    const int tap = tc / p.Cw, cw = tc - tap * p.Cw;
                    uint4 lo, hi;
                    expand_word(table, wv[k], &lo, &hi);
                    uint4 *dst = reinterpret_cast<uint4 *>(sB + tap * b_tap_bytes) + (size_t)(2 * cw) * p.n_blk + ch;
                    dst[0] = lo;
                    dst[p.n_blk] = hi;
                }
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("bar.sync 1, %0;" ::"n"(2 * kWorkers) : "memory");  // weights complete before any full_a arrival

        uint32_t par_full_d[2] = {0, 0};
        if (tid < kWorkers) {
            // ---- loaders ---------------------------------------------------------------------------
            int tile = first_tile;
            for (int it = 0; tile < p.n_tiles && ok; tile += tile_step, ++it) {
                const int sbuf = it & 1;
                if (it >= 2) {  // A buffer sbuf was read by the MMAs of tile it-2
                    ok = mbar_wait_bounded(&bars[BAR_FULL_D0 + sbuf], par_full_d[sbuf]);
                    par_full_d[sbuf] ^= 1u;
                    if (!ok) break;
                }
                expand_a(p, table, raw0 + sbuf * raw_words, sA0 + sbuf * a_bytes, tid);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(&bars[BAR_FULL_A0 + sbuf]);
                // only now the words of the next tile: every thread reads back just its own copies, and
                // the MMAs of this tile must not wait for loads they do not need
                const int next = tile + tile_step;
                if (next < p.n_tiles) prefetch_raw(p, next * kTileM, raw0 + (sbuf ^ 1) * raw_words, tid);
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        } else {
            // ---- finishers -------------------------------------------------------------------------
            const int ftid = tid - kWorkers;
            int tile = first_tile;
            for (int it = 0; tile < p.n_tiles && ok; tile += tile_step, ++it) {
                const int sbuf = it & 1;
                ok = mbar_wait_bounded(&bars[BAR_FULL_D0 + sbuf], par_full_d[sbuf]);
                par_full_d[sbuf] ^= 1u;
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                epilogue(p, tmem_base + (uint32_t)(sbuf * p.n_blk), tile * kTileM, ch0, sMult, sBias, sThr, ftid);
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                mbar_arrive(&bars[BAR_EMPTY_D0 + sbuf]);
            }
        }
    }
    if (!ok) g_tensor_status = 1;

    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}


// ---- pixels as the N dimension ---------------------------------------------------------------------
// An i8 MMA streams (M + N) * 32 bytes of operands from shared memory for M * N * 32 products, so a
// layer with few output channels is better served with the operands swapped: D[channel][pixel] =
// W[channel][k] x X[pixel][k]^T, M = 128 channel rows (channels past Cout are zero words = +1 bytes,
// their lanes are ignored), N = 256 pixels per MMA: four times the work per instruction of the M =
// 128 pixels x N = 64 channels form for 1.5 times the operand bytes.  The shifted window now applies
// to the B operand (same [chunk][position][16 bytes] buffer, same descriptors with N = 256).  A TMEM
// lane is a channel and a column a pixel, which suits bit-packed output (a lane's 32 compare bits,
// then a 32 x 32 bit transpose across the warp gives every lane the finished word of one pixel);
// float and int32 output of up to 64 channels go through a shared-memory stage (see
// epilogue_swapped_staged), wider ones stay with the pixel-row form.  Roles and barriers as in the split kernel, with 16 loader warps.
constexpr int kTileN = 256;
constexpr int kSwLoaders = 512;                                  // 16 loader warps: one position per thread for P <= 512
constexpr int kSwThreads = kSwLoaders + kWorkers + 32;           // + 8 finisher warps + the issuer warp

__device__ __forceinline__ void epilogue_swapped(const TensorParams &p, uint32_t tmem_d, const int32_t *sPix, int ch0,
                                                 const int32_t *sThr, int ftid)
{
    const int warp = ftid >> 5, lane = ftid & 31;
    const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31 = channels of this warp
    if (ch0 + quarter * 32 >= p.Cout) return;     // whole warp: no real channel in its lanes
    const int32_t thr = sThr[quarter * 32 + lane];  // INT32_MIN for pad channels: bit 0
    // acc - pad_corr < thr  <=>  acc - (thr + pad_corr) < 0; the threshold is clamped to +-2^30 so that
    // the subtraction cannot overflow (|acc| <= 9 * 32 * 32 here)
    const int32_t thr_biased = max(-(1 << 30), min(1 << 30, thr > (1 << 30) ? (1 << 30) : thr + p.pad_corr));
    const uint32_t lane_addr = tmem_d + ((uint32_t)(quarter * 32) << 16);
    const int c_begin = (warp >> 2) * (kTileN / 2);
    for (int c0 = c_begin; c0 < c_begin + kTileN / 2; c0 += 32) {
        int32_t v[32];
        tmem_ld32(lane_addr + (uint32_t)c0, v);
        const int my_pix = sPix[c0 + lane];       // output pixel of column c0 + lane, or -1
        // this lane's channel against the 32 pixels of the chunk, bit j = pixel c0 + j (the sign bit
        // of acc - threshold, shifted in from the top: two chains of 16) ...
        uint32_t m_lo = 0u, m_hi = 0u;
#pragma unroll
        for (int j = 15; j >= 0; --j) {
            m_lo = __funnelshift_l((uint32_t)(v[j] - thr_biased), m_lo, 1);
            m_hi = __funnelshift_l((uint32_t)(v[16 + j] - thr_biased), m_hi, 1);
        }
        uint32_t m = m_lo | (m_hi << 16);
        // ... then a 32 x 32 bit transpose across the warp (five butterfly steps), after which lane j
        // holds the output word of pixel c0 + j: bit i = channel 32*quarter + i
#pragma unroll
        for (int k = 16; k >= 1; k >>= 1) {
            const uint32_t keep = k == 16 ? 0x0000FFFFu : k == 8 ? 0x00FF00FFu : k == 4 ? 0x0F0F0F0Fu : k == 2 ? 0x33333333u : 0x55555555u;
            const uint32_t y = __shfl_xor_sync(0xffffffffu, m, k);
            m = (lane & k) ? (((y >> k) & keep) | (m & ~keep)) : ((m & keep) | ((y & keep) << k));
        }
        if (my_pix >= 0) static_cast<uint32_t *>(p.out)[(int64_t)my_pix * p.Cow + ((ch0 >> 5) + quarter)] = m;
    }
}

// Float / int32 output of the pixels-as-N kernel (Cout <= 64): a lane holds ONE channel of 32 pixels, the
// output wants 64 consecutive channels per pixel.  The values go through a shared-memory stage
// [256 pixels][64 channels]: the warps that own real channels write it (lanes = consecutive channels:
// no bank conflicts; the multiplier and bias of a lane's channel sit in two registers), all eight
// finisher warps then copy whole pixel rows out with 16-byte accesses, two rows per instruction.
// Two named-barrier phases per tile (256 finisher threads): stage complete / stage free again.
constexpr int kStageCh = 64;
__device__ __forceinline__ void epilogue_swapped_staged(const TensorParams &p, uint32_t tmem_d, const int32_t *sPix, int ch0,
                                                        uint32_t *stage, float mult, float bias, int ftid, uint64_t *empty_d)
{
    const int warp = ftid >> 5, lane = ftid & 31;
    const int quarter = warp & 3;
    if (ch0 + quarter * 32 < p.Cout) {
        const uint32_t lane_addr = tmem_d + ((uint32_t)(quarter * 32) << 16);
        const int c_begin = (warp >> 2) * (kTileN / 2);
        const bool relu = p.activation == LCE_ACT_RELU;
        uint32_t *col = stage + quarter * 32 + lane;
        for (int c0 = c_begin; c0 < c_begin + kTileN / 2; c0 += 32) {
            int32_t v[32];
            tmem_ld32(lane_addr + (uint32_t)c0, v);
            if (p.out_type == LCE_OUT_FLOAT32) {
                // int -> float without the conversion unit (the active finisher warps share two of the four
                // SM sub-partitions): v + 0x4B400000 is the bit pattern of 12582912 + v for |v| < 2^22, so one
                // exact FADD gives (float)v; ReLU is a max against the same constant
                const int32_t add = 0x4B400000 - p.pad_corr;
                if (relu) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        col[(c0 + j) * kStageCh] = __float_as_uint(
                            __fmaf_rn(__fadd_rn(__int_as_float(max(v[j] + add, 0x4B400000)), -12582912.0f), mult, bias));
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        col[(c0 + j) * kStageCh] = __float_as_uint(__fmaf_rn(__fadd_rn(__int_as_float(v[j] + add), -12582912.0f), mult, bias));
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) col[(c0 + j) * kStageCh] = (uint32_t)(v[j] - p.pad_corr);
            }
        }
    }
    // the accumulator buffer has been read: hand it back before the copy out
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    mbar_arrive(empty_d);
    if (p.Cout == kStageCh) {
        // A stage row is an output row: runs of consecutive valid columns are contiguous in both, so the
        // copy engine moves them (one bulk copy per run, at most 32 columns = 8 KB) while the warps go
        // on to the next tile.  The caller waits for the reads of the stage before it is written again.
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("bar.sync 2, %0;" ::"n"(kWorkers) : "memory");  // the stage holds the whole tile
        const int col_px = warp * 32 + lane;
        const int pix = sPix[col_px];
        const int prev = __shfl_up_sync(0xffffffffu, pix, 1);
        const bool valid = pix >= 0;
        const bool start = valid && (lane == 0 || prev < 0 || prev + 1 != pix);
        const uint32_t stops = ~__ballot_sync(0xffffffffu, valid) | __ballot_sync(0xffffffffu, start);  // a run ends before these lanes
        if (start) {
            const uint32_t later = lane == 31 ? 0u : (stops >> (lane + 1));
            const int len = later == 0u ? 32 - lane : 1 + __ffs(later) - 1;  // columns lane .. lane+len-1
            const uint32_t src = smem_u32(stage + col_px * kStageCh);
            uint32_t *dst = static_cast<uint32_t *>(p.out) + (int64_t)pix * kStageCh;
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"((uint32_t)(len * kStageCh * 4))
                         : "memory");
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        return;
    }
    asm volatile("bar.sync 2, %0;" ::"n"(kWorkers) : "memory");  // the stage holds the whole tile
    // rows out: warp w takes pixels 32w .. 32w+31; a row of Cout values is Cout/4 16-byte pieces
    const int pieces = p.Cout >> 2;                       // 1 .. 16 (Cout is a multiple of 4 here)
    const int rows_per_inst = 32 / pieces >= 2 ? 2 : 1;   // Cout <= 32: still two rows per instruction
    const int sub = lane / pieces, piece = lane - sub * pieces;
    if (sub < rows_per_inst) {
        // four rows in flight per lane: the loads do not wait for one another's stores
        for (int r = 0; r < 32; r += 4 * rows_per_inst) {
            int pix[4];
            uint4 q[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int col_px = warp * 32 + r + u * rows_per_inst + sub;  // rows_per_inst divides 8: stays inside the warp's 32
                pix[u] = sPix[col_px];
                q[u] = *reinterpret_cast<const uint4 *>(stage + col_px * kStageCh + piece * 4);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (pix[u] >= 0) *reinterpret_cast<uint4 *>(static_cast<uint32_t *>(p.out) + (int64_t)pix[u] * p.Cout + piece * 4) = q[u];
        }
    }
    asm volatile("bar.sync 2, %0;" ::"n"(kWorkers) : "memory");  // everybody has read the stage
}

__global__ void __launch_bounds__(kSwThreads, 1)
bconv3x3_tensor_swapped_kernel(const TensorParams p)  // p.P, p.n_tiles are for tiles of kTileN positions; p.n_blk = 128
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    uint2 *table = reinterpret_cast<uint2 *>(smem_raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + 2048);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_raw + 2048 + 96);
    int32_t *sThr = reinterpret_cast<int32_t *>(smem_raw + 2048 + 128);
    // [4][kTileN] output pixel of a column, or -1.  A ring of four: the loaders of tile t+2 must not wait
    // for the finishers of tile t (that would chain the three roles one after the other); slot t&3 is
    // rewritten for tile t+4, whose X buffer is free only after the MMAs of tile t+2, which wait for
    // the finishers of tile t.
    int32_t *sPix = sThr + 128;
    uint2 *offs = reinterpret_cast<uint2 *>(sPix + 4 * kTileN);         // [9*Cw] operand start offsets of a tile's MMAs
    uint32_t *raw0 = reinterpret_cast<uint32_t *>(offs + ((9 * p.Cw + 1) / 2) * 2);
    const int raw_words = ((p.P * p.Cw + 3) / 4) * 4;
    uint8_t *sW = reinterpret_cast<uint8_t *>(raw0 + 2 * raw_words);    // A operand: [tap][2*Cw chunks][128 channels][16]
    const size_t w_tap_bytes = (size_t)2 * p.Cw * 128 * 16;
    uint8_t *sX0 = sW + 9 * w_tap_bytes;                                // B operand: 2 x [2*Cw chunks][P positions][16]
    const size_t x_bytes = (size_t)2 * p.Cw * p.P * 16;
    uint32_t *stage = reinterpret_cast<uint32_t *>(sX0 + 2 * x_bytes);  // float / int32 output only: [kTileN][kStageCh]

    const int tid = threadIdx.x, warp = tid >> 5;
    const int ch0 = blockIdx.y * 128;

    for (int e = tid; e < 256; e += kSwThreads) {
        uint32_t lo = 0, hi = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            lo |= (((e >> j) & 1) ? 0xFFu : 0x01u) << (8 * j);
            hi |= (((e >> (j + 4)) & 1) ? 0xFFu : 0x01u) << (8 * j);
        }
        table[e] = make_uint2(lo, hi);
    }
    for (int e = tid; e < 128; e += kSwThreads) {
        sThr[e] = (p.out_type == LCE_OUT_BITPACKED && ch0 + e < p.Cout) ? __ldg(p.thr + ch0 + e) : INT32_MIN;
    }
    for (int e = tid; e < 9 * p.Cw; e += kSwThreads) {
        const int tap = e / p.Cw, cw = e - tap * p.Cw;
        // A (weights): the tap's block + K step (two planes of 128 rows); B (positions): window shift of
        // the tap + K step (two planes of P rows).  Units of 16 bytes.
        const uint32_t a_off = (uint32_t)(tap * 2 * p.Cw * 128 + 2 * cw * 128);
        const uint32_t b_off = (uint32_t)((tap / 3) * p.Wp + (tap % 3) + 2 * cw * p.P);
        offs[e] = make_uint2(a_off, b_off);
    }
    if (tid == 0) {
        mbar_init(&bars[BAR_FULL_A0], kSwLoaders);   // here: positions expanded into X buffer 0 / 1
        mbar_init(&bars[BAR_FULL_A1], kSwLoaders);
        mbar_init(&bars[BAR_FULL_D0], 1);
        mbar_init(&bars[BAR_FULL_D1], 1);
        mbar_init(&bars[BAR_EMPTY_D0], kWorkers);
        mbar_init(&bars[BAR_EMPTY_D1], kWorkers);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    // instruction descriptor: D = S32, A and B signed 8-bit, both K-major, N = 256, M = 128
    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTileN >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    const uint32_t desc_hi = 8u | (1u << 14);
    const int first_tile = blockIdx.x, tile_step = gridDim.x;
    bool ok = true;

    if (tid >= kSwLoaders + kWorkers) {
        if (tid == kSwLoaders + kWorkers) {
            uint32_t par_full_x[2] = {0, 0}, par_empty_d[2] = {0, 0};
            const uint32_t a_lo0 = (smem_u32(sW) >> 4) | (128u << 16);
            for (int tile = first_tile, it = 0; tile < p.n_tiles && ok; tile += tile_step, ++it) {
                const int sbuf = it & 1;
                ok = mbar_wait_bounded(&bars[BAR_FULL_A0 + sbuf], par_full_x[sbuf]);
                par_full_x[sbuf] ^= 1u;
                if (ok && it >= 2) {
                    ok = mbar_wait_bounded(&bars[BAR_EMPTY_D0 + sbuf], par_empty_d[sbuf]);
                    par_empty_d[sbuf] ^= 1u;
                }
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmem_d = tmem_base + (uint32_t)(sbuf * kTileN);
                const uint32_t b_lo0 = (smem_u32(sX0 + sbuf * x_bytes) >> 4) | ((uint32_t)p.P << 16);
                uint32_t accumulate = 0;
                issue_mmas(tmem_d, offs, 0, 9 * p.Cw, a_lo0, b_lo0, desc_hi, idesc, accumulate);
                mma_commit(&bars[BAR_FULL_D0 + sbuf]);
            }
        }
    } else {
        if (tid < kSwLoaders && first_tile < p.n_tiles) prefetch_raw<kSwLoaders>(p, first_tile * kTileN, raw0, tid);
        // weights of this channel block, once: packed [o][tap][cw] -> bytes [tap][chunk][channel][16]
        const int words = 9 * 128 * p.Cw;
        const bool pairs = (p.Cw & 1) == 0 && (reinterpret_cast<uintptr_t>(p.w) & 7) == 0;
        if (pairs) {
            // two consecutive channel words per 64-bit load, channel-fastest over the lanes: half the load
            // requests; one word of a pair is expanded through the table, the other on the integer pipes
            const int units = words / 2;  // (channel, pair) pairs; a pair lies inside one tap
            for (int u0 = tid; u0 < units; u0 += (kSwLoaders + kWorkers) * 4) {
                uint2 q[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int u = u0 + k * (kSwLoaders + kWorkers);
                    const int ch = u & 127, tc = (u >> 7) * 2;
                    q[k] = (u < units && ch0 + ch < p.Cout) ? __ldg(reinterpret_cast<const uint2 *>(p.w + (int64_t)(ch0 + ch) * 9 * p.Cw + tc))
                                                            : make_uint2(0u, 0u);
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int u = u0 + k * (kSwLoaders + kWorkers);
                    if (u < units) {
                        const int ch = u & 127, tc = (u >> 7) * 2;
                        const int tap = tc / p.Cw, cw = tc - tap * p.Cw;
                        uint4 *dst = reinterpret_cast<uint4 *>(sW + tap * w_tap_bytes) + (size_t)(2 * cw) * 128 + ch;
                        uint4 lo, hi;
                        expand_word(table, q[k].x, &lo, &hi);
                        dst[0] = lo;
                        dst[128] = hi;
                        expand_word_alu(q[k].y, &lo, &hi);
                        dst[256] = lo;
                        dst[384] = hi;
                    }
                }
            }
        }
        for (int e0 = tid; !pairs && e0 < words; e0 += (kSwLoaders + kWorkers) * 8) {
            uint32_t wv[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int e = e0 + k * (kSwLoaders + kWorkers);
                const int ch = e & 127, tc = e >> 7;  // tc = tap*Cw + cw
                const int tap = tc / p.Cw, cw = tc - tap * p.Cw;
                wv[k] = (e < words && ch0 + ch < p.Cout) ? __ldg(p.w + ((int64_t)(ch0 + ch) * 9 + tap) * p.Cw + cw) : 0u;
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int e = e0 + k * (kSwLoaders + kWorkers);
                if (e < words) {
                    const int ch = e & 127, tc = e >> 7;
                    const int tap = tc / p.Cw, cw = tc - tap * p.Cw;
                    uint4 lo, hi;
                    expand_word(table, wv[k], &lo, &hi);
                    uint4 *dst = reinterpret_cast<uint4 *>(sW + tap * w_tap_bytes) + (size_t)(2 * cw) * 128 + ch;
                    dst[0] = lo;
                    dst[128] = hi;
                }
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("bar.sync 1, %0;" ::"n"(kSwLoaders + kWorkers) : "memory");

        uint32_t par_full_d[2] = {0, 0};
        if (tid < kSwLoaders) {
            // ---- loaders: expand the positions of a tile, note which output pixel each column is ------
            int tile = first_tile;
            for (int it = 0; tile < p.n_tiles && ok; tile += tile_step, ++it) {
                const int sbuf = it & 1;
                if (it >= 2) {  // X buffer sbuf was read by the MMAs of tile it-2
                    ok = mbar_wait_bounded(&bars[BAR_FULL_D0 + sbuf], par_full_d[sbuf]);
                    par_full_d[sbuf] ^= 1u;
                    if (!ok) break;
                }
                expand_a<kSwLoaders, false>(p, table, raw0 + sbuf * raw_words, sX0 + sbuf * x_bytes, tid);
                if (tid < kTileN) {
                    const int q = tile * kTileN + tid;  // one column per thread of the first eight loader warps
                    const int rr = q / p.Wp, c = q - rr * p.Wp;
                    const int n = rr / p.Hs, oh = rr - n * p.Hs;
                    const bool col_ok = q < p.total_q && n < p.N && oh < p.H && c < p.W;
                    sPix[(it & 3) * kTileN + tid] = col_ok ? (n * p.H + oh) * p.W + c : -1;
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(&bars[BAR_FULL_A0 + sbuf]);
                const int next = tile + tile_step;
                if (next < p.n_tiles) prefetch_raw<kSwLoaders>(p, next * kTileN, raw0 + (sbuf ^ 1) * raw_words, tid);
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        } else {
            // ---- finishers -------------------------------------------------------------------------------
            const int ftid = tid - kSwLoaders;
            const bool staged = p.out_type != LCE_OUT_BITPACKED;
            const int my_channel = ch0 + ((ftid >> 5) & 3) * 32 + (ftid & 31);
            const bool has_params = p.out_type == LCE_OUT_FLOAT32 && my_channel < p.Cout;
            const float my_mult = has_params ? __ldg(p.mult + my_channel) : 0.f, my_bias = has_params ? __ldg(p.bias + my_channel) : 0.f;
            int tile = first_tile;
            for (int it = 0; tile < p.n_tiles && ok; tile += tile_step, ++it) {
                const int sbuf = it & 1;
                ok = mbar_wait_bounded(&bars[BAR_FULL_D0 + sbuf], par_full_d[sbuf]);
                par_full_d[sbuf] ^= 1u;
                if (staged) {
                    // the staged form synchronises the finisher warps among themselves: they go on only
                    // if the wait succeeded in every one of them
                    uint32_t all_ok;
                    asm volatile("{\n\t.reg .pred q, r;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred r, 3, %2, q;\n\tselp.u32 %0, 1, 0, r;\n\t}"
                                 : "=r"(all_ok)
                                 : "r"((uint32_t)ok), "n"(kWorkers)
                                 : "memory");
                    ok = all_ok != 0;
                }
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (staged && p.Cout == kStageCh && it > 0) {
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // this thread's copies have read the stage
                    asm volatile("bar.sync 2, %0;" ::"n"(kWorkers) : "memory");     // ... and so have everybody's
                }
                if (staged) {
                    epilogue_swapped_staged(p, tmem_base + (uint32_t)(sbuf * kTileN), sPix + (it & 3) * kTileN, ch0, stage, my_mult, my_bias,
                                            ftid, &bars[BAR_EMPTY_D0 + sbuf]);
                } else {
                    epilogue_swapped(p, tmem_base + (uint32_t)(sbuf * kTileN), sPix + (it & 3) * kTileN, ch0, sThr, ftid);
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    mbar_arrive(&bars[BAR_EMPTY_D0 + sbuf]);
                }
            }
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // staged form: the last tile's copies are complete
        }
    }
    if (!ok) g_tensor_status = 1;

    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

}  // namespace

bool tensor_covers(const ConvGeom &g)
{
    return g.KH == 3 && g.KW == 3 && g.sh == 1 && g.sw == 1 && g.padding == LCE_PAD_SAME_ONE && g.Cw <= 32 &&
           (int64_t)g.N * (g.H + 1) * (g.W + 1) < (1ll << 31) - 4096;
}

lce_status launch_bconv_tensor(const ConvGeom &g, const uint32_t *in, const uint32_t *w, const float *mult,
                               const float *bias, const int32_t *thr, void *out, cudaStream_t s)
{
    if (!tensor_covers(g)) return LCE_ERR_UNSUPPORTED;
    TensorParams p{};
    p.in = in; p.w = w; p.mult = mult; p.bias = bias; p.thr = thr; p.out = out;
    p.N = g.N; p.H = g.H; p.W = g.W; p.Cin = g.Cin; p.Cw = g.Cw; p.Cout = g.Cout; p.Cow = g.Cow;
    p.Wp = g.W + 1; p.Hs = g.H + 1;
    p.P = kTileM + 2 * p.Wp + 2;
    p.total_q = g.N * p.Hs * p.Wp;
    p.n_tiles = (p.total_q + kTileM - 1) / kTileM;
    p.pad_corr = 9 * (32 * g.Cw - g.Cin);
    p.out_type = g.out_type; p.activation = g.activation;
    p.vec_store = ((g.Cout & 7) == 0 && aligned(out, 32)) ? 2 : ((g.Cout & 3) == 0 && aligned(out, 16)) ? 1 : 0;
    if (p.P > 16383) return LCE_ERR_UNSUPPORTED;  // descriptor offsets are 14-bit counts of 16 bytes

    // Bit-packed output with few output channels: pixels as the N dimension (M = 128 channel rows, N =
    // 256 pixels per MMA), when the resident weights of a 128-channel block and two position buffers fit.
    {
        TensorParams q = p;
        q.P = kTileN + 2 * p.Wp + 2;
        q.n_tiles = (p.total_q + kTileN - 1) / kTileN;
        q.n_blk = 128;
        q.n_blk_log2 = 7;
        q.tmem_cols = 512;
        const size_t raw_b = (size_t)2 * (((size_t)q.P * g.Cw + 3) / 4) * 16;
        size_t need = (size_t)2048 + 128 + 128 * 4 + 4 * kTileN * 4 + 8 * (size_t)(((9 * g.Cw + 1) / 2) * 2) + raw_b +
                            9 * (size_t)2 * g.Cw * 128 * 16 + 2 * (size_t)2 * g.Cw * q.P * 16;
        // float / int32 output goes through a [256][64] stage in shared memory: Cout <= 64, 16-byte rows
        const bool staged = g.out_type != LCE_OUT_BITPACKED;
        if (staged) need += (size_t)kTileN * kStageCh * 4;
        bool swapped = (staged ? (g.Cout <= kStageCh && p.vec_store != 0) : g.Cout <= 128) && need <= 226 * 1024 && q.P <= 16383 &&
                       (int64_t)g.N * g.H * g.W < (1ll << 31);
#ifdef LCE_TUNING
        if (const char *e = getenv("LCE_TENSOR_SWAP")) swapped = swapped && atoi(e) != 0;
#endif
        if (swapped) {
            int sms2 = 148, dev = 0;
            if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms2, cudaDevAttrMultiProcessorCount, dev);
            const int n_blocks = (g.Cout + 127) / 128;
            int ctas_x = sms2 / n_blocks;
            if (ctas_x < 1) ctas_x = 1;
            if (ctas_x > q.n_tiles) ctas_x = q.n_tiles;
            if (cudaFuncSetAttribute(bconv3x3_tensor_swapped_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need) != cudaSuccess)
                return LCE_ERR_CUDA;
            bconv3x3_tensor_swapped_kernel<<<dim3((unsigned)ctas_x, (unsigned)n_blocks), kSwThreads, need, s>>>(q);
            return launch_status();
        }
    }

    // Channel block (32..256, a power of two) and schedule, by a rule that matches what was
    // measured on the ResNet-18 shapes: weights resident if the full channel width (up to 256)
    // fits beside two input buffers; otherwise stream one tap at a time with the widest block
    // that fits (wide MMAs amortise the A-operand traffic); a narrower resident block last.
    int sms = 148;
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    const size_t a_bytes = (size_t)2 * g.Cw * p.P * 16;
    const size_t raw_bytes = (size_t)2 * (((size_t)p.P * g.Cw + 3) / 4) * 16;
    auto fixed = [&](int blk) { return (size_t)2048 + 128 + 12 * (size_t)blk + 8 * (size_t)(((9 * g.Cw + 1) / 2) * 2) + raw_bytes; };
    auto tap_bytes = [&](int blk) { return (size_t)2 * g.Cw * blk * 16; };
    auto need_bytes = [&](int blk, bool res) {
        return res ? fixed(blk) + 9 * tap_bytes(blk) + 2 * a_bytes : fixed(blk) + 2 * tap_bytes(blk) + a_bytes;
    };
    auto feasible = [&](int blk, bool res) {
        if (need_bytes(blk, res) > 226 * 1024) return false;
        return res || (blk * g.Cw + kWorkers - 1) / kWorkers <= kMaxWordsPerThread;
    };
    int cout_pow2 = 32;
    while (cout_pow2 < g.Cout && cout_pow2 < 256) cout_pow2 *= 2;
    int n_blk = 0;
    bool resident = false;
    int force_blk = 0, force_res = -1;
#ifdef LCE_TUNING
    if (const char *e = getenv("LCE_TENSOR_BLK")) force_blk = atoi(e);
    if (const char *e = getenv("LCE_TENSOR_RES")) force_res = atoi(e);
#endif
    if (force_blk) {
        if (feasible(force_blk, force_res != 0)) { n_blk = force_blk; resident = force_res != 0; }
    } else if (feasible(cout_pow2, true)) {
        n_blk = cout_pow2; resident = true;
    } else {
        for (int blk = cout_pow2; blk >= 32 && n_blk == 0; blk /= 2)
            if (feasible(blk, false)) { n_blk = blk; resident = false; }
        for (int blk = cout_pow2 / 2; blk >= 32 && n_blk == 0; blk /= 2)
            if (feasible(blk, true)) { n_blk = blk; resident = true; }
    }
    if (n_blk == 0) return LCE_ERR_UNSUPPORTED;
    size_t smem = need_bytes(n_blk, resident);
    p.n_blk = n_blk;
    p.n_blk_log2 = 0;
    while ((1 << p.n_blk_log2) < n_blk) ++p.n_blk_log2;
    int cols = 32;
    while (cols < (resident ? 2 * n_blk : n_blk)) cols *= 2;
    p.tmem_cols = cols;
    const int n_blocks = (g.Cout + n_blk - 1) / n_blk;
    // Persistent grid.  A kernel that allocates TMEM is given one CTA per SM (the occupancy query
    // reports 1 for any such kernel, whatever its registers and shared memory), so the grid is one
    // CTA per SM.  The shared-memory carve-out is left to the driver: forcing the largest one leaves
    // no L1 for the streaming schedule's weight loads (measured: 24 -> 19 us at 14x14x256).
    int ctas_x = sms / n_blocks;
    if (ctas_x < 1) ctas_x = 1;
    if (ctas_x > p.n_tiles) ctas_x = p.n_tiles;
    const dim3 grid((unsigned)ctas_x, (unsigned)n_blocks);
    bool split = resident;
#ifdef LCE_TUNING
    if (const char *e = getenv("LCE_TENSOR_SPLIT")) split = resident && atoi(e) != 0;
    if (getenv("LCE_VERBOSE"))
        fprintf(stderr, "tensor: resident=%d split=%d n_blk=%d smem=%zu ctas_x=%d n_blocks=%d tiles=%d\n", (int)resident, (int)split, n_blk,
                smem, ctas_x, n_blocks, p.n_tiles);
#endif
    if (split) {
        if (cudaFuncSetAttribute(bconv3x3_tensor_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return LCE_ERR_CUDA;
        bconv3x3_tensor_split_kernel<<<grid, kSplitThreads, smem, s>>>(p);
    } else if (resident) {
        if (cudaFuncSetAttribute(bconv3x3_tensor_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return LCE_ERR_CUDA;
        bconv3x3_tensor_kernel<true><<<grid, kThreads, smem, s>>>(p);
    } else {
        if (cudaFuncSetAttribute(bconv3x3_tensor_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return LCE_ERR_CUDA;
        bconv3x3_tensor_kernel<false><<<grid, kThreads, smem, s>>>(p);
    }
    return launch_status();
}

#ifdef LCE_TUNING
extern "C" int lce_debug_write(const long long *host, int n)
{
    return cudaMemcpyToSymbol(g_dbg, host, sizeof(long long) * n) == cudaSuccess ? 0 : 1;
}
extern "C" int lce_debug_read(long long *host, int n)
{
    return cudaMemcpyFromSymbol(host, g_dbg, sizeof(long long) * n) == cudaSuccess ? 0 : 1;
}
#endif

// 0 = no bounded wait has expired on the current device since the library was loaded.
lce_status tensor_device_status(int *status)
{
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_tensor_status, sizeof(int)) != cudaSuccess) return LCE_ERR_CUDA;
    *status = v;
    return LCE_OK;
}

}  // namespace lce
