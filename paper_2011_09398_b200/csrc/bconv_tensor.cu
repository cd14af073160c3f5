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
//   * one CTA = 128 GEMM rows (TMEM lanes) x up to 256 output channels (TMEM columns); weights of
//     its channel block are expanded once per CTA and stay in shared memory; CTAs are persistent
//     over row tiles.  Per tile: expand the input rows -> issue 9*Cw MMAs from one thread ->
//     tcgen05.commit to an mbarrier -> all 128 threads read their accumulator row from TMEM and
//     apply the output transform.
// Every wait on the mbarrier is bounded; on expiry the kernel records a status word, skips the
// rest of its work, frees its TMEM and returns.
#include "common.cuh"

namespace lce {
namespace {

constexpr int kThreads = 128;
constexpr int kTileM = 128;
constexpr uint32_t kSpinLimit = 1u << 22;  // bounded wait: about a second at worst, far above any real tile

__device__ int g_tensor_status = 0;  // 0 ok, 1 = an mbarrier wait expired

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
    int32_t n_blk;       // output channels per CTA (multiple of 16, <= 256)
    int32_t tmem_cols;   // power of two >= max(32, n_blk)
    int32_t pad_corr;    // 9 * (32*Cw - Cin): what the zero pad bits (+1 * +1) add to every accumulator
    int32_t out_type, activation;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// K-major, no-swizzle operand descriptor; offsets in units of 16 bytes.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_units, uint32_t sbo_units)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)(lbo_units & 0x3FFFu) << 16;
    d |= (uint64_t)(sbo_units & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of this architecture
    return d;
}

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
        if (i > 64) __nanosleep(64);
    }
    return false;
}

__device__ __forceinline__ void mma_i8(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        :
        : "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, int32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}

// byte j of the result = +1 (0x01) where bit j of b is 0, -1 (0xFF) where it is 1
__device__ __forceinline__ uint2 expand_byte(const uint2 *table, uint32_t b) { return table[b & 0xFFu]; }

// 32 bits -> 32 bytes, written as two 16-byte chunks
__device__ __forceinline__ void expand_word(const uint2 *table, uint32_t word, uint4 *chunk_lo, uint4 *chunk_hi)
{
    const uint2 a = expand_byte(table, word), b = expand_byte(table, word >> 8);
    const uint2 c = expand_byte(table, word >> 16), d = expand_byte(table, word >> 24);
    *chunk_lo = make_uint4(a.x, a.y, b.x, b.y);
    *chunk_hi = make_uint4(c.x, c.y, d.x, d.y);
}

__global__ void __launch_bounds__(kThreads, 1)
bconv3x3_tensor_kernel(const TensorParams p)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    // layout: [table 2 KB][barrier + tmem slot 64 B][B operand][A operand]
    uint2 *table = reinterpret_cast<uint2 *>(smem_raw);
    uint64_t *mma_bar = reinterpret_cast<uint64_t *>(smem_raw + 2048);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_raw + 2048 + 16);
    uint8_t *sB = smem_raw + 2048 + 64;                        // [9 taps][2*Cw chunks][n_blk][16]
    uint8_t *sA = sB + (size_t)9 * 2 * p.Cw * p.n_blk * 16;    // [2*Cw chunks][P][16]

    const int tid = threadIdx.x, warp = tid >> 5;
    const int ch0 = blockIdx.y * p.n_blk;

    // ---- one-time set-up: expansion table, barrier, TMEM, this CTA's weights --------------------
    for (int e = tid; e < 256; e += kThreads) {
        uint32_t lo = 0, hi = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            lo |= (((e >> j) & 1) ? 0xFFu : 0x01u) << (8 * j);
            hi |= (((e >> (j + 4)) & 1) ? 0xFFu : 0x01u) << (8 * j);
        }
        table[e] = make_uint2(lo, hi);
    }
    if (tid == 0) {
        mbar_init(mma_bar, 1);
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

    // weights: packed [o][tap][cw] -> bytes [tap][chunk][channel in block][16]
    for (int e = tid; e < p.n_blk * 9 * p.Cw; e += kThreads) {
        const int cw = e % p.Cw;
        const int ot = e / p.Cw;
        const int tap = ot % 9, ch = ot / 9;
        const uint32_t word = (ch0 + ch < p.Cout) ? __ldg(p.w + ((int64_t)(ch0 + ch) * 9 + tap) * p.Cw + cw) : 0u;
        uint4 lo, hi;
        expand_word(table, word, &lo, &hi);
        uint4 *dst = reinterpret_cast<uint4 *>(sB) + (size_t)(tap * 2 * p.Cw + 2 * cw) * p.n_blk + ch;
        dst[0] = lo;
        dst[p.n_blk] = hi;
    }

    // instruction descriptor: D = S32, A and B signed 8-bit, both K-major, N = n_blk, M = 128
    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_blk >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
    const uint32_t a_saddr = smem_u32(sA), b_saddr = smem_u32(sB);
    uint32_t parity = 0;
    bool alive = true;

    for (int tile = blockIdx.x; tile < p.n_tiles && alive; tile += gridDim.x) {
        const int q0 = tile * kTileM;
        // ---- expand the grid positions q0 .. q0+P-1 of the stacked padded input ----------------
        for (int e = tid; e < p.P * p.Cw; e += kThreads) {
            const int row = e % p.P, cw = e / p.P;
            const int f = q0 + row;
            const int rr = f / p.Wp, cc = f - rr * p.Wp;
            const int n = rr / p.Hs, ry = rr - n * p.Hs;
            uint32_t word = 0u;  // pad position: all +1
            if (cc != 0 && ry != 0 && n < p.N)
                word = __ldg(p.in + (((int64_t)n * p.H + (ry - 1)) * p.W + (cc - 1)) * p.Cw + cw);
            uint4 lo, hi;
            expand_word(table, word, &lo, &hi);
            uint4 *dst = reinterpret_cast<uint4 *>(sA) + (size_t)(2 * cw) * p.P + row;
            dst[0] = lo;
            dst[p.P] = hi;
        }
        // make the generic-proxy writes visible to the tensor core's (async proxy) reads
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();

        // ---- MMAs: 9 taps x Cw K-steps of 32 channels, one issuing thread ------------------------
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            uint32_t accumulate = 0;
            for (int tap = 0; tap < 9; ++tap) {
                const int shift = (tap / 3) * p.Wp + (tap % 3);
                for (int cw = 0; cw < p.Cw; ++cw) {
                    const uint64_t adesc = make_desc(a_saddr + (uint32_t)((2 * cw) * p.P + shift) * 16u, (uint32_t)p.P, 8u);
                    const uint64_t bdesc =
                        make_desc(b_saddr + (uint32_t)((tap * 2 * p.Cw + 2 * cw) * p.n_blk) * 16u, (uint32_t)p.n_blk, 8u);
                    mma_i8(tmem_base, adesc, bdesc, idesc, accumulate);
                    accumulate = 1;
                }
            }
            // arrives on the barrier when every MMA above has finished (reads of sA/sB included)
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(mma_bar))
                         : "memory");
        }
        if (!mbar_wait_bounded(mma_bar, parity)) {
            g_tensor_status = 1;
            alive = false;
        }
        parity ^= 1u;
        // all threads agree on whether to go on (a thread that timed out must not strand the others)
        alive = __syncthreads_and(alive ? 1 : 0) != 0;
        if (!alive) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

        // ---- output transform: thread = TMEM lane = GEMM row -----------------------------------
        const int q = q0 + tid;
        const int rr = q / p.Wp, c = q - rr * p.Wp;
        const int n = rr / p.Hs, oh = rr - n * p.Hs;
        const bool row_ok = q < p.total_q && n < p.N && oh < p.H && c < p.W;
        const int64_t pix = ((int64_t)n * p.H + oh) * p.W + c;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);
        for (int c0 = 0; c0 < p.n_blk; c0 += 32) {
            uint32_t bits = 0u;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int cb = c0 + 16 * half;
                if (cb >= p.n_blk) break;  // uniform across the CTA
                int32_t v[16];
                tmem_ld16(lane_addr + (uint32_t)cb, v);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int o = ch0 + cb + j;
                    const int32_t acc = v[j] - p.pad_corr;
                    if (p.out_type == LCE_OUT_BITPACKED) {
                        const bool bit = o < p.Cout && acc < __ldg(p.thr + (o < p.Cout ? o : 0));
                        bits |= (bit ? 1u : 0u) << (16 * half + j);
                    } else if (row_ok && o < p.Cout) {
                        if (p.out_type == LCE_OUT_FLOAT32) {
                            const int32_t a = (p.activation == LCE_ACT_RELU && acc < 0) ? 0 : acc;
                            static_cast<float *>(p.out)[pix * p.Cout + o] = __fmaf_rn((float)a, __ldg(p.mult + o), __ldg(p.bias + o));
                        } else {
                            static_cast<int32_t *>(p.out)[pix * p.Cout + o] = acc;
                        }
                    }
                }
            }
            if (p.out_type == LCE_OUT_BITPACKED && row_ok && ch0 + c0 < p.Cout)
                static_cast<uint32_t *>(p.out)[pix * p.Cow + ((ch0 + c0) >> 5)] = bits;
        }
        // the next tile's MMAs overwrite the accumulators and the next expansion overwrites sA
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
    }

    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
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
    if (p.P > 16383) return LCE_ERR_UNSUPPORTED;  // descriptor offsets are 14-bit counts of 16 bytes

    // channel block: the widest of 256..32 whose expanded weights fit beside the input tile; a
    // block is a multiple of 32 so that a bit-packed output word never spans two CTAs
    const size_t a_bytes = (size_t)2 * g.Cw * p.P * 16;
    const size_t budget = 226 * 1024;  // of the 227 KB a CTA may have
    const int cout_pad = ((g.Cout + 31) / 32) * 32;
    int n_blk = 0;
    for (int cand = 256; cand >= 32; cand /= 2) {
        const int blk = cand < cout_pad ? cand : cout_pad;
        if (blk > 256) continue;
        const size_t b_bytes = (size_t)9 * 2 * g.Cw * blk * 16;
        if (2048 + 64 + a_bytes + b_bytes <= budget) { n_blk = blk; break; }
    }
    if (n_blk == 0) return LCE_ERR_UNSUPPORTED;
    p.n_blk = n_blk;
    int cols = 32;
    while (cols < n_blk) cols *= 2;
    p.tmem_cols = cols;
    size_t smem = 2048 + 64 + a_bytes + (size_t)9 * 2 * g.Cw * n_blk * 16;
    // no more CTAs per SM than the 512 TMEM columns can serve: pad the request if need be
    const size_t min_smem_for_tmem = (size_t)(227 * 1024) / (512 / cols) - 1024;
    if (smem < min_smem_for_tmem && (227 * 1024) / (smem + 1024) > (size_t)(512 / cols)) smem = min_smem_for_tmem;
    const int n_blocks = (g.Cout + n_blk - 1) / n_blk;
    int sms = 148;
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    int per_sm = (int)((227 * 1024) / (smem + 1024));
    if (per_sm < 1) per_sm = 1;
    if (per_sm > 512 / cols) per_sm = 512 / cols;
    if (per_sm > 8) per_sm = 8;
    int ctas_x = (sms * per_sm) / n_blocks;
    if (ctas_x < 1) ctas_x = 1;
    if (ctas_x > p.n_tiles) ctas_x = p.n_tiles;
    if (cudaFuncSetAttribute(bconv3x3_tensor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return LCE_ERR_CUDA;
    bconv3x3_tensor_kernel<<<dim3((unsigned)ctas_x, (unsigned)n_blocks), kThreads, smem, s>>>(p);
    return launch_status();
}

// 0 = no bounded wait has expired on the current device since the library was loaded.
lce_status tensor_device_status(int *status)
{
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_tensor_status, sizeof(int)) != cudaSuccess) return LCE_ERR_CUDA;
    *status = v;
    return LCE_OK;
}

}  // namespace lce
