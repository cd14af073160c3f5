// Carry-save popcount accumulation for the binary GEMM inner loop.
//
// The paper's BGEMM multiplies with XOR and accumulates with POPCOUNT (Section 2, Section 3.2):
// for one output, cnt = sum_k popc(a_k ^ w_k).  On this GPU POPC issues at a quarter of the
// rate of the logic unit, so instead of one POPC per word the mismatch words x_k = a_k ^ w_k of
// nine consecutive k are first compressed bitwise with full adders (3:2 carry-save counters,
// one LOP3 per output bit-plane) into four words S, C, T, F with
//     sum_{k<9} popc(x_k) = popc(S) + 2*popc(C) + 2*popc(T) + 4*popc(F)
// which needs 4 POPC instead of 9.  The XORs with the weights are folded into the adders:
// within a triple (x0,x1,x2)
//     s = x0^x1^x2 = (a0^a1^a2) ^ (w0^w1^w2)         -- both factors are precomputed once per
//     d = x0^x1    = (a0^a1)    ^ (w0^w1)               pixel resp. once per output channel
//     c = maj(x0,x1,x2) = d ? ~s&... : x0  =  (d & ~s) | (~d & x0),   x0 = a0 ^ w0
// so a triple costs 4 LOP3 per output instead of 5, and a nine-word group 16 LOP3 + 4 POPC.
#pragma once
#include <stdint.h>

namespace lce {

template <int LUT>
__device__ __forceinline__ uint32_t lop3(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, %4;" : "=r"(r) : "r"(a), "r"(b), "r"(c), "n"(LUT));
    return r;
}
__device__ __forceinline__ uint32_t xor3(uint32_t a, uint32_t b, uint32_t c) { return lop3<0x96>(a, b, c); }
__device__ __forceinline__ uint32_t maj3(uint32_t a, uint32_t b, uint32_t c) { return lop3<0xE8>(a, b, c); }
// carry of the triple from d = x0^x1, s = x0^x1^x2 and x0:  (d & ~s) | (~d & x0)
__device__ __forceinline__ uint32_t carry_dsx(uint32_t d, uint32_t s, uint32_t x0) { return lop3<0x3A>(d, s, x0); }

// Per-pixel (activation side) and per-channel (weight side) operands of one triple.
struct Triple {
    uint32_t all;    // v0 ^ v1 ^ v2
    uint32_t pair;   // v0 ^ v1
    uint32_t first;  // v0
};

__device__ __forceinline__ Triple make_triple(uint32_t v0, uint32_t v1, uint32_t v2)
{
    Triple t;
    t.pair = v0 ^ v1;
    t.all = t.pair ^ v2;
    t.first = v0;
    return t;
}

// popcount of the nine mismatch words of one (pixel, channel) pair, given the three triples of
// each side: 16 LOP3 + 4 POPC + the weighted sum.
__device__ __forceinline__ uint32_t popc9(const Triple (&a)[3], const Triple (&w)[3])
{
    uint32_t s[3], c[3];
#pragma unroll
    for (int g = 0; g < 3; ++g) {
        s[g] = a[g].all ^ w[g].all;
        const uint32_t d = a[g].pair ^ w[g].pair;
        const uint32_t x0 = a[g].first ^ w[g].first;
        c[g] = carry_dsx(d, s[g], x0);
    }
    const uint32_t S = xor3(s[0], s[1], s[2]);  // weight 1
    const uint32_t C = maj3(s[0], s[1], s[2]);  // weight 2
    const uint32_t T = xor3(c[0], c[1], c[2]);  // weight 2
    const uint32_t F = maj3(c[0], c[1], c[2]);  // weight 4
    return __popc(S) + 2u * (__popc(C) + __popc(T)) + 4u * __popc(F);
}

// The same nine-word count added onto an accumulator with four multiply-adds whose multipliers
// (1, 2, 2, 4) arrive in registers: integer multiply-add issues on the FMA pipe, so the
// weighted sum costs the logic pipe nothing.  `k` must hold {1, 2, 4}.
struct Weights124 {
    uint32_t one, two, four;
};
__device__ __forceinline__ uint32_t mad_u32(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t r;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
__device__ __forceinline__ void popc9_mad(const Triple (&a)[3], const Triple (&w)[3], const Weights124 &k,
                                          uint32_t &acc)
{
    uint32_t s[3], c[3];
#pragma unroll
    for (int g = 0; g < 3; ++g) {
        s[g] = a[g].all ^ w[g].all;
        const uint32_t d = a[g].pair ^ w[g].pair;
        const uint32_t x0 = a[g].first ^ w[g].first;
        c[g] = carry_dsx(d, s[g], x0);
    }
    const uint32_t S = xor3(s[0], s[1], s[2]);
    const uint32_t C = maj3(s[0], s[1], s[2]);
    const uint32_t T = xor3(c[0], c[1], c[2]);
    const uint32_t F = maj3(c[0], c[1], c[2]);
    acc = mad_u32(__popc(S), k.one, acc);
    acc = mad_u32(__popc(C), k.two, acc);
    acc = mad_u32(__popc(T), k.two, acc);
    acc = mad_u32(__popc(F), k.four, acc);
}

// The nine-word count of TP pixels against one channel, written stage by stage across the pixels
// so that neighbouring instructions are independent (TP-way instruction-level parallelism inside
// one warp): all first-level sums and carries, then the second level, then the popcounts, then
// the multiply-adds.  acc is the thread's accumulator tile, column `J` is the channel.
template <int TP, int NCH, int J>
__device__ __forceinline__ void popc9_mad_pixels(const Triple (&a)[TP][3], const Triple (&w)[3], const Weights124 &k,
                                                 uint32_t (&acc)[TP][NCH])
{
    uint32_t s[TP][3], c[TP][3];
#pragma unroll
    for (int g = 0; g < 3; ++g)
#pragma unroll
        for (int i = 0; i < TP; ++i) s[i][g] = a[i][g].all ^ w[g].all;
#pragma unroll
    for (int g = 0; g < 3; ++g)
#pragma unroll
        for (int i = 0; i < TP; ++i) {
            const uint32_t d = a[i][g].pair ^ w[g].pair;
            const uint32_t x0 = a[i][g].first ^ w[g].first;
            c[i][g] = carry_dsx(d, s[i][g], x0);
        }
    uint32_t S[TP], C[TP], T[TP], F[TP];
#pragma unroll
    for (int i = 0; i < TP; ++i) {
        S[i] = xor3(s[i][0], s[i][1], s[i][2]);
        C[i] = maj3(s[i][0], s[i][1], s[i][2]);
    }
#pragma unroll
    for (int i = 0; i < TP; ++i) {
        T[i] = xor3(c[i][0], c[i][1], c[i][2]);
        F[i] = maj3(c[i][0], c[i][1], c[i][2]);
    }
    uint32_t pS[TP], pC[TP], pT[TP], pF[TP];
#pragma unroll
    for (int i = 0; i < TP; ++i) { pS[i] = __popc(S[i]); pC[i] = __popc(C[i]); }
#pragma unroll
    for (int i = 0; i < TP; ++i) { pT[i] = __popc(T[i]); pF[i] = __popc(F[i]); }
#pragma unroll
    for (int i = 0; i < TP; ++i) acc[i][J] = mad_u32(pS[i], k.one, acc[i][J]);
#pragma unroll
    for (int i = 0; i < TP; ++i) acc[i][J] = mad_u32(pC[i], k.two, acc[i][J]);
#pragma unroll
    for (int i = 0; i < TP; ++i) acc[i][J] = mad_u32(pT[i], k.two, acc[i][J]);
#pragma unroll
    for (int i = 0; i < TP; ++i) acc[i][J] = mad_u32(pF[i], k.four, acc[i][J]);
}

// The same with two pixels' counts per accumulator register: pixel i < H = ceil(TP/2) in the low 16
// bits of acc[i], pixel i >= H in the high 16 bits of acc[i - H], its multiply-adds using the
// multipliers shifted left by 16 (`khi` = {1<<16, 2<<16, 4<<16}).  Counts must stay below 65536.
template <int TP, int NCH, int J>
__device__ __forceinline__ void popc9_mad_pixels_packed(const Triple (&a)[TP][3], const Triple (&w)[3], const Weights124 &k,
                                                        const Weights124 &khi, uint32_t (&acc)[(TP + 1) / 2][NCH])
{
    constexpr int H = (TP + 1) / 2;
    uint32_t s[TP][3], c[TP][3];
#pragma unroll
    for (int g = 0; g < 3; ++g)
#pragma unroll
        for (int i = 0; i < TP; ++i) s[i][g] = a[i][g].all ^ w[g].all;
#pragma unroll
    for (int g = 0; g < 3; ++g)
#pragma unroll
        for (int i = 0; i < TP; ++i) {
            const uint32_t d = a[i][g].pair ^ w[g].pair;
            const uint32_t x0 = a[i][g].first ^ w[g].first;
            c[i][g] = carry_dsx(d, s[i][g], x0);
        }
    uint32_t S[TP], C[TP], T[TP], F[TP];
#pragma unroll
    for (int i = 0; i < TP; ++i) {
        S[i] = xor3(s[i][0], s[i][1], s[i][2]);
        C[i] = maj3(s[i][0], s[i][1], s[i][2]);
    }
#pragma unroll
    for (int i = 0; i < TP; ++i) {
        T[i] = xor3(c[i][0], c[i][1], c[i][2]);
        F[i] = maj3(c[i][0], c[i][1], c[i][2]);
    }
    uint32_t pS[TP], pC[TP], pT[TP], pF[TP];
#pragma unroll
    for (int i = 0; i < TP; ++i) { pS[i] = __popc(S[i]); pC[i] = __popc(C[i]); }
#pragma unroll
    for (int i = 0; i < TP; ++i) { pT[i] = __popc(T[i]); pF[i] = __popc(F[i]); }
#pragma unroll
    for (int i = 0; i < TP; ++i) acc[i % H][J] = mad_u32(pS[i], i < H ? k.one : khi.one, acc[i % H][J]);
#pragma unroll
    for (int i = 0; i < TP; ++i) acc[i % H][J] = mad_u32(pC[i], i < H ? k.two : khi.two, acc[i % H][J]);
#pragma unroll
    for (int i = 0; i < TP; ++i) acc[i % H][J] = mad_u32(pT[i], i < H ? k.two : khi.two, acc[i % H][J]);
#pragma unroll
    for (int i = 0; i < TP; ++i) acc[i % H][J] = mad_u32(pF[i], i < H ? k.four : khi.four, acc[i % H][J]);
}

// One triple added onto an accumulator with multiply-adds (K tails of the pointwise kernel).
__device__ __forceinline__ void popc3_mad(const Triple &a, const Triple &w, const Weights124 &k, uint32_t &acc)
{
    const uint32_t s = a.all ^ w.all;
    const uint32_t d = a.pair ^ w.pair;
    const uint32_t x0 = a.first ^ w.first;
    acc = mad_u32(__popc(s), k.one, acc);
    acc = mad_u32(__popc(carry_dsx(d, s, x0)), k.two, acc);
}

// popcount of one triple alone (used for K tails and by the 3:2 probe): 4 LOP3 + 2 POPC.
__device__ __forceinline__ uint32_t popc3(const Triple &a, const Triple &w)
{
    const uint32_t s = a.all ^ w.all;
    const uint32_t d = a.pair ^ w.pair;
    const uint32_t x0 = a.first ^ w.first;
    return __popc(s) + 2u * __popc(carry_dsx(d, s, x0));
}

}  // namespace lce
