// Device-side building blocks of the tensor-core kernel: mbarriers with time-bounded waits, the bulk
// copy engine, tcgen05 commit / TMEM loads, small asynchronous copies and the bit -> e2m1 expansion.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace lce {

// A wait on an mbarrier gives up after this long (far above any tile's work, short enough that a
// stalled kernel hands the GPU back quickly).
constexpr uint64_t kWaitLimitNs = 200ull * 1000 * 1000;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t globaltimer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
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
// Wait bounded by time, not by iterations; false when the limit was reached.  (try_wait with a
// suspend-time hint was measured here: a suspended thread often slept out its whole hint, microseconds
// after the barrier had flipped, so the plain form is polled, with a short sleep once the wait is long.)
// The waiting itself is one copy of code shared by all call sites (inlined and unrolled, the loops below were
// 4 KB per call site and two thirds of the kernel: four roles running side by side then miss the
// instruction caches all the time).
__device__ __noinline__ bool mbar_wait_slow(uint64_t *bar, uint32_t parity, uint64_t limit_ns)
{
#pragma unroll 1
    for (int i = 0; i < 16; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    // a longer wait: sleep between polls, a little longer every time (polling warps take issue slots from
    // the warps that work)
    const uint64_t t0 = globaltimer_ns();
    uint32_t nap = 32;
    do {
#pragma unroll 1
        for (int i = 0; i < 64; ++i) {
            __nanosleep(nap);
            if (mbar_try_wait(bar, parity)) return true;
            if (nap < 64) nap += nap >> 1;
        }
    } while (globaltimer_ns() - t0 < limit_ns);
    return false;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, uint64_t limit_ns = kWaitLimitNs)
{
    if (mbar_try_wait(bar, parity)) return true;  // already there: the common case on the critical path
    return mbar_wait_slow(bar, parity, limit_ns);
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// one arrival that also announces `bytes` of asynchronous copies to this barrier
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// global -> shared copy by the bulk copy engine (both addresses 16-byte aligned, size a multiple of 16);
// completion is counted on the barrier.  This GPU's memory only, no multicast.
__device__ __forceinline__ void bulk_copy_g2s(void *smem_dst, const void *gmem_src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(smem_dst)),
                 "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// arrives on the barrier when every MMA issued so far by this thread has finished (operand reads included)
__device__ __forceinline__ void mma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 32 (16) consecutive TMEM columns of this warp's 32 lanes, as floats
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32])
{
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, "
        "[%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[32])
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
#pragma unroll
    for (int j = 16; j < 32; ++j) v[j] = 0.f;
}

// 16 consecutive TMEM columns into a 16-element array
__device__ __forceinline__ void tmem_ld16x(uint32_t taddr, float (&v)[16])
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
}

// asynchronous global -> shared copy of BYTES (4, 8 or 16); with valid == false zeros are written
template <int BYTES>
__device__ __forceinline__ void cp_async_zfill(uint32_t *smem_dst, const uint32_t *gmem_src, bool valid)
{
    const int src_size = valid ? BYTES : 0;
    if (BYTES == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(src_size) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;" ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "n"(BYTES), "r"(src_size) : "memory");
}

// 32 packed bits -> 32 e2m1 values (16 bytes): 0 bit -> +1.0 (nibble 0x2), 1 bit -> -1.0 (nibble 0xA).
// Value (register j, nibble i) is bit 4 i + j of the word; activations and weights use the same
// order, and the contraction sums over all of them, so the order itself is free.
__host__ __device__ __forceinline__ uint4 mx_expand_word(uint32_t w)
{
    uint4 v;
    v.x = ((w << 3) & 0x88888888u) | 0x22222222u;
    v.y = ((w << 2) & 0x88888888u) | 0x22222222u;
    v.z = ((w << 1) & 0x88888888u) | 0x22222222u;
    v.w = (w & 0x88888888u) | 0x22222222u;
    return v;
}

}  // namespace lce
