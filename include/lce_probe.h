/*
 * lce_probe.h -- C ABI of the measurement-only companion library (liblce_probe.so): micro-benchmarks of
 * the SM's integer pipes.  Not part of the convolution library; bench.py loads it to measure the
 * ceiling the XOR/POPC kernels are judged against (the paper's Section 3.2 and Table 1 count
 * instructions per binary MAC on a Cortex-A76; this is the same exercise on an SM).
 */
#ifndef LCE_PROBE_B200_H_
#define LCE_PROBE_B200_H_

#include "lce.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Integer-pipe probe: runs a register/shared-memory resident loop of one instruction mix on
 * every SM of the current device and reports how many 32-bit word operations (one XOR +
 * POPCOUNT + accumulate of a packed word, i.e. 32 binary MACs) it retired per second.
 * mix: 0 plain xor+popc+add, 1 3:2 carry-save, 2 9-word carry-save tree, 10 LOP3 only,
 * 11 POPC only, 12 IADD3 only, 13 IMAD only (the last four count instructions, not word-ops),
 * 20 mma.sync b1 xor.popc, 21 mma.sync b1 and.popc (count 32-bit word pairs); 30 / 31 the logic
 * group / the MMA group of a combined run (even warps mix 3, odd warps mix 21, at the same time;
 * the per-second figure is the group's per-clock rate at the maximum SM clock); 32 / 33 the same
 * two groups each running alone (the other half of the warps idle).
 * Synchronous (times itself with CUDA events on `stream`); allocates a few KB and frees them.
 *   ops_per_second, ops_per_clock_per_sm: HOST pointers, written on success; the per-clock
 *   figure uses the SM cycle counter read inside the kernel. */
lce_status lce_probe_pipe(int32_t mix, int32_t iterations, double *ops_per_second,
                          double *ops_per_clock_per_sm, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* LCE_PROBE_B200_H_ */
