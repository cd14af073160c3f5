/*
 * lce_probe.h -- C ABI of the measurement-only companion library (liblce_probe.so): micro-benchmarks of
 * the SM's integer pipes and of the ways to stage activation tiles in shared memory.  Not part of the convolution library; bench.py loads it to measure the
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

/* Staging probe: times how fast CTAs of 256 threads (two per SM, two alternating buffers, no arithmetic
 * behind the copies) bring tiles of a bit-packed activation tensor [batch][in_h][in_w][in_words] into
 * shared memory, a tile being rows_per_tile image rows plus one halo row on each side:
 *   mode 0: one 4-byte asynchronous copy per word into word planes [word][row][x] (what the XOR/POPC
 *           kernel's loader does), mode 1: one 16-byte asynchronous copy per four words into
 *           [row][x][word], mode 2: one tensor-map bulk copy per tile into [row][x][word] (this GPU's
 *           memory, no multicast; rows outside the tensor arrive as zeros).
 * in_words: a power of two <= 32, and >= 4 for modes 1 and 2 (LCE_ERR_UNSUPPORTED otherwise).
 * Synchronous; allocates the tensor (filled with a constant) and frees it.  Waits on the copy barrier
 * are time-bounded; LCE_ERR_DEVICE_TIMEOUT if one ran out.
 *   us_per_pass:   HOST pointer: microseconds for all CTAs together to stage the whole tensor once.
 *   first_tile_us: HOST pointer: median over the CTAs of the time from kernel entry to the first
 *                  tile being readable in shared memory. */
lce_status lce_probe_stage(int32_t mode, int32_t batch, int32_t in_h, int32_t in_w, int32_t in_words,
                           int32_t rows_per_tile, int32_t passes, double *us_per_pass, double *first_tile_us,
                           void *stream);

#ifdef __cplusplus
}
#endif
#endif /* LCE_PROBE_B200_H_ */
