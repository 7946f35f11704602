/*
 * darkattn_bench.h -- instruments of the benchmark and of profiling runs (libdarkattn_bench.so). Not part of the
 * product's interface: they time the product's kernels and probe the tensor pipe, and share the plan object
 * of darkattn.h. The paper has no counterpart to any of them.
 */
#ifndef DARKATTN_BENCH_H_
#define DARKATTN_BENCH_H_

#include "darkattn.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Number of kernel launches one forward (which = 0) or one backward (which = 1) call enqueues
 * (backward: when it is given O and `saved`; otherwise the forward launches come on top), in the
 * plan's current mode: with per-kernel timing on, the tensor-core backward launches one fewer.   */
int32_t darkattn_plan_launches(darkattn_plan_t plan, int32_t which);

/* Per-kernel device times, for benchmarks. While enabled, forward and backward record a CUDA event on
 * the call's stream in front of every kernel they launch and one behind the last (events are host
 * objects created by the first enabling call; no device memory is involved). Enabling also clears the
 * accumulated times. Leave it off when measuring whole-call throughput.                           */
darkattn_status_t darkattn_kernel_timing(darkattn_plan_t plan, int32_t enable);

/* Wait for the events recorded since the last harvest, add the elapsed time between consecutive events
 * to the kernel in front of which the first was recorded, and report the totals since timing was
 * enabled: names (HOST buffer of 64 * max_entries bytes, one NUL-terminated name per 64 bytes),
 * total_ms and launches (HOST arrays of max_entries), *count = entries written. Call it at least once
 * per 96 kernels, since only that many events are kept.                                            */
darkattn_status_t darkattn_kernel_times(darkattn_plan_t plan, int32_t max_entries, char *names, float *total_ms,
                                        int32_t *launches, int32_t *count);

/* Measure what one tcgen05.mma (bf16, M = 128, K = 16) costs on this GPU in the forms the scan kernels
 * issue, so that their tensor-pipe time can be told apart from the hand-over between MMA batches and
 * the warps that consume them. variant: 0 both operands in shared memory, K-major, N = 128; 1 B MN-major;
 * 2 A and B MN-major; 3 A in tensor memory, B K-major; 4 A in tensor memory, B MN-major; 5 as 0 with
 * N = 256; 6 as 0 with N = 64; 7 A MN-major, N = 16. One CTA per SM issues two batches of dependent MMAs
 * (32 and 288) and waits for each batch's commit with a bounded wait; busy_epilogue != 0 makes the 16
 * other warps read tensor memory and write shared memory meanwhile. Writes the SM-clock cycles per MMA
 * (slope) and the fixed cycles per batch (intercept) to the two host pointers. Synchronises the
 * stream. DARKATTN_ERR_TIMEOUT if a commit did not arrive within the wait's limit.                 */
darkattn_status_t darkattn_measure_mma_cycles(int32_t variant, int32_t busy_epilogue, double *cycles_per_mma,
                                              double *batch_overhead_cycles, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* DARKATTN_BENCH_H_ */
