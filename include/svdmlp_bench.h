/*
 * svdmlp_bench.h - measurement, test and diagnostic hooks of libsvdmlp.
 *
 * None of these is a step of the method and none has a counterpart in the paper: they exist so
 * that the benchmark can count and time the library's kernels one by one and so that the tests
 * can exercise the bounded device-side waits.  The computational interface is svdmlp.h.
 */
#ifndef SVDMLP_BENCH_H_
#define SVDMLP_BENCH_H_

#include "svdmlp.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Failure-detection self-test.  Enqueues a one-warp kernel that waits - through the same bounded-wait routine
 * every production kernel uses - on a barrier that nothing will ever signal, with a limit of `limit_us`
 * microseconds (1 .. 1000000) instead of the production limit of 2 s.  When the limit passes the kernel
 * records SVDMLP_ERR_TIMEOUT in the handle's device status word and returns normally: nothing faults or traps,
 * the context and the handle stay usable, and svdmlp_last_device_status reports (and clears) the timeout.
 * Setting SVDMLP_LOG=1 in the environment makes forward calls print the kernel path they choose (stderr).
 */
int svdmlp_selftest_timeout(svdmlp_t* h, unsigned limit_us, void* stream);

/* Number of kernels this handle has launched since creation (for benchmark accounting). */
unsigned long long svdmlp_launch_count(const svdmlp_t* h);

/*
 * Per-kernel timing for benchmarks.  With profiling enabled every later forward call records a
 * CUDA event pair around each kernel it launches on the call's stream (a small serialising
 * overhead; leave it off for throughput runs and stream capture).  svdmlp_profile_read waits
 * for the most recent forward, writes the duration in milliseconds of each of its kernels to
 * ms[0 .. min(count, capacity)) in launch order and returns count (or a negative status);
 * svdmlp_profile_name gives the kernel's label ("stage1", "gateup", ...), NULL if out of range.
 */
int svdmlp_profile_enable(svdmlp_t* h, int enable);
int svdmlp_profile_read(svdmlp_t* h, float* ms, int capacity);
const char* svdmlp_profile_name(const svdmlp_t* h, int index);

/*
 * Measurement aid: restrict later forward calls of this handle to a subset of the path's kernels
 * so that one kernel can be timed or profiled back to back.  Bits: 1 first projection
 * (X V^T), 2 gate/up expansion with SiLU (small T: fused with the first half of the down chain),
 * 4 first half of the down chain (large T only), 8 second half of the down chain, 16 RMSNorm.
 * With anything but all bits set the outputs are meaningless.  Default: all bits.
 */
int svdmlp_stage_mask(svdmlp_t* h, unsigned mask);

/* Name of the kernel path the handle would use for T tokens: "skinny", "tensor", or "tensor-fused" (large T with
 * gate/up and the first down product in one kernel: ranks up to 128). */
const char* svdmlp_path_name(const svdmlp_t* h, int T);

/* Test aid: how long svdmlp_forward_finish_gather waits for its peers' flags before it gives up (default 2 s). */
int svdmlp_tp_wait_limit_ns(svdmlp_t* h, unsigned long long limit_ns);

#ifdef __cplusplus
}
#endif
#endif /* SVDMLP_BENCH_H_ */
