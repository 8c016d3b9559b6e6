/*
 * cachefocus_debug.h -- test, debugging and benchmarking aids of the CacheFocus library.
 *
 * None of these is part of the method (the paper has no counterpart).  They act on process-wide
 * state guarded by one mutex: calls are safe from several host threads, but the switches apply to
 * every thread's later library calls, so use them from test and benchmark programs only.
 */
#ifndef CACHEFOCUS_DEBUG_H_
#define CACHEFOCUS_DEBUG_H_

#include "cachefocus.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Selects the attention kernel: 0 = automatic (tensor-core kernel when the geometry allows),
 * 1 = force the portable CUDA-core kernel.  Process-wide. */
int cf_set_attn_path(int32_t path);

/* Timing aid for benchmarks (not part of the method).  cf_profile_begin(n) makes every later
 * cf_query_prefill_attn call bracket its main attention kernel (the fused re-position +
 * QK^T + softmax + PV kernel, without the small merge kernels) with a pair of CUDA events on
 * the launching stream, for at most n calls.  cf_profile_end() waits for those events, writes
 * the kernel durations in milliseconds to the host array `ms` (capacity entries), the number
 * of recorded launches to *count, and switches recording off.  Do not use inside stream
 * capture.  The events are created by cf_profile_begin and destroyed by cf_profile_end. */
int cf_profile_begin(int32_t max_records);
int cf_profile_end(float* ms, int32_t capacity, int32_t* count);

/* Runs the library's bounded device-side wait until it gives up: a one-block kernel waits on an
 * mbarrier that nothing arrives on, with a limit of `limit_cycles` SM clocks (1 .. 2e9; 2e6 is about
 * a millisecond), then raises CF_ERR_TIMEOUT in the plan's status word and returns normally -- the
 * same reporting path the attention kernel takes when one of its waits expires.  The device stays
 * usable; cf_plan_init clears the status word again.  Returns the launch status. */
int cf_debug_wait_timeout(const cf_geom* geom, const cf_batch* batch, void* plan, int64_t limit_cycles,
                          void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CACHEFOCUS_DEBUG_H_ */
