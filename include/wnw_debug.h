/*
 * wnw_debug.h -- test and measurement hooks of the WnW library (not part of the decode path's interface).
 *
 * Same conventions as wnw.h.  Production code needs none of these: the bounded-wait test hook, per-kernel event
 * timing, and the host-link probe the benchmark reports recall traffic against.
 */
#ifndef WNW_DEBUG_H_
#define WNW_DEBUG_H_

#include "wnw.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Test hook for the bounded waits: adds `delta` to the device's step-epoch word, so that the tidal CTAs of the next
 * replayed step wait for a recall epoch that nothing will publish.  Every such wait gives up after about a second of
 * SM clocks, the kernel finishes on what it has and sets the sticky status that wnw_sync reports as WNW_ERR_TIMEOUT.
 * The cache's results are meaningless afterwards; destroy it.  Not for production use. */
wnw_status_t wnw_debug_advance_step_epoch(wnw_cache_t *cache, int32_t delta);

/* Optional per-kernel timing: when enabled the library brackets its attention-kernel launches with CUDA events
 * on the launching stream; wnw_get_kernel_time returns the accumulated milliseconds and launch count since the
 * last call (drains the stream).  Off by default. */
wnw_status_t wnw_set_kernel_timing(wnw_cache_t *cache, int32_t enable);
wnw_status_t wnw_get_kernel_time(wnw_cache_t *cache, float *attn_ms, int32_t *attn_launches);

/* Host-link probe used by the benchmark: copies `bytes` from pinned host memory into device memory `reps` times
 * (a) with cudaMemcpyAsync and (b) with the library's recall kernel on a synthetic plan, and returns GB/s of each. */
wnw_status_t wnw_measure_host_link(int32_t device, int64_t bytes, int32_t reps, double *memcpy_gbs, double *kernel_gbs);

#ifdef __cplusplus
}
#endif
#endif /* WNW_DEBUG_H_ */
