/*
 * gf_bench.h -- instrumentation of libgf_b200 for benchmarks and tests.
 *
 * None of these calls is part of the method (the paper has no counterpart): they count
 * and time the kernels that the calls of gf.h launch.  The event pool behind the timing
 * is process-wide state of the library, created on first use.
 */
#ifndef GF_BENCH_H_
#define GF_BENCH_H_

#include "gf.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Number of kernels this library has launched in this process so far. */
uint64_t gf_kernel_launch_count(void);

/* Optional per-kernel timing.  mode 0: off (default).  mode 1: every launch of kernel
 * `kernel_id` is bracketed by a pair of CUDA events recorded on the stream it is launched
 * on.  mode 2: every kernel is bracketed (kernel_id ignored).  Events come from an internal
 * pool that is created on first use; when the pool is exhausted further launches are not
 * timed.  Not for use while a stream is being captured. */
gf_status gf_profile_configure(int32_t mode, int32_t kernel_id);

typedef struct gf_kernel_time {
    int32_t kernel_id;
    int32_t launches;   /* timed launches since the last read */
    double total_ms;    /* sum of their event-to-event durations */
} gf_kernel_time;

/* Waits for the recorded events, writes one entry per kernel that was timed since the last
 * read (at most max_entries) and clears the records.  Returns the number of entries
 * written, or -1 if a CUDA call failed. */
int32_t gf_profile_read(gf_kernel_time* out, int32_t max_entries);

/* Self-test of the bounded device-side waits (no counterpart in the paper).  Every wait a
 * kernel of this library makes on an mbarrier gives up after a limit of clocks, sets a bit of
 * the workspace's error word and lets the kernel return, so that a copy that never lands is
 * reported (GF_ERR_TIMEOUT from gf_last_async_status) instead of hanging the GPU.  This call
 * launches one small block that waits, with that same wait and a limit of `limit_cycles`
 * clocks (1 .. 2e9; about 0.5 ns each), on a barrier that nothing ever arrives on: the wait
 * runs out, the block records it in the error word at the head of `workspace` (device
 * memory, >= 256 bytes, 16-byte aligned) and ends normally.  The next gf_backward on that
 * workspace clears the word again. */
gf_status gf_selftest_bounded_wait(void* workspace, int64_t limit_cycles, void* stream);

/* Name of a kernel id (ids are 0 .. gf_kernel_id_count()-1), NULL if out of range. */
const char* gf_kernel_name(int32_t kernel_id);
int32_t gf_kernel_id_count(void);

#ifdef __cplusplus
}
#endif
#endif /* GF_BENCH_H_ */
