/*
 * fastsgd_debug.h -- profiling and test aids of libfastsgd_b200.so.
 *
 * Nothing here is part of the codec (the paper has no counterpart for any of
 * it): per-kernel event timing and a launch counter for the benchmark, a way
 * for tests to shorten the kernels' bounded waits, and the byte offsets of a few
 * workspace fields that tests and the benchmark read or set.
 */
#ifndef FASTSGD_DEBUG_H
#define FASTSGD_DEBUG_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* While enabled, every kernel launch is bracketed by a pair of CUDA events
 * recorded on its stream.  fastsgd_kernel_timing_read synchronises those
 * events, adds up the elapsed milliseconds and the launches per kernel (index
 * 0 abs-sum, 1 encode, 2 decode-accumulate) since the last read, and forgets
 * them.  Off by default; the events add a little launch overhead. */
int fastsgd_kernel_timing_enable(int enable);
int fastsgd_kernel_timing_read(double ms_total[3], uint64_t launches[3]);

/* number of kernels the library has launched since it was loaded */
uint64_t fastsgd_launch_count(void);

/* Iteration limits of the kernels' bounded waits, for the launches that follow:
 *   block_polls  polls of a flag, descriptor or prefix another thread block writes
 *   copy_tries   tries (about 10 us each) of a wait on a bulk copy
 *   queue_polls  polls of the decoder's queue of large groups (0xFFFFFFFF: give
 *                up at the first poll that finds the slot empty)
 * 0 restores a default.  Tests shorten them so that a wait that cannot complete
 * (a counter they have set beyond reach) ends in FASTSGD_ST_TIMEOUT within
 * milliseconds; production code never calls this. */
int fastsgd_debug_set_wait_limits(uint32_t block_polls, uint32_t copy_tries, uint32_t queue_polls);

/* Caps the number of thread blocks of the encoders' launches (fastsgd_compress,
 * _batch, _kv) that follow; 0 restores the default (as many as are resident at
 * once).  With a cap the batch encoder does not split its blocks into two
 * teams.  The stream never depends on the grid: tests use this to show it. */
int fastsgd_debug_set_grid(uint32_t blocks);

/* Byte offsets inside the registered workspace (all of them in its fixed first
 * part): [0] u32 bar_count[8], arrivals at each gradient's grid barrier;
 * [1] u32 ne_count[8], tiles the last encoder launch read a second time, per
 * gradient; [2] u32 error; [3] decoder trace; [4] encoder trace, [5] its size
 * in bytes; [6] u32 decoder queue slots; [7] u32 decoder queue counters[6]. */
#define FASTSGD_DEBUG_LAYOUT_FIELDS 8
int fastsgd_debug_layout(uint64_t* offsets, uint32_t count);

/* 1 if the library was built with -DFASTSGD_TRACE (the kernels then write
 * %globaltimer stamps of their phases into the trace areas), else 0 */
int fastsgd_debug_trace_compiled(void);

#ifdef __cplusplus
}
#endif
#endif /* FASTSGD_DEBUG_H */
