/*
 * lisa_debug.h -- test and measurement hooks of the LiSA library.  Not part of the product interface
 * (include/lisa.h): nothing here is needed to run the method, and the state behind these calls is process-global
 * and not thread-safe.
 */
#ifndef LISA_DEBUG_H_
#define LISA_DEBUG_H_

#include "lisa.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Measurement aid for the tensor-core path of lisa_attn_shared_prefill, which runs as several kernels (pack the
 * low-rank operands, emit score planes, align, attention).  lisa_prefill_phase_timing(1) makes every later call
 * record CUDA events around each of them on the caller's stream (it creates the events; 0 destroys them; not
 * thread-safe, single device); lisa_prefill_phase_times waits for the recorded work and returns the device time
 * in milliseconds summed per phase since the last read: ms4[0] pack, [1] emit, [2] align, [3] attention. */
lisa_status_t lisa_prefill_phase_timing(int enable);
lisa_status_t lisa_prefill_phase_times(float* ms4);

/* on != 0: every later call in this process uses the general SIMT kernels even where a tensor-core kernel
 * exists (for cross-checking the two paths against each other); on == 0 restores the default choice. */
void lisa_force_general_kernels(int on);

/* Enqueues a one-warp kernel whose only thread waits, with the library's bounded wait, for an arrival that never
 * comes; after limit_cycles SM cycles (1 .. 1e8) the wait gives up and records it, so the next lisa_check() on the
 * stream returns LISA_ERR_TIMEOUT and the one after that LISA_OK.  Nothing else is touched: the device context stays
 * usable.  This is the path a tensor-core kernel takes when one of its hand-offs stalls. */
lisa_status_t lisa_debug_wait_timeout(int64_t limit_cycles, lisa_stream_t stream);

/* Number of kernels this library has enqueued so far in this process (all threads). */
uint64_t lisa_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* LISA_DEBUG_H_ */
