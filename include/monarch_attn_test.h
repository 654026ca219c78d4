/* libmonarch_attn -- test and profiling hooks.  Not part of the production interface: both calls
 * change process-wide state, and knob 2 makes the library return garbage on purpose.  They exist so
 * that the tests can watch a bounded device-side wait run out without faulting or hanging a GPU,
 * and so that the pipeline of the persistent kernels can be timed stage by stage. */
#ifndef MONARCH_ATTN_TEST_H_
#define MONARCH_ATTN_TEST_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Profiling aid for the persistent tensor path.  With a DEVICE buffer of at least 4*64*8 int64
 * set, CTAs 0-3 of later MA_PATH_TENSOR / MA_PATH_TENSOR_TMEM launches write SM-clock stamps
 * [cta][tile][event] for their first 64 tiles; events: 0 operands requested, 1 score MMA issued,
 * 2 softmax group sees the scores, 3 P written, 4 apply MMA issued, 5 softmax group sees O,
 * 6 rows staged, 7 rows stored and signalled (MA_PATH_TENSOR_TMEM: output unit given back).  NULL switches it off (the default).  Process-wide;
 * the buffer stays owned by the caller. */
int monarch_attn_set_trace_buffer(void* device_buffer, size_t bytes);

/* Test and tuning knobs (process-wide; not for production use).  Knobs 1 and 2 belong to the
 * persistent tensor path:
 *   knob 1: bound, in SM clocks, of every device-side wait (value <= 0 restores the default 2e9);
 *   knob 2: non-zero leaves the first half-step out of later single-launch runs, so that the
 *           dependency waits of the second half-step can never be satisfied.  Together they let a
 *           test watch a wait run out: the kernel ends by itself, results are garbage, and
 *           monarch_attn_device_status reports MA_ERR_TIMEOUT.  Nothing faults or hangs.
 *   knob 3: number of chunks monarch_attn_fwd_host cuts a call into (1..8, default 4). */
int monarch_attn_debug_knob(int knob, long long value);

#ifdef __cplusplus
}
#endif
#endif /* MONARCH_ATTN_TEST_H_ */
