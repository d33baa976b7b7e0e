/*
 * qf_testing.h -- test, diagnostic and measurement hooks of the Q-First
 * decode-attention library.  Same shared library as qf.h, separate header:
 * nothing here is needed to use the method, and none of it has a counterpart
 * in the paper.  The hooks exist so that the schedule's arithmetic, the bounded
 * waits and the status plumbing can be exercised without faulting a GPU, and
 * so that a benchmark can time one kernel of a call.
 *
 * State these hooks add: qf_set_profile_events stores two event handles per
 * HOST THREAD (thread-local; no other thread sees them) until they are cleared;
 * qf_last_launch_count reads a thread-local counter that every enqueueing call
 * of qf.h on that thread overwrites.
 */
#ifndef QF_TESTING_H_
#define QF_TESTING_H_

#include "qf.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * qf_params.flags bit, default sweep kernel only: hand out the tail of the work
 * as drawn chunks however short the sweep is (by default only sweeps long enough
 * to gain from it do).  Same results up to fp32 summation order; lets small
 * parity cases reach the drawn-chunk path.
 */
enum { QF_FLAG_DRAW_ALWAYS = 8 };

/*
 * qf_params.flags bit: qf_decode_step treats no sweep as small (see there): the
 * finish and merge kernels run as for large problems.  Lets small parity cases
 * reach those kernels through that call too.
 */
enum { QF_FLAG_NO_SMALL_MERGE = 32 };

/*
 * Every wait inside the kernels is bounded: when its limit runs out the kernel
 * records QF_STATUS_TIMEOUT and returns instead of hanging.  This call enqueues
 * a one-warp kernel that waits, with a limit of a few thousand polls (under a
 * millisecond), on a barrier that nothing will ever complete, through the same
 * wait routine; afterwards qf_read_status(workspace) must report
 * QF_STATUS_TIMEOUT and the context must still be usable.  `workspace`: at
 * least 256 bytes of device memory, 256-byte aligned (its header words are
 * overwritten).
 */
int qf_selftest_bounded_wait(void *workspace, void *cuda_stream);

/*
 * Host only, no GPU needed.  The sweep cuts its work, `total_units` stage units
 * of 128 tokens of one KV head, into pieces: one static slice per CTA, then, for
 * sweeps long enough (or any sweep of at least two units per CTA with
 * draw_always != 0), chunks of halving size that CTAs draw from a counter.
 * This returns the number of pieces the kernels would use for (total_units,
 * n_ctas) and writes the first min(pieces, capacity) ranges [piece_begin[p],
 * piece_end[p]); it also checks that the kernels' position-to-piece map agrees
 * with the ranges.  Negative return: QF_ERR_BAD_SHAPE (arguments out of range,
 * or the two maps disagree), QF_ERR_NULL.  n_ctas is at most 160.
 */
int qf_plan_pieces(int total_units, int n_ctas, int draw_always, int32_t *piece_begin,
                   int32_t *piece_end, int capacity);

/*
 * Number of kernels the last enqueueing call of qf.h on this host thread
 * launched (for launch accounting in benchmarks).
 */
int qf_last_launch_count(void);

/*
 * While set, every qf_decode_partial on this host thread records `start_event`
 * just before and `stop_event` just after its sweep kernel on the call's stream,
 * so that a benchmark can time that one kernel live.  Both are cudaEvent_t
 * handles passed as void*; pass NULL, NULL to switch it off (the default).
 */
int qf_set_profile_events(void *start_event, void *stop_event);

/*
 * Host-made failure for tests of the projection pair's status plumbing: ORs
 * `bits` into the pair's status word in `workspace` exactly as a kernel whose
 * bounded wait ran out would, without any kernel waiting on anything.
 * Enqueues one tiny kernel on cuda_stream.
 */
int qf_project_status_inject(void *workspace, int32_t bits, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* QF_TESTING_H_ */
