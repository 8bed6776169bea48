/*
 * pevlm_trace.h -- optional tracing facility of libpevlm.so (not part of the product ABI).
 *
 * A library built with -DPEVLM_TRACE (PEVLM_TRACE=1 python -m paper_2506_19651_b200.build --force) compiles
 * clock64 time stamps into the attention kernel at the hand-offs between its roles (scores seen by the
 * softmax, probabilities handed to the MMA warp, MMA issue, work-item boundaries) for thread block 0 and
 * exports the two read-back calls below; `python -m paper_2506_19651_b200.timeline` prints the intervals.
 * A library built without the flag has neither the stamps nor these symbols.
 */
#ifndef PEVLM_TRACE_H_
#define PEVLM_TRACE_H_
#ifdef __cplusplus
extern "C" {
#endif

/* host_out: 8 x 16 words, [event][key tile - 8] of thread block 0's first work item.  Returns 0 or -1. */
int pevlm_debug_trace(unsigned* host_out);
/* host_out: 8 x 16 words, [event][work item - 2] of thread block 0's work items 2..17.  Returns 0 or -1. */
int pevlm_debug_trace_items(unsigned* host_out);

#ifdef __cplusplus
}
#endif
#endif /* PEVLM_TRACE_H_ */
