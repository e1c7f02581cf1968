/*
 * smartgen_testing.h -- test and measurement hooks of libsmartgen.so.  Not part of the hot path: nothing
 * here computes anything of the method, and a production caller never needs these calls.  They exist so
 * that tests can make a bounded device-side wait run out without hanging or faulting anything, and so
 * that the benchmark can read the SM clock a scoring kernel actually ran at.  The paper has no counterpart.
 *
 * All are process-wide switches read by the next call of the named entry point on any thread.
 */
#ifndef SMARTGEN_TESTING_H_
#define SMARTGEN_TESTING_H_

#include <stdint.h>

#include "smartgen.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * sg_testing_score_fault -- make the scoring kernel's bounded waits observable.
 *   withhold_unit   >= 0: pass-1 work items of this (layer * H_kv + kv_head) unit are computed but never counted
 *                   as done, so every pass-2 item of the unit waits for a count that never comes; -1: off.
 *   wait_limit_ms   > 0: every bounded wait in the kernel gives up after this many milliseconds (the wait for a
 *                   unit's count after twice that) instead of about a second; 0: the normal limits.
 * A wait that gives up sets the SG_ERR_TIMEOUT bit in the call's device status word; its CTA stops taking work,
 * waits (bounded) for its own outstanding copies and MMAs, frees its tensor memory and returns.  The importance
 * array is then only partly written.  Nothing traps and nothing spins without a limit.
 */
void sg_testing_score_fault(int32_t withhold_unit, int32_t wait_limit_ms);

/*
 * sg_testing_score_clock -- record the clock of the scoring kernel.  dev_buffer: device memory of at least
 * sg_testing_score_grid(shape) * 32 uint64 words (NULL switches the recording off).  CTA c of the next scoring
 * kernels writes words [32c .. 32c+3] (a library built without -DSG_SCORE_PROFILE packs them as [4c .. 4c+3]):
 * clock64() at its start and end, %globaltimer (ns) at its start and end.  (end - start) cycles / nanoseconds is
 * the SM clock in GHz the kernel really ran at, which a 200 ms nvidia-smi sample cannot show for a 0.2 ms kernel.
 */
void sg_testing_score_clock(void* dev_buffer);

/* Number of CTAs sg_score launches for this shape on a 148-SM device (the persistent grid). */
int32_t sg_testing_score_grid(const sg_shape* shape);

/*
 * sg_testing_decode_overlap -- allowed = 0: the following sg_sparse_decode_attn calls are launched without
 * programmatic stream serialization, i.e. fully ordered behind everything earlier in the stream, so that the
 * benchmark can report the time of a call that may not overlap its predecessor; 1 (the default) restores the
 * documented behaviour (a call overlaps the previous call up to its own output stores).
 */
void sg_testing_decode_overlap(int32_t allowed);

#ifdef __cplusplus
}
#endif
#endif /* SMARTGEN_TESTING_H_ */
