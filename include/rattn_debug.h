/*
 * rattn_debug.h -- the one extra entry point of the DEBUG build of the library
 * (librattn_dbg.so: the same sources compiled with -DRATTN_DEBUG_KNOBS; librattn.so does
 * not export it and contains none of its code).
 *
 * Every device-side wait of the kernels is bounded: when one expires the kernel raises an
 * abort flag, every role stops, the CTA frees its tensor memory and returns, and the status
 * word of the workspace reads RATTN_ERR_TIMEOUT.  That path cannot be reached by valid
 * input, so the debug build offers a host-selected way to reach it without faulting
 * anything: while the switch is on, the tensor-core forward's first row group leaves out ONE
 * mbarrier arrival (a plain arrive with no asynchronous copy behind it) in the first work
 * unit of every CTA, and the waits of the debug build give up after 2^15 polls instead of
 * 2^21.  The paper has no counterpart; this exists for the failure-detection test.
 */
#ifndef RATTN_DEBUG_H_
#define RATTN_DEBUG_H_

#ifdef __cplusplus
extern "C" {
#endif

/* on != 0: the next tensor-core forwards withhold that arrival; 0: normal operation.
 * Process-wide switch, host side only.  Returns RATTN_OK. */
int rattn_debug_withhold_arrival(int on);

#ifdef __cplusplus
}
#endif
#endif /* RATTN_DEBUG_H_ */
