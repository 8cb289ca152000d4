/*
 * speckv_internal.h -- entry points of libspeckv that are NOT part of its interface: a measurement
 * aid for the benchmark and two hooks for the library's own tests.  They are exported from the same
 * shared object, may change without notice, and nothing a user of the library does should call them.
 * (The paper has no counterpart for any of them.)
 */
#ifndef SPECKV_INTERNAL_H
#define SPECKV_INTERNAL_H

#include "speckv.h"

#ifdef __cplusplus
extern "C" {
#endif

/* speckv_step with three caller-created CUDA events (cudaEvent_t passed as void*) recorded on the
 * stream before the dominant kernel, after it, and after the kernel that draws the fresh tokens, so
 * that a benchmark can time the dominant kernel alone on the launching stream.  Where one launch does
 * the whole step the last two events coincide.  Results are identical to speckv_step.  Any event may
 * be NULL.                                                                                          */
speckv_status speckv_step_profiled(const speckv_batch* batch, const float* comp, const speckv_mlp* mlp,
                                   float* H, float* C, float* feat, float* scores,
                                   int32_t* gamma_next, int32_t* n_accepted, int32_t* out_tokens,
                                   int32_t* row_status, void* workspace, size_t workspace_bytes,
                                   void* cuda_stream, void* ev_before_sweep, void* ev_after_sweep,
                                   void* ev_after_resample);

/* Number of polls a CTA spends on a wait inside a kernel before it gives up and the row at hand gets
 * SPECKV_ROW_TIMEOUT (default 2^20).  Returns the previous value.  Process-wide; for tests.         */
int speckv_internal_set_wait_limit(int polls);

/* Runs the kernel that draws the fresh tokens on its own, one CTA per batch row, waiting for row
 * completion flags that nothing raises, followed by a row epilogue that arrives after the CTAs have
 * given up.  The waits must run out (the kernel returns), every row must end with
 * row_status == SPECKV_ROW_TIMEOUT and its two token slots at -1.  row_status: [B], out_tokens:
 * [B, 2], workspace: at least 8*B bytes, 256-byte aligned; all device memory.  B <= 4096.           */
speckv_status speckv_internal_wait_probe(int32_t B, int32_t* row_status, int32_t* out_tokens, void* workspace,
                                         size_t workspace_bytes, void* cuda_stream);

/* Bounds-checked build only (the library built with -DSPECKV_DEBUG, `python -m paper_2605_02888_b200.build
 * --debug`; the ordinary build returns SPECKV_ERR_UNSUPPORTED).  In that build every kernel compares the
 * address of each logit load and of each workspace access with the extents of the call's buffers, and
 * skips and counts an access that lies outside.  This call synchronises the device and returns
 * out4 = {violations so far, address of the first one, its size in bytes, its kind}; reset != 0 clears
 * the record afterwards; selftest != 0 first has a kernel check two addresses that no call registered
 * (they are only compared, never dereferenced), so that the record must then show violations.        */
speckv_status speckv_internal_debug_report(unsigned long long* out4, int reset, int selftest);

#ifdef __cplusplus
}
#endif
#endif
