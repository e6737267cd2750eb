/*
 * fpsk_test.h - entry points of libfpsk that exist for its tests and its benchmark, not for users.
 */
#ifndef FPSK_TEST_H
#define FPSK_TEST_H

#include "fpsk.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Self-test of the give-up path that every device-side wait of this library has (no counterpart in
 * the paper).  One thread waits for *d_flag (device, 4 bytes) to become non-zero, with a limit of about
 * half a millisecond instead of the library's usual second, then writes d_result->status: FPSK_OK if the
 * flag was set, FPSK_ERR_TIMEOUT if the wait gave up.  The kernel always returns; the context stays usable.
 * Asynchronous on `stream`. */
fpsk_status fpsk_selftest_bounded_wait(uint32_t *d_flag, fpsk_probe_result *d_result, void *stream);

/* Number of kernels launched by this library since load (all entry points, all threads). */
uint64_t fpsk_launch_count(void);

/* Number of auxiliary stream sets and pinned buffers the library has created by itself since load (calls made
 * with a context create none). */
uint64_t fpsk_lazy_resource_count(void);

/* The bounds-checked build of the library (compiled with -DFPSK_DEBUG_BOUNDS: every index a kernel takes from a
 * table is checked before it addresses memory; a bad one is recorded and the access skipped).  Returns 1 and the
 * number of violations since the last clear (with line, index and limit of the first one, and its source file)
 * from that build, 0 and *violations = -1 from the product build, -1 on a CUDA error.  Any pointer may be NULL.
 * Synchronises the device. */
int32_t fpsk_debug_bounds_report(int64_t *violations, int32_t *line, int64_t *index, int64_t *limit, char *file,
                                 size_t file_cap);
fpsk_status fpsk_debug_bounds_clear(void);

#ifdef __cplusplus
}
#endif
#endif /* FPSK_TEST_H */
