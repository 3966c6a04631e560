/* Self-test entry points of libspecpv: not part of the SpecPV path (the paper has no counterpart), kept
 * apart from specpv.h.  They exercise machinery of the kernels that ordinary inputs never reach. */
#ifndef SPECPV_SELFTEST_H
#define SPECPV_SELFTEST_H

#include "specpv.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Runs a one-CTA kernel on `stream` that initialises a shared-memory barrier on which nothing ever
 * arrives, waits on it through the very bounded wait the tensor-core kernels use, with a limit of
 * `limit_us` microseconds (1..1000000), and returns when the wait has given up: the kernel then
 * records SPECPV_ERR_TIMEOUT with info[0] = SPECPV_SELFTEST_WHERE in the workspace's status word,
 * raises its abort flag, frees the tensor memory it had allocated and exits.  Nothing faults or
 * hangs: the wait ends by construction.  workspace (device): at least SPECPV_WORKSPACE_HEAD_BYTES,
 * zeroed as for every other call.  observed_ns (device, nullable) receives how long the wait lasted.
 * Read the outcome with specpv_poll_status, which returns SPECPV_ERR_TIMEOUT and clears it. */
#define SPECPV_SELFTEST_WHERE 99
specpv_status specpv_selftest_wait_timeout(void *workspace, size_t workspace_bytes, int limit_us,
                                           unsigned long long *observed_ns, void *stream);

#ifdef __cplusplus
}
#endif
#endif
