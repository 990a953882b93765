/*
 * sdq_diag.h -- measurement and self-test aids of the SDQ library (no counterpart in the paper; not part of the
 * method's C-ABI in sdq.h).  Same conventions as sdq.h: plain pointers, status codes, nothing allocates.
 */
#ifndef SDQ_DIAG_H_
#define SDQ_DIAG_H_

#include "sdq.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Measurement aid: enqueues a copy-only kernel in which every SM keeps `nslot` bulk
 * copies of `slot_bytes` in flight from its own region of `src` (device, 16-byte aligned; walked cyclically) into
 * shared memory, `iters` copies per SM, nothing consuming them.  *bytes_moved receives the bytes the launch stages
 * in total; the caller times the launch with events.  With a source smaller than L2 this is the ceiling of the
 * L2 -> shared-memory path that bounds the many-token product kernel.
 *   slot_bytes a multiple of 128, >= 1024; nslot 1..16; nslot * slot_bytes <= 220 KB; src_bytes / #SMs >= slot_bytes;
 *   issuers 1..4: threads per SM that issue the copies (the slots are dealt out over them).
 *   Asynchronous on `stream`.  Errors: INVALID_ARG, ALIGNMENT, SHAPE, CUDA; a bounded wait that gives up sets the
 *   sticky device status. */
sdq_status_t sdq_diag_l2_copy(const void* src, size_t src_bytes, int slot_bytes, int nslot, int issuers, int iters,
                              size_t* bytes_moved, void* stream);


/* Self-test of the failure detection: every device-side wait of the library is bounded and reports through the sticky
 * status word instead of hanging.  This enqueues a one-thread kernel that waits, for at most `polls` polls (1 .. 4096),
 * on a shared-memory barrier that nothing ever completes; the wait gives up, the kernel sets the status word and
 * returns.  sdq_device_status(stream) then returns SDQ_ERR_TIMEOUT once (and clears it).  Nothing traps, nothing hangs,
 * the context stays usable.  Asynchronous on `stream`.  Errors: SHAPE (polls out of range), CUDA. */
sdq_status_t sdq_diag_wait_timeout(int polls, void* stream);

#ifdef __cplusplus
}
#endif

#endif /* SDQ_DIAG_H_ */
