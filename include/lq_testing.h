/*
 * lq_testing.h -- hooks for the library's own tests.  Not part of the stable surface of lq.h:
 * nothing here is needed to run the pass.
 */
#ifndef LQ_TESTING_H_
#define LQ_TESTING_H_

#include <stdint.h>

#include "lq.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Every wait inside a kernel (on an mbarrier of the tensor-core contraction) gives up after a time
 * limit, records LQ_ERR_TIMEOUT in the handle's status word and lets the kernel return; the default
 * limit is five seconds.  This sets the limit of the kernels launched through `h` from now on
 * (0 restores the default), so that a test can make a wait of a healthy launch run out and check that
 * the call returns, the status is reported and the handle stays usable.  The results of a launch
 * whose wait ran out are unspecified. */
int lq_testing_set_wait_limit_ns(lq_handle* h, uint64_t ns);

/* Makes the failure those waits exist for, from the host: while `on` is nonzero, every load barrier of the
 * tensor-core contractions launched through `h` expects 16 bytes more than its loads deliver, so it never
 * completes -- a load that does not arrive.  Every wait in the kernel then runs into its limit (set a short one
 * first), the kernel records LQ_ERR_TIMEOUT, waits for the copies it has in flight, frees its tensor memory and
 * returns.  Nothing faults and nothing waits without limit. */
int lq_testing_inject_stall(lq_handle* h, int32_t on);

/* lq_prepare_hinv sends the updates of far tiles through the bf16 tensor cores (digit slices) only for matrices of
 * at least 48 blocks of 128 columns; smaller ones stay on the FP64 MMA throughout, which is faster there.  This sets
 * that threshold for `h` (0: always defer when there is more than one outer block of 1024 columns; negative: the
 * default), so that tests can run the deferred path on matrices small enough for a float64 check in full. */
int lq_testing_set_prepare_defer_min_blocks(lq_handle* h, int32_t n_blocks);

/* The deferred updates of lq_prepare_hinv multiply digit slices of their fp64 operands: as 8-bit integers on the integer
 * tensor-core path (the default) or, with on = 0, as bf16 values on the bf16 path.  Both are exact products; tests run
 * both and compare. */
int lq_testing_set_prepare_slices_int8(lq_handle* h, int32_t on);

#ifdef __cplusplus
}
#endif
#endif /* LQ_TESTING_H_ */
