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

#ifdef __cplusplus
}
#endif
#endif /* LQ_TESTING_H_ */
