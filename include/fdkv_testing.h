/*
 * Test hooks of libfdkv.  Not part of the product API (include/fdkv.h): nothing here computes a step of the method.
 * They let the test-suite reach two pieces of failure handling that a healthy run never enters, without making a GPU
 * fault, trap or hang.  (The paper has no counterpart.)
 */
#ifndef FDKV_TESTING_H
#define FDKV_TESTING_H

#include "fdkv.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Launches one thread block whose thread 0 waits, with the library's bounded mbarrier wait, on a barrier that nobody
 * ever arrives at, with a limit of `poll_cap` polls (1 .. 65536; a thousand polls take microseconds).  The wait runs
 * out, raises the block's abort flag and the context's device status word and the kernel returns normally: afterwards
 * fdkv_device_status(ctx) reports FDKV_ERR_TIMEOUT, exactly as after a copy that never landed in a decode or probe
 * kernel.  Nothing faults and nothing hangs; the context stays usable.  fdkv_test_clear_device_status resets the word.
 */
fdkv_status fdkv_test_wait_expiry(fdkv_ctx* ctx, int32_t poll_cap, void* stream);
fdkv_status fdkv_test_clear_device_status(fdkv_ctx* ctx, void* stream);

/*
 * The per-device set-up table of the launchers (function attributes are per device, not per process), driven with a
 * list of device ids instead of the current device: returns how many of the n visits `devs` (HOST) would run the
 * set-up on a fresh table.  Host only; no GPU is touched.
 */
int32_t fdkv_test_per_device_visits(const int32_t* devs /*HOST*/, int32_t n);

#ifdef __cplusplus
}
#endif
#endif /* FDKV_TESTING_H */
