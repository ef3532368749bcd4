/*
 * libmoe — hooks for the library's own tests.  Not part of the public interface:
 * nothing here belongs on a production path, and the paper has no counterpart
 * for any of it.  They exist so that the error paths of the library (a bounded
 * wait that runs out inside a kernel, scratch that does not fit) can be driven
 * without faulting, trapping or hanging a GPU and without exhausting its memory.
 */
#ifndef MOE_TEST_HOOKS_H_
#define MOE_TEST_HOOKS_H_

#include "moe.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Enqueue, on the handle's stream, one CTA that sets up the barrier block of the
 * grouped GEMMs, allocates tensor memory, and then waits with the GEMMs' own
 * bounded wait on a barrier nobody ever arrives on, with a limit of `limit_us`
 * microseconds (1 .. 100000) instead of the kernels' seconds.  The wait runs
 * out, the CTA takes the GEMMs' own abort path (abort flag, drain, release of
 * tensor memory) and sets the handle's device status word, exactly as a GEMM
 * whose pipeline stalled would.  If `poison_tail` is non-zero the call also
 * leaves non-zero arrival counters in the handle's K-slice buffer, as an aborted
 * small-batch GEMM may.  The next moe_device_status() (or any call that reads the
 * status) then returns MOE_ERR_DEVICE_TIMEOUT once, clears the status word and
 * the counters, and the handle is usable again.
 * Errors: MOE_ERR_INVALID_ARG, MOE_ERR_OOM, MOE_ERR_CUDA.
 */
int moe_test_wait_expiry(moe_layer_t* layer, unsigned limit_us, int poison_tail);

/*
 * Host side only.  Make every later scratch or weight allocation of this process
 * see at most `bytes` of free device memory (the library compares its request
 * with cudaMemGetInfo before it calls cudaMalloc), so that MOE_ERR_OOM can be
 * provoked without filling the device.  A negative value removes the limit.
 */
void moe_test_set_free_bytes_limit(long long bytes);

#ifdef __cplusplus
}
#endif
#endif /* MOE_TEST_HOOKS_H_ */
