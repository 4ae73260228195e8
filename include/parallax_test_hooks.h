/*
 * parallax_test_hooks.h -- entry points that exist for the library's own tests.  Not part of the
 * decode interface (that is parallax.h); nothing here computes attention.
 */
#ifndef PARALLAX_TEST_HOOKS_H_
#define PARALLAX_TEST_HOOKS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Makes a bounded device-side wait run out, on purpose and harmlessly.  Every kernel of the library
 * waits for its asynchronous copies with a bounded number of mbarrier polls; a wait that gives up sets
 * the status word to PLX_ERR_DEVICE_TIMEOUT and the kernel returns in an orderly way (no trap, the
 * context stays usable).  This hook launches one warp that initialises a barrier on which nothing ever
 * arrives (no copy is in flight), polls it `attempts` times (1 .. 65536) with the same wait routine
 * the kernels use, then writes PLX_ERR_DEVICE_TIMEOUT to `*status` (device int32) and `attempts` to
 * `*polls_done` (device int32, may be NULL) and returns.  One launch on `stream`.
 */
int plx_test_bounded_wait(int32_t* status, uint32_t attempts, int32_t* polls_done, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PARALLAX_TEST_HOOKS_H_ */
