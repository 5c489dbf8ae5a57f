/*
 * Test-only entry points of libgdn.  Not part of the public boundary (include/gdn.h): they exist so
 * that a test can run code paths that no valid input reaches.  Private to this source tree.
 */
#ifndef GDN_TEST_HOOKS_H_
#define GDN_TEST_HOOKS_H_

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Makes a bounded device-side wait run out, safely, and takes the failure path the prefill
 * kernels take: one CTA sets up an mbarrier that nobody ever arrives at and allocates tensor
 * memory; one warp waits on the barrier with a limit of `limit_cycles` SM clocks (pass a small
 * number, e.g. 20000) while two other warps wait on a second orphan barrier with the library's
 * normal (about one second) limit.  When the short wait gives up it raises the CTA's abort
 * flag; the other warps see the flag at their next poll and leave; every thread then runs the
 * common unwind (status word := 1, tensor memory released) and the kernel returns.  Nothing
 * faults, traps or waits without a limit.
 *
 *   status_word   DEVICE pointer to an int the caller has set to 0 (the same role as word 0 of a
 *                 prefill workspace; gdn_last_device_status reads and clears it)
 *   elapsed       DEVICE pointer to a long long: SM clocks the short wait took, or NULL
 * Returns GDN_OK once the kernel is enqueued.
 */
int gdn_test_bounded_wait(int* status_word, long long* elapsed, long long limit_cycles, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GDN_TEST_HOOKS_H_ */
