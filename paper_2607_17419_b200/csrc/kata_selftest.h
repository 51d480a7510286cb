/* Test-only entry point of libkata.so.  Not part of the public interface (include/kata.h): the tests call it to
 * check what a launch does when one of its bounded waits runs out. */
#ifndef KATA_SELFTEST_H
#define KATA_SELFTEST_H

#ifdef __cplusplus
extern "C" {
#endif

/* Launches one warp that waits, first with the time-bounded wait of the tensor-core kernels (0.1 s) and then with the
 * poll-bounded one (max_polls tries of at most 1 us each, 1 <= max_polls <= 2^20), on a barrier that nobody arrives
 * at.  Both waits give up; the kernel then writes KATA_ERR_DEVICE_TIMEOUT to *device_status (device pointer, may be
 * NULL) and {time-bounded wait gave up, poll-bounded wait gave up, abort flag} to report[0..2] (device pointer to
 * EIGHT ints, may be NULL), and runs the bounded wait on a flag in global memory (the one the CTAs of the single-launch
 * first-order scan publish their group states with) on report[7], which must be 0 on entry: report[3] = the wait for
 * the flag nobody sets gave up (2 ms limit), report[4] = the wait returned after the flag was published, report[5] =
 * the wait on the poisoned flag gave up, report[6] = and did so at once.  Nothing faults or traps and the context
 * stays usable.  The call is
 * asynchronous on `stream` (a cudaStream_t, NULL = the default stream); it allocates nothing.
 * Returns KATA_OK, KATA_ERR_INVALID_ARG (max_polls out of range) or KATA_ERR_CUDA (the launch failed). */
int kata_selftest_wait_timeout(int* device_status, int* report, unsigned max_polls, void* stream);

#ifdef __cplusplus
}
#endif
#endif
