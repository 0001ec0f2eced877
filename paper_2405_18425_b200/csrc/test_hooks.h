/* Hooks for the library's own tests (exported from libvig_bigla.so, not part of the public C ABI:
 * include/vig_bigla.h does not declare them and applications must not call them).
 *
 * vig_test_set_kernel_preference: which kernel family the bf16 forward entry points use from now on,
 * process-wide and without any synchronisation against calls in flight on other threads.
 *   VIG_TEST_KERNEL_AUTO   the default dispatch
 *   VIG_TEST_KERNEL_SIMT   always the fp32 SIMT recurrence kernel
 *   VIG_TEST_KERNEL_CHUNK_TASKS  sequences of more than 256 tokens always take the three chunk-task launches
 *   VIG_TEST_KERNEL_SEGMENTS     sequences of 257 .. 8192 tokens always take the segmented single launch
 *                          (the default chooses between the two by segment count and unit count).
 *                          vig_bigla_workspace_bytes follows the setting: query it under the setting the call
 *                          will run with
 * Returns VIG_OK, or VIG_ERR_UNSUPPORTED for an unknown value (the setting is then unchanged). */
#ifndef VIG_TEST_HOOKS_H
#define VIG_TEST_HOOKS_H

#ifdef __cplusplus
extern "C" {
#endif

enum vig_test_kernel { VIG_TEST_KERNEL_AUTO = 0, VIG_TEST_KERNEL_SIMT = 2, VIG_TEST_KERNEL_CHUNK_TASKS = 3, VIG_TEST_KERNEL_SEGMENTS = 4 };
int vig_test_set_kernel_preference(int preference);

/* Synchronises `stream`, then returns and clears the number of (batch, head) units that the tensor-core kernels of the
 * current device handed to their in-kernel fp32 recurrence because a gate left the range of the factorised tiles
 * (negative: a vig_status error). */
int vig_test_take_fallback_count(void* stream);

/* The next launch of the single-block tensor-core kernel (sequences of at most 256 tokens) makes every block wait, with
 * a limit of a few dozen polls, on an mbarrier that nothing ever completes: the bounded wait runs out within
 * microseconds, the blocks finish their unit without storing anything, and vig_last_device_status reports
 * VIG_ERR_DEVICE_TIMEOUT.  Nothing faults and nothing spins beyond that limit. */
void vig_test_expire_next_wait(void);

#ifdef __cplusplus
}
#endif
#endif /* VIG_TEST_HOOKS_H */
