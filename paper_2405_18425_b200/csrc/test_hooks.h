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

#ifdef __cplusplus
}
#endif
#endif /* VIG_TEST_HOOKS_H */
