/*
 * rbs_selftest.h -- operational self-tests of the RBS prefill library (no counterpart in the paper).
 *
 * These entry points exercise the library's own safety machinery without disturbing the GPU: nothing here
 * faults, traps or spins without a limit.
 */
#ifndef RBS_SELFTEST_H_
#define RBS_SELFTEST_H_

#include "rbs.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Host only, needs no GPU.  Checks the table through which per-device values (the device address of the
 * status word, the SM count) are looked up once per device and never shared between devices, using a fake
 * lookup.  Returns 0 when every check passes, otherwise the number of the first failed check.
 */
RBS_API int rbs_selftest_device_table(void);

/*
 * Launches one single-thread CTA on `stream` that waits, with the library's bounded mbarrier wait, on a barrier
 * that nothing ever arrives on, with `spin_limit` probes (1 .. 65536) instead of the production limit.  The wait
 * runs out, records its code in the device status word and the kernel returns normally: afterwards
 * rbs_device_status() reports RBS_ERR_TIMEOUT until cleared, *gave_up (device, one uint32) is 1, and the CUDA
 * context is fully usable.  Returns RBS_ERR_INVALID_ARG for a null pointer or a limit outside the range.
 */
RBS_API rbs_status rbs_selftest_wait_timeout(unsigned int spin_limit, unsigned int* gave_up, void* stream);

/*
 * Debug build only (the library compiled with -DRBS_DEBUG; rbs_version() says "debug checks"): launches one thread
 * on `stream` that runs one of the kernels' index checks with an index equal to its bound.  The check fails, records
 * 0x100 + 0xff in the device status word and the guarded access is skipped: afterwards *skipped (device, one
 * uint32) is 1, rbs_device_status() reports RBS_ERR_DEBUG_CHECK until cleared, and the CUDA context is fully usable
 * (nothing traps or faults).  The release build has no such checks and returns RBS_ERR_UNSUPPORTED without a launch.
 */
RBS_API rbs_status rbs_selftest_debug_check(unsigned int* skipped, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RBS_SELFTEST_H_ */
