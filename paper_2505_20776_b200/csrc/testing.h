/*
 * Entry points of the TEST library (libspecext_testing.so, built with -DSPECEXT_TESTING).  They are
 * not part of the product ABI (include/specext.h) and the product library does not export them.
 */
#ifndef SPECEXT_TESTING_H_
#define SPECEXT_TESTING_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Forces, for every later call in the process, which attention kernel specext_verify_attn launches
 * and a lower bound on the 128-key tiles per worker:
 *   attn_kernel       : 0 = the product's choice; 1 = the CUDA-core cross-check kernel; 2 / 3 = the
 *                       one-CTA / paired-CTA tensor-core kernel (3 falls back to 2 for shapes the
 *                       paired kernel is not built for).
 *   min_tiles_per_cta : > 0 to change (fewer, longer splits).
 * Both change the workspace size: query specext_verify_attn_workspace after setting them.
 */
int specext_test_set_tuning(int32_t attn_kernel, int32_t min_tiles_per_cta);

/*
 * Launches a one-CTA kernel that waits, with the library's bounded mbarrier wait and the given limit
 * in SM cycles, on a barrier whose last arrival never comes.  The wait must run out, the kernel must
 * OR (1 << SPECEXT_ERR_TIMEOUT) into *device_status and return normally (no trap), leaving the
 * context usable.  Returns a specext_status for the launch.
 */
int specext_test_wait_timeout(int64_t limit_cycles, int32_t* device_status, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SPECEXT_TESTING_H_ */
