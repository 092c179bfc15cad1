/* pyramidsd_diag.h -- measurement and self-test entry points of the verification library. Nothing a caller of the
 * verification path (pyramidsd.h) needs; benchmarks and tests use them. No counterpart in the paper. */
#ifndef PYRAMIDSD_DIAG_H_
#define PYRAMIDSD_DIAG_H_

#include "pyramidsd.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Per-kernel device timing for benchmarks. Between _begin and _end the library brackets each of its
 * kernel launches (on the calling thread) with CUDA events on the launch stream, up to 4096 launches.
 * _end synchronises those events, switches timing off, and returns the summed milliseconds and launch
 * counts of the row-statistics kernel and of the finalisation kernel (any output may be NULL). */
int pyramidsd_kernel_timing_begin(void);
int pyramidsd_kernel_timing_end(double* ms_rowstats, int* n_rowstats, double* ms_finalize, int* n_finalize);

/* Number of kernels the library has launched from this process since load (all entry points). */
uint64_t pyramidsd_launch_count(void);

/* The cluster size (CTAs per row pair) the library picks for a [B, K, V] stage of this dtype and the
 * number of such clusters the current device keeps resident at once; 0 and 0 when the shape takes the
 * baseline kernel. Lets a caller size batches to whole waves. Needs a CUDA device. */
int pyramidsd_cluster_occupancy(int B, int K, int V, psd_dtype dtype, int* out_cluster_size, int* out_max_active_clusters);

/* Self-test of the path by which a bounded device-side wait reports that it gave up. Launches one small kernel
 * on `cuda_stream` (NULL = the legacy default stream) in which a warp waits, for a few thousand polls, on a
 * shared-memory barrier that nothing ever signals; the wait runs out, the kernel records the fact in the
 * stream's status word exactly as the verification kernels do, and ends normally. Afterwards
 * pyramidsd_last_status() returns PSD_ERR_TIMEOUT once, and the stream and the library stay usable. Returns
 * PSD_OK when the kernel was launched. */
int pyramidsd_selftest_wait_timeout(void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* PYRAMIDSD_DIAG_H_ */
