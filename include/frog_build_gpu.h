/* frog_build_gpu.h -- C ABI of the GPU index builder (exported by libfrog.so).
 *
 * Builds the same kind of index as frog_index_build (frog_build.h) with the per-object work of
 * the paper's construction (Sec. 6.1: brute-force leaves, then per layer the own-child
 * neighbours plus a greedy search, Alg. 1, in the sibling's temporary graph; RNG pruning; fusion
 * re-ranking, Eq. 3; patience early termination, Sec. 6.2.2) running as CUDA kernels, one warp
 * per object, all objects of a layer concurrently (the paper's intra-layer parallelism, Sec. 6.2.1).
 * The two builders follow the same steps in the same floating-point order with the same tie rules
 * ((delta_v, rank) and (delta_f, rank)), so they write the same file bit for bit (with the default
 * gamma = 0.5, where delta_a^gamma is a square root; for another gamma the two pow implementations
 * may disagree in the last place and exchange candidates that are that close).
 */
#ifndef FROG_BUILD_GPU_H_
#define FROG_BUILD_GPU_H_

#include <stdint.h>

#include "frog_build.h"

#ifdef __cplusplus
extern "C" {
#endif

/* frog_index_build_gpu: build the index of n objects on `device` and write it to `path`.
 *   vectors  HOST, n x d fp32 row-major, row i = object i
 *   attrs    HOST, n int32
 *   params   HOST, may be null; same meaning and defaults as frog_index_build (threads ignored).
 *            Limits of the kernels: m <= 32, ef_c <= 256, leaves of at most 256 objects.
 * Device memory: vectors + ENC array + about 1.2 KB per object of work space + n/8 bytes per
 * resident warp; everything is released before returning.  Returns 0 or a FROG_ERR_* code
 * (1 invalid argument, 2 I/O, 4 out of memory, 5 CUDA error, 6 unsupported parameters).  If a bulk
 * copy of a kernel does not complete within its polling limit the call returns 5 and writes no file.
 * Test hook: a nonzero value v in bits 16..31 of params->reserved makes the kernels issue no copy and
 * give up every wait after v polls, so that this report can be exercised without a fault. */
int frog_index_build_gpu(const float* vectors, const int32_t* attrs, int64_t n, int32_t d,
                         const frog_build_params_t* params, int device, const char* path);

#ifdef __cplusplus
}
#endif
#endif /* FROG_BUILD_GPU_H_ */
