/* frog_build.h -- C ABI of the FROG index builder (host tooling that produces the file the
 * search library loads).
 *
 * Follows the paper's Sec. 4 (attribute -> rank domain, implicit segment tree, n x H x m ENC
 * array), Sec. 5.2 (fusion distance, Eq. 3) and Sec. 6.1 (bottom-up construction: brute-force
 * leaves, then per layer the own-child graph neighbours plus a greedy search, Alg. 1, in the
 * sibling's temporary graph; the 2m candidates are RNG-pruned into the parent graph and
 * re-ranked by fusion distance into the layer's ENCs), with the patience rule of Sec. 6.2.2.
 * Every object works on at most 64 candidates per layer; m <= 32.
 * The search path never calls this; it only reads the file.
 */
#ifndef FROG_BUILD_H_
#define FROG_BUILD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
    int32_t m;         /* ENCs per vertex per layer; 0 = 16 if d <= 300 else 32 (Sec. 8.1.4) */
    int32_t ef_c;      /* pool width of construction-time searches; 0 = 128 / 256 */
    int32_t n_inv;     /* deepest layers omitted; -1 = 7 / 6 */
    int32_t patience;  /* consecutive non-improving iterations allowed; 0 = 30 */
    float beta;        /* Eq. 3; negative = 0.2 */
    float gamma;       /* Eq. 3; <= 0 = 0.5 */
    uint64_t seed;     /* recorded in the header (the build itself is deterministic) */
    int32_t threads;   /* worker threads; 0 = all cores.  The result does not depend on it. */
    int32_t reserved;  /* FROG_BUILD_* switches below, or 0 */
} frog_build_params_t;

/* Switches (bits of `reserved`, recorded in the file header at byte 68).  The builders add two steps
 * to the construction of Sec. 6.1; each bit removes one, both together give the section as written. */
#define FROG_BUILD_NO_REVERSE_EDGES 1   /* candidates are not extended by the sources of incoming edges */
#define FROG_BUILD_ENC_FUSION_NEAREST 2 /* ENCs = the m fusion-nearest candidates (no RNG rule on them) */
#define FROG_BUILD_LITERAL 3            /* both */

/* frog_index_build: build the index of n objects and write it to `path`.
 *   vectors  HOST, n x d fp32 row-major, row i = object i
 *   attrs    HOST, n int32, attribute of object i
 * Objects are ranked by (attribute, object id).  H = max(1, ceil(log2 n) + 1 - n_inv).
 * Returns 0, or 1 invalid argument, 2 I/O error, 4 out of memory (the FROG_ERR_* values of
 * frog.h).  The caller keeps ownership of its arrays. */
int frog_index_build(const float* vectors, const int32_t* attrs, int64_t n, int32_t d,
                     const frog_build_params_t* params, const char* path);

/* Fusion distance of Eq. 3: delta_v * (1 - beta * (1 - delta_a^gamma)), in double. */
double frog_fusion_distance(double delta_v, double delta_a, double beta, double gamma);

/* Retained depth for n objects and n_inv omitted layers. */
int32_t frog_retained_depth(int64_t n, int32_t n_inv);

#ifdef __cplusplus
}
#endif
#endif /* FROG_BUILD_H_ */
