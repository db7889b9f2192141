/* frog.h -- C ABI of the FROG range-filtering k-ANN search library (CUDA, sm_100a).
 *
 * The calls follow the paper's problem statement (Sec. 2.1: objects (v_i, a_i), a query
 * (v_q, [l_q, r_q], k), L2 distance) and the argument list of its Alg. 2
 * FROGSearch(ENC, v_q, l_q, r_q, k, ef_s, epn, H, N, B).  All of the search runs in CUDA
 * kernels; there is no CPU fallback.  Nothing here throws, aborts or traps: every call
 * returns an int status (0 = FROG_OK) that frog_strerror() turns into text.
 *
 * Index file (little-endian): a 256-byte header
 *     char magic[8]="FROGIDX1"; u32 version=1, d, d_pad, H, m, n_inv, ef_c, patience;
 *     f32 beta, gamma; u64 n, seed; u32 bot=0xFFFFFFFF, reserved;
 *     u64 off_sorted_attr, off_rank2id, off_vectors, off_enc, file_bytes;
 * followed, at 128-byte-aligned offsets, by
 *     sorted_attr[n]   int32   attribute of the object of rank r, ascending (Sec. 4)
 *     rank2id[n]       int32   original object id of rank r
 *     vectors[n*d_pad] fp32    row r = vector of rank r, zero-padded to d_pad = 4*ceil(d/4)
 *     enc[n*H*m]       uint32  ENC block of rank r: H rows (layer 0 = root) of m ranks,
 *                              0xFFFFFFFF = empty (the n x H x m array of Sec. 4)
 */
#ifndef FROG_H_
#define FROG_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct frog_index frog_index_t; /* opaque; owns its device and host buffers */

enum {
    FROG_OK = 0,
    FROG_ERR_INVALID_ARG = 1,   /* null pointer, k < 1, k > beam_width, beam_width out of range ... */
    FROG_ERR_IO = 2,            /* file cannot be opened / read */
    FROG_ERR_FORMAT = 3,        /* magic, version, sizes or offsets inconsistent */
    FROG_ERR_NOMEM = 4,         /* host or device allocation failed */
    FROG_ERR_CUDA = 5,          /* a CUDA runtime call failed; see frog_last_cuda_error() */
    FROG_ERR_UNSUPPORTED = 6,   /* parameter combination the kernels do not cover */
    FROG_ERR_TOO_LARGE = 7      /* frog_search_static: the index exceeds FROG_STATIC_MAX_N objects */
};

/* Limits of the search kernels. */
#define FROG_MAX_BEAM_WIDTH 512 /* ef_s */
#define FROG_MAX_BUDGET 128     /* expansion budget B */
#define FROG_MAX_EPN 32         /* entry points */

typedef struct {
    int64_t n;          /* objects */
    int32_t d;          /* dimensionality of the data */
    int32_t d_pad;      /* floats per stored row (multiple of 4) */
    int32_t H;          /* retained layers of the segment tree (Sec. 4) */
    int32_t m;          /* ENCs per vertex per layer */
    int32_t n_inv;      /* deepest layers omitted */
    int32_t ef_c;       /* construction-time pool width */
    int32_t patience;   /* construction-time early-termination patience */
    float beta, gamma;  /* fusion-distance parameters (Eq. 3) used at construction */
    uint64_t seed;
    int32_t device;     /* CUDA device holding the index */
    int64_t device_bytes; /* bytes of device memory owned by the index */
} frog_index_info_t;

/* Optional query-time parameters (Alg. 2 arguments other than k and ef_s). */
typedef struct {
    int32_t epn;        /* entry points, 1..32; 0 = default 16 (paper Sec. 8.1.4) */
    int32_t budget;     /* expansion budget B, 1..128; 0 = default 16 */
    int32_t max_iters;  /* hard cap on expansions per query; 0 = default 16 * beam_width */
    int32_t no_hotspot; /* nonzero: scan all H layers instead of the hotspot (ablation) */
    uint64_t seed;      /* seed of the entry-point generator */
    int32_t hash_bits;  /* FROG_VISITED_HASH: log2 of the table slots; 0 = chosen from beam_width */
    int32_t visited;    /* FROG_VISITED_*: where the visited set lives */
    int32_t storage;    /* FROG_STORAGE_*: which copy of the vectors the gather reads */
    int32_t debug_flags;/* bit 0: with `trace`, record per-phase cycle counts instead of EN lists;
                           bit 1: process queries in input order (no heaviest-first planning pass);
                           bit 2: use the general kernel where a kernel specialised for the row size exists
                                  (same results; for comparing the two);
                           bit 3: use the visited hash table (see FROG_VISITED_AUTO) on small indexes too;
                           bit 4: record CUDA events around the search kernel alone (frog_search_kernel_ms);
                           bit 5: test of the error path: the kernel requests no row copy and its (bounded)
                                  waits give up after 64 polls, so every gather ends as a copy time-out would,
                                  with nothing in flight: the affected rows are padding, their status carries
                                  FROG_ST_COPY_TIMEOUT, frog_search_last_status reports it, and the next call
                                  works.  Honoured by the kernel for 384- and 512-byte rows (bitmap visited set,
                                  beam widths up to 32, budgets up to 64) and, when `stats` is given, by the
                                  general kernel; ignored otherwise;
                           bits 8-11: log2 of that table's slots, 6..12 (0 = 12), to make queries outgrow it */
    int32_t exact_below;/* ranges holding at most max(beam_width, exact_below) objects are answered by
                           scanning their contiguous rank slab (exact, status FROG_ST_EXACT) instead of
                           the graph search; 0 = default: only ranges that fit the pool.  Not in the
                           paper, whose smallest ranges hold thousands of objects (Sec. 8.1.2) */
    int32_t eager_hash; /* nonzero: ablation of the lazy hash check (Sec. 6.2): the visited test moves into
                           the predicate of Alg. 4, so evaluated ids neither take a slot nor consume
                           budget.  Bitmap visited form, fp32 storage and no trace only */
} frog_params_t;

/* Vector storage read by the search.  F32 (default): the index's fp32 rows.  F16: an fp16 copy made
 * by frog_index_enable_f16 (half the gathered bytes; values are converted back to fp32 and all
 * arithmetic stays fp32, so the result equals a search over the fp16-rounded vectors exactly; the
 * paper's own GPU programs read float16 data, Sec. 8.1.4).  F16 needs the bitmap visited form. */
#define FROG_STORAGE_F32 0
#define FROG_STORAGE_F16 1

/* Visited set (hashCheck of Alg. 2).  BITMAP: one bit per rank in a per-warp slab of device
 * scratch memory owned by the index (n/8 bytes per resident warp, allocated on first use, exact).
 * HASH: a bounded table in shared memory, no scratch; a crowded table drops entries, which repeats
 * distance evaluations but never changes results.  AUTO = BITMAP (HASH if the slabs do not fit);
 * for indexes of 4,194,304 objects and more searched with 384- or 512-byte rows and beam_width <= 64, AUTO
 * keeps the set in a 16 KB hash table of ranks per resident warp instead (exact; small enough to stay
 * in L2, where the bitmap of a large index costs a DRAM read-modify-write per candidate); a query
 * that fills half the table moves to its bitmap slab.  The results do not depend on the form. */
#define FROG_VISITED_AUTO 0
#define FROG_VISITED_BITMAP 1
#define FROG_VISITED_HASH 2

/* Per-query status bits written by frog_search_ex. */
#define FROG_ST_EMPTY 1u     /* lo > hi or no object in [lo, hi]: row is all padding */
#define FROG_ST_EXACT 2u     /* range holds <= max(beam_width, exact_below) objects: answered by exact scan */
#define FROG_ST_ITER_CAP 4u  /* expansion cap hit; the current pool was returned */
#define FROG_ST_SHORT 8u     /* fewer than k results; tail is padding */
#define FROG_ST_COPY_TIMEOUT 32u /* a bulk copy into shared memory did not complete within the kernel's
                                    polling limit; the row is written as padding (-1, +inf), with
                                    FROG_ST_SHORT set as well (never expected) */
#define FROG_ST_FORGOT 16u   /* the visited table overflowed and dropped entries: some distances were
                                evaluated twice; the results are unaffected */

/* frog_index_load: read an index file, copy its four arrays to `device`, return a handle.
 * (Paper Sec. 8.1.3: index and database stay resident in GPU memory.)  Host pointer in, the
 * handle is owned by the caller until frog_index_free.  Errors: INVALID_ARG, IO, FORMAT,
 * NOMEM, CUDA. */
int frog_index_load(const char* path, int device, frog_index_t** out);

/* frog_index_from_host: the same from arrays already in host memory (layout as in the file;
 * vectors are n x d_pad).  The arrays are copied; the caller keeps ownership of its own. */
int frog_index_from_host(const int32_t* sorted_attr, const int32_t* rank2id, const float* vectors,
                         const uint32_t* enc, const frog_index_info_t* shape, int device,
                         frog_index_t** out);

/* Release device and host memory of an index (null is allowed).  Synchronises the device. */
void frog_index_free(frog_index_t* index);

int frog_index_info(const frog_index_t* index, frog_index_info_t* out);

/* frog_index_enable_f16: add an fp16 copy of the vectors to the index (round to nearest even,
 * rows padded to a multiple of 8 elements; n * 2 * 8 * ceil(d / 8) more bytes of device memory).
 * Idempotent.  Searches select it with params->storage = FROG_STORAGE_F16. */
int frog_index_enable_f16(frog_index_t* index);

/* frog_search: batched FROGSearch (Alg. 2, with Alg. 3 once per query and Alg. 4 plus the lazy
 * hash check of Sec. 7.3.2 at every expansion), one query per warp of a persistent kernel.
 *   queries    DEVICE, nq x d fp32 row-major (d = index dimensionality)
 *   lo, hi     DEVICE, nq int32, inclusive attribute bounds of each query
 *   k          results per query, 1 <= k <= beam_width
 *   beam_width ef_s of Alg. 2, 1..FROG_MAX_BEAM_WIDTH
 *   out_ids    DEVICE, nq x k int32: ORIGINAL object ids, ascending (distance, rank); -1 padding
 *   out_dists  DEVICE, nq x k fp32: L2 distances (not squared), ascending; +inf padding
 *   stream     cudaStream_t (as void*); the call only enqueues work and returns
 * The caller owns all buffers and keeps them alive until the stream reaches the end of the
 * call.  One index may be searched from several streams and host threads at once: a launch
 * borrows one of up to four scratch sets owned by the index (work counter, visited slabs,
 * planning arrays); a stream keeps the set it used last, another stream gets an idle or a new
 * set, and when all four are busy the stream is made to wait for the one unused the longest.
 * Launches on different streams can therefore overlap on the GPU (the next batch fills the warps
 * that the last queries of the previous one leave idle).  The first call on a stream (and any
 * call that needs more resident warps than the calls before it) allocates visited slabs with
 * cudaMalloc after a device synchronise.  nq == 0 is a no-op.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA (launch failure).  Per-query conditions (empty range,
 * iteration cap, fewer than k results) are not errors; see frog_search_ex. */
int frog_search(const frog_index_t* index, const float* queries, const int32_t* lo, const int32_t* hi,
                int nq, int k, int beam_width, int32_t* out_ids, float* out_dists, void* stream);

/* frog_search_ex: frog_search with explicit parameters and optional per-query outputs.
 *   params  HOST, may be null (defaults)
 *   status  DEVICE nq uint32 or null: FROG_ST_* bits
 *   stats   DEVICE nq x 4 uint32 or null: {expansions, ENC rows the scan needed, ENs admitted
 *           by Alg. 4, distance evaluations}.  Asking for them selects a variant of the kernel
 *           that keeps these counters (a few per cent slower than the plain one; same results)
 *   trace   DEVICE nq x trace_cap uint32 or null: row q = [len, then per expansion
 *           u, |EN(u)|, EN(u)[0..]] (ranks); records are appended while at least 2 + max(64, B)
 *           words remain in the row.  Selects a slower kernel instantiation; meant for tests. */
int frog_search_ex(const frog_index_t* index, const float* queries, const int32_t* lo, const int32_t* hi,
                   int nq, int k, int beam_width, const frog_params_t* params,
                   int32_t* out_ids, float* out_dists, uint32_t* status, uint32_t* stats,
                   uint32_t* trace, int trace_cap, void* stream);

/* frog_exact_search: exact filtered kNN (Def. 2 of Sec. 2.1) by scanning the contiguous rank
 * slab of each query (Sec. 4: an attribute range is a contiguous rank interval), one CTA per
 * query.  Same buffers and conventions as frog_search; 1 <= k <= FROG_MAX_BEAM_WIDTH.  Used for ground truth
 * and as the pre-filtering reference. */
int frog_exact_search(const frog_index_t* index, const float* queries, const int32_t* lo, const int32_t* hi,
                      int nq, int k, int32_t* out_ids, float* out_dists, void* stream);

/* frog_search_host: the end-to-end call of the paper's timing scope (Sec. 8.1.3: transfer of
 * query vectors and ranges, then execution).  All pointers are HOST memory.  If all five buffers
 * are page-locked and device-mapped (cudaHostAlloc / cudaHostRegister) the kernels read the inputs
 * and write the results across the bus themselves, overlapping the transfers with the search;
 * otherwise the call copies in through staging buffers owned by the index (grown on first use),
 * searches and copies the results out.  Either way it returns after synchronising the stream. */
int frog_search_host(frog_index_t* index, const float* queries, const int32_t* lo, const int32_t* hi,
                     int nq, int k, int beam_width, const frog_params_t* params /* HOST, may be null */,
                     int32_t* out_ids, float* out_dists, void* stream);

/* frog_search_static: frog_search_ex (without the optional per-query outputs) for callers that
 * cannot allocate device memory at search time.  The paper has no counterpart; this entry point
 * exists for deployment reasons only.  Who needs it: a serving loop or a captured stream where the
 * device-wide synchronisation hidden in cudaMalloc/cudaFree is not acceptable; a plug-in that was
 * handed a fixed memory budget by its host application; a process that shares the GPU with
 * another framework's caching allocator, which has already claimed the free memory, so that an
 * allocation here would fail or fragment it.
 *
 * All scratch of the search (the work counter and the per-warp visited bitmaps) lives in one
 * file-scope device array inside the library, 16 MiB + 256 bytes, which every GPU that loads the
 * library holds until the process exits.  The call itself performs no cudaMalloc, cudaFree or
 * other allocating routine.  Consequences:
 *   - an index may hold at most FROG_STATIC_MAX_N objects, so that the bitmaps of at least
 *     FROG_STATIC_MIN_SLOTS warps fit; larger indexes are refused with FROG_ERR_TOO_LARGE.  The
 *     number of resident warps is capped by what fits, so large indexes run with less
 *     parallelism than frog_search gives them;
 *   - the first call on a device looks up the device address of the array (once per device,
 *     with that device current); make that first call before starting any stream capture;
 *   - every call, on every index and stream of the device, shares the one array, and the array
 *     keeps what the last call left in it.  The call resets the counter and each warp clears the
 *     bitmap words it is about to use, so consecutive calls are independent; calls that overlap
 *     on the GPU race on it and must be serialised by the caller.
 * Arguments, results and errors otherwise as frog_search_ex; `params` may be null;
 * params->visited is ignored (the bitmap form is always used). */
#define FROG_STATIC_MAX_N 2097152 /* objects: 256 KiB of visited bits per warp */
#define FROG_STATIC_MIN_SLOTS 64  /* resident warps guaranteed at FROG_STATIC_MAX_N */
int frog_search_static(const frog_index_t* index, const float* queries, const int32_t* lo, const int32_t* hi,
                       int nq, int k, int beam_width, const frog_params_t* params,
                       int32_t* out_ids, float* out_dists, void* stream);

/* FROG_ST_* conditions of the last frog_search / frog_search_ex / frog_search_host launch on `stream`
 * that concern the whole launch rather than one query: today FROG_ST_COPY_TIMEOUT (some row of the
 * result was written as padding because a bulk copy never completed; never expected).  Lets a caller
 * that passes no `status` array notice it.  Waits for that launch to finish.  INVALID_ARG if there
 * was no launch on the stream.  frog_search_static keeps no such word. */
int frog_search_last_status(const frog_index_t* index, void* stream, uint32_t* flags);

/* Device time, in milliseconds, of the search kernel of the last frog_search_ex call on `stream` that
 * was made with params->debug_flags bit 4 set (the call also runs two small planning kernels, which
 * this figure leaves out).  Waits for that kernel to finish.  INVALID_ARG if there was no such call. */
int frog_search_kernel_ms(const frog_index_t* index, void* stream, float* ms);

/* Launch shape of the search kernel for the given beam width (for reporting): CTAs, threads per
 * CTA, dynamic shared memory per CTA, query slots resident per SM. */
int frog_search_launch_info(const frog_index_t* index, int beam_width, const frog_params_t* params,
                            int* grid, int* block, int* smem_bytes, int* queries_per_sm);

const char* frog_strerror(int code);

/* cudaError_t value of the last failing CUDA call seen by this library on this thread. */
int frog_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FROG_H_ */
