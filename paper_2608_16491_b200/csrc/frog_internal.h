// Host-side definitions shared by the translation units of libfrog.so (not part of the ABI).
#pragma once

#include <cstdint>
#include <mutex>
#include <cuda.h>
#include <cuda_runtime.h>

#include "frog.h"

// One set of search scratch: the work counter of the persistent kernel (+ planning histogram), the
// per-warp visited slabs, the per-query planning arrays, and an event marking the end of the last
// launch that used the set.
struct FrogScratch {
    unsigned int* d_work = nullptr;  // 1 KB
    uint32_t* d_bitmap = nullptr;    // bitmap_slots x (words of visited bits + log of evaluated ranks)
    size_t bitmap_slots = 0;
    uint32_t* d_table = nullptr;     // table_slots visited hash tables of FROG_TABLE_SLOTS ranks (all 0xFFFFFFFF at rest)
    size_t table_slots = 0;
    int table_bits = 0;              // log2 of the ranks per table of the last launch
    size_t table_bytes = 0;
    int32_t* d_plan = nullptr;       // per query: rank interval (2 ints) and processing order (1 int)
    size_t plan_queries = 0;
    cudaEvent_t done = nullptr;
    cudaEvent_t k_begin = nullptr, k_end = nullptr;   // around the search kernel of the last timed launch
    bool k_timed = false;
    cudaStream_t stream = nullptr;   // stream of the last launch
    unsigned long long tick = 0;
};
constexpr int FROG_SCRATCH_SETS = 4;
constexpr int FROG_TABLE_BITS = 12;    // 4,096 ranks = 16 KB per resident warp: 78 MB for a full grid, inside L2
constexpr int FROG_TABLE_BITS_WIDE = 13;   // beam widths 65..128: 8,192 ranks (a query evaluates ~2,000 there)

struct frog_index {
    frog_index_info_t info;
    int32_t* d_sorted_attr = nullptr;
    int32_t* d_rank2id = nullptr;
    float* d_vectors = nullptr;      // n x d_pad, rank order
    void* d_vectors_h = nullptr;     // optional fp16 copy, n x d_pad_h (d_pad_h = 8 * ceil(d / 8))
    uint32_t* d_enc = nullptr;       // n x H x m
    // Scratch of the search launches.  A launch borrows one set; sets are handed out so that launches
    // on different streams never share one while either may still be running (see acquire_scratch).
    FrogScratch scratch[FROG_SCRATCH_SETS];
    int n_scratch = 0;
    unsigned long long tick = 0;     // launch counter, for least-recently-used selection
    std::mutex mu;                   // guards the scratch sets and the order of launches into them
    // Tensor maps of the two row stores for the 4-row gather of the copy engine (box = one row or
    // one 512-byte column chunk of it); absent when the driver entry point is missing or the row
    // shape does not qualify, in which case rows are copied one by one.
    CUtensorMap tmap_f32, tmap_f16;
    bool has_tmap_f32 = false, has_tmap_f16 = false;
    // staging for frog_search_host, grown on demand
    void* d_stage = nullptr;
    size_t stage_bytes = 0;
    std::mutex stage_mu;             // one staged host call at a time
    int sm_count = 0;
};

// Arguments of the search kernel (passed by value).
struct FrogSearchArgs {
    const int32_t* sorted_attr;
    const int32_t* rank2id;
    const float* vectors;
    const uint32_t* enc;
    int n, d, d_pad, H, m;
    const float* queries;
    const int32_t* lo;
    const int32_t* hi;
    int nq, k, ef_s, epn, B, max_iters, no_hotspot, hash_bits;
    int exact_w;               // ranges of at most this many objects are scanned exactly (>= ef_s)
    unsigned long long seed;
    int32_t* out_ids;
    float* out_dists;
    uint32_t* status;
    uint32_t* stats;
    uint32_t* trace;
    int trace_cap;
    unsigned int* work_counter;
    uint32_t* bitmap;          // visited slabs, or null when the shared-memory table is used
    size_t bitmap_words;       // words of visited bits per slab
    size_t slab_stride;        // words from one warp's slab to the next (bits, then the log of evaluated ranks)
    int log_cap;               // entries of the per-warp log of evaluated ranks that follows the bits (0: none)
    int slab_clean;            // nonzero: every slab is all-zero between queries (the kernel restores that
                               // when a query ends); zero: a query clears the words of its range before use
    uint32_t* table;           // visited hash tables (1 << table_bits ranks per resident warp, all empty
                               // between queries), or null
    int table_bits;
    const int2* ranges;        // precomputed [l_q, r_q] per query, or null: computed in the kernel
    const int32_t* order;      // processing order (heaviest first), or null: input order
    const void* rows;          // gather source: fp32 vectors, or their fp16 copy
    int row_bytes;             // bytes per stored row
    int slot_bytes;            // bytes of one row slot in the stage buffer (multiple of 16, <= 512)
    int q_len;                 // floats of the query held in shared memory (8 * ceil(d / 8))
    int gather4;               // nonzero: `tmap` is valid and rows are fetched four per copy instruction
    int no_copies;             // test hook of the counting variant: no row copy is armed or issued, waits give up
                               // after 64 polls (every gather takes the time-out branch, nothing is in flight)
    alignas(64) CUtensorMap tmap;
};

typedef void (*frog_kernel_fn)(const FrogSearchArgs);

namespace froghost {
// frog_search_lean.cu: the trimmed kernel for 384- and 512-byte fp32 rows (null: shape not covered)
frog_kernel_fn lean_kernel(int ef_s, int budget, int row_bytes, bool table, bool hook, size_t* smem_per_warp,
                           int* warps_per_cta);
void set_cuda_error(cudaError_t e);
int resolve_params(const frog_index* ix, int beam_width, const frog_params_t* in, frog_params_t* out);
bool make_row_tensor_map(const void* base, bool f16, int row_elems, size_t row_bytes, size_t n, CUtensorMap* out);
int acquire_scratch(frog_index* ix, cudaStream_t s, FrogScratch** out);
int ensure_bitmap(const frog_index* ix, FrogScratch* sc, size_t slots);
int ensure_table(FrogScratch* sc, size_t slots, int bits);
int ensure_plan(FrogScratch* sc, size_t nq);
}  // namespace froghost

#define FROG_CUDA_TRY(expr)                                  \
    do {                                                     \
        cudaError_t _e = (expr);                             \
        if (_e != cudaSuccess) {                             \
            froghost::set_cuda_error(_e);                    \
            return FROG_ERR_CUDA;                            \
        }                                                    \
    } while (0)
