// frog_exact_search: exact filtered kNN (paper Def. 2) by scanning each query's contiguous rank
// slab (Sec. 4).  One CTA per query; each warp streams batches of 16 consecutive rows through the
// same distance routine the beam search uses, keeps its own sorted top-k in shared memory, and
// warp 0 merges the per-warp lists at the end.  Ordering: (squared distance, original object id)
// ascending, the total order of Def. 2's tie rule (objects with equal attributes are ranked by id, so
// this differs from rank order only between equidistant objects with different attributes).
#include "frog_device.cuh"
#include "frog_internal.h"

using namespace frogdev;

namespace {

constexpr int EXACT_WARPS = 8;

struct ExactArgs {
    const int32_t* sorted_attr;
    const int32_t* rank2id;
    const float* vectors;
    int n, d, d_pad;
    const float* queries;
    const int32_t* lo;
    const int32_t* hi;
    int nq, k;
    int32_t* out_ids;
    float* out_dists;
};

template <int EPL>
__global__ void __launch_bounds__(EXACT_WARPS * 32)
frog_exact_kernel(const ExactArgs A) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int POOL = 32 * EPL;
    const int lane = lane_id();
    const int warp = threadIdx.x >> 5;
    const int q = blockIdx.x;
    float4* qs = reinterpret_cast<float4*>(smem_raw);
    uint64_t* pools = reinterpret_cast<uint64_t*>(smem_raw + (size_t)A.d_pad * 4);
    uint64_t* pool = pools + (size_t)warp * POOL;

    {
        float* qf = reinterpret_cast<float*>(qs);
        const float* src = A.queries + (size_t)q * A.d;
        for (int i = threadIdx.x; i < A.d_pad; i += blockDim.x) qf[i] = i < A.d ? __ldg(src + i) : 0.f;
        for (int i = lane; i < POOL; i += 32) pool[i] = KEY_EMPTY;
    }
    const int32_t lo = __ldg(A.lo + q), hi = __ldg(A.hi + q);
    int l_q, r_q;
    warp_rank_interval(A.sorted_attr, A.n, lo, hi, lane, l_q, r_q);
    const int w = (lo > hi) ? 0 : (r_q - l_q + 1);
    __syncthreads();

    for (int b0 = warp * 16; b0 < w; b0 += EXACT_WARPS * 16) {
        const int cnt = min(16, w - b0);
        const uint32_t rank = (uint32_t)(l_q + b0 + (lane & 15));
        float d2 = batch_dist2<4>(A.vectors, A.d_pad, qs, rank, cnt, lane);
        uint64_t key = KEY_EMPTY;
        if (lane < cnt) key = make_key(d2, (uint32_t)__ldg(A.rank2id + rank), 1u);   // keyed by object id
        // (merge_batch itself rejects candidates not better than the current k-th best)
        merge_batch<EPL>(pool, key, A.k, lane);
    }
    __syncthreads();
    if (warp == 0) {
        for (int ow = 1; ow < EXACT_WARPS; ++ow) {
            const uint64_t* other = pools + (size_t)ow * POOL;
            for (int j0 = 0; j0 < A.k; j0 += 32) {
                uint64_t key = (j0 + lane < A.k) ? other[j0 + lane] : KEY_EMPTY;
                merge_batch<EPL>(pool, key, A.k, lane);
            }
        }
        __syncwarp();
        for (int j = lane; j < A.k; j += 32) {
            uint64_t key = pool[j];
            int32_t oid = -1;
            float dist = __int_as_float(0x7F800000);
            if (key != KEY_EMPTY) {
                oid = (int32_t)key_rank(key);
                dist = __fsqrt_rn(key_dist2(key));
            }
            A.out_ids[(size_t)q * A.k + j] = oid;
            A.out_dists[(size_t)q * A.k + j] = dist;
        }
    }
}

typedef void (*exact_fn)(const ExactArgs);

}  // namespace

extern "C" int frog_exact_search(const frog_index_t* index, const float* queries, const int32_t* lo,
                                 const int32_t* hi, int nq, int k, int32_t* out_ids, float* out_dists,
                                 void* stream) {
    if (!index || nq < 0 || k < 1 || k > FROG_MAX_BEAM_WIDTH) return FROG_ERR_INVALID_ARG;
    if (nq == 0) return FROG_OK;
    if (!queries || !lo || !hi || !out_ids || !out_dists) return FROG_ERR_INVALID_ARG;
    FROG_CUDA_TRY(cudaSetDevice(index->info.device));
    exact_fn fn;
    int pool_slots;
    if (k <= 32) { fn = frog_exact_kernel<1>; pool_slots = 32; }
    else if (k <= 64) { fn = frog_exact_kernel<2>; pool_slots = 64; }
    else if (k <= 128) { fn = frog_exact_kernel<4>; pool_slots = 128; }
    else if (k <= 256) { fn = frog_exact_kernel<8>; pool_slots = 256; }
    else { fn = frog_exact_kernel<16>; pool_slots = 512; }
    size_t smem = (size_t)index->info.d_pad * 4 + (size_t)EXACT_WARPS * pool_slots * 8;
    FROG_CUDA_TRY(cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    ExactArgs A;
    A.sorted_attr = index->d_sorted_attr;
    A.rank2id = index->d_rank2id;
    A.vectors = index->d_vectors;
    A.n = (int)index->info.n;
    A.d = index->info.d;
    A.d_pad = index->info.d_pad;
    A.queries = queries;
    A.lo = lo;
    A.hi = hi;
    A.nq = nq;
    A.k = k;
    A.out_ids = out_ids;
    A.out_dists = out_dists;
    fn<<<nq, EXACT_WARPS * 32, smem, static_cast<cudaStream_t>(stream)>>>(A);
    FROG_CUDA_TRY(cudaGetLastError());
    return FROG_OK;
}
