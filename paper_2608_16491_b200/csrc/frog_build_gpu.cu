// GPU index builder: the construction of paper Sec. 6 with one warp per object and all objects
// of a layer in flight together (Sec. 6.2.1).  Per layer, bottom-up:
//   candidates   leaf: distances to every other object of the leaf, nearest 64 kept;
//                inner layer: the object's m nearest of its own child segment + the m best of a
//                greedy search (Alg. 1, pool ef_c, patience rule of Sec. 6.2.2) in the sibling's
//                temporary graph;
//   forward row  RNG selection of the candidates in vector-distance order;
//   reverse      the sources of an object's incoming forward edges join its candidates (nearest
//                64 of the union are kept);
//   final        nearest list (m), temporary graph row (RNG selection, vector order) and the
//                layer's ENC row (same selection in ascending fusion distance, Eq. 3).
// The selection needs d(c, p) between candidates: the <= 64 candidate rows of an object are staged
// in shared memory by bulk copies and all pair distances are accumulated there, so the selection
// itself is a loop over shared-memory look-ups.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <memory>
#include <numeric>
#include <vector>

#include <thrust/execution_policy.h>
#include <thrust/scan.h>

#include "frog_build_gpu.h"
#include "frog_device.cuh"
#include "frog_internal.h"

using namespace frogdev;

namespace {

constexpr int CAND = 64;                 // candidate slots per object
constexpr int BWARPS = 2;                // warps per CTA of the candidate / search / pool kernels
constexpr int STAGE8 = 8 * STAGE_CHUNK;  // stage buffer of staged_dist2<8>

__device__ __forceinline__ void segment_of(int n, int h, int x, int& L, int& R) {
    L = 0;
    R = n - 1;
    for (int depth = 0; depth < h; ++depth) {
        const int mid = L + ((R - L) >> 1);
        if (x <= mid) R = mid; else L = mid + 1;
    }
}

struct BuildArgs {
    const float* V;          // n x d_pad, rank order
    int n, d_pad, H, m, ef_c, patience;
    double beta, gamma, inv_span;
    uint64_t* c1;            // n x CAND keys (d2 bits << 32 | rank << 1 | 1), ascending, KEY_EMPTY tail
    uint64_t* c2;
    uint32_t* ann_cur; float* pd_cur; uint32_t* pg_cur;
    uint32_t* ann_nxt; float* pd_nxt; uint32_t* pg_nxt;
    uint32_t* fwd;           // forward graph rows of the layer under construction
    uint32_t* enc;           // n x H x m
    uint32_t* rev_cnt;       // n + 1
    uint32_t* rev_off;       // n + 1
    uint32_t* rev_cur;       // n
    uint32_t* rev_src;       // n x m
    uint32_t* bitmap;        // visited slabs of the sibling searches
    size_t bitmap_words;
    int h;                   // layer under construction
    int fusion_nearest;      // ENCs = the m fusion-nearest candidates (no RNG rule on them)
    int wait_limit;          // polls a wait on a bulk copy may take before giving up
    int skip_copies;         // test hook: expect the bytes but issue no copy, so that every wait runs out
    uint32_t* fail;          // set to 1 when a wait gave up: the build is not valid
};

// bounded wait on the bulk copies of a pass; records a give-up in *fail
__device__ __forceinline__ void wait_copies(const BuildArgs& A, uint64_t* bar, uint32_t phase) {
    if (!mbar_wait_limit(bar, phase, A.wait_limit)) *A.fail = 1u;
}

// shared-memory slice of one warp in the candidate / search / pool kernels
struct BWarp {
    float4* q;
    uint64_t* pool;      // CAND keys
    uint64_t* spool;     // search pool (sibling search only)
    uint32_t* cand;
    uint64_t* bar;
    float4* stage;
};
__host__ __device__ inline size_t bwarp_bytes(int d_pad, int spool_slots) {
    return (size_t)d_pad * 4 + CAND * 8 + (size_t)spool_slots * 8 + 32 * 4 + 16 + STAGE8;
}
__device__ __forceinline__ BWarp bwarp_carve(unsigned char* base, int d_pad, int spool_slots) {
    BWarp W;
    W.q = reinterpret_cast<float4*>(base);
    W.pool = reinterpret_cast<uint64_t*>(base + (size_t)d_pad * 4);
    W.spool = W.pool + CAND;
    W.cand = reinterpret_cast<uint32_t*>(W.spool + spool_slots);
    W.bar = reinterpret_cast<uint64_t*>(W.cand + 32);
    W.stage = reinterpret_cast<float4*>(W.bar + 2);
    return W;
}

__device__ __forceinline__ void load_query(const BuildArgs& A, const BWarp& W, int u, int lane) {
    const float4* src = reinterpret_cast<const float4*>(A.V + (size_t)u * A.d_pad);
    for (int i = lane; i < (A.d_pad >> 2); i += 32) W.q[i] = __ldg(src + i);
}

// distances of the ns (<= 32, pairwise distinct) ranks in W.cand to the query, as keys
__device__ __forceinline__ uint64_t cand_keys(const BuildArgs& A, const BWarp& W, int ns, uint32_t flag,
                                              uint32_t& phase, int lane) {
    const uint32_t id = lane < ns ? W.cand[lane] : 0u;
    float d2 = 0.f;
    bool ok = true;
    if (ns > 0) d2 = staged_dist2<8>(A.V, A.d_pad, W.q, W.stage, W.bar, phase, ok, id, ns, lane, A.wait_limit, !A.skip_copies);
    if (!ok) *A.fail = 1u;
    return lane < ns ? make_key(d2, id, flag) : KEY_EMPTY;
}

// ---- leaf layer: nearest CAND of the leaf -----------------------------------------------------
__global__ void __launch_bounds__(BWARPS * 32)
leaf_cand_kernel(const BuildArgs A) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    const BWarp W = bwarp_carve(smem_raw + bwarp_bytes(A.d_pad, 0) * warp, A.d_pad, 0);
    if (lane == 0) mbar_init(W.bar, 1u);
    __syncwarp();
    uint32_t phase = 0;
    const uint32_t lt_mask = (1u << lane) - 1u;
    const int nwarps = gridDim.x * BWARPS;
    for (int u = blockIdx.x * BWARPS + warp; u < A.n; u += nwarps) {
        int L, R;
        segment_of(A.n, A.H - 1, u, L, R);
        load_query(A, W, u, lane);
        W.pool[lane] = KEY_EMPTY;
        W.pool[lane + 32] = KEY_EMPTY;
        __syncwarp();
        for (int b0 = L; b0 <= R; b0 += 32) {
            const int v = b0 + lane;
            const bool keep = v <= R && v != u;
            const uint32_t M = __ballot_sync(FULL, keep);
            if (keep) W.cand[__popc(M & lt_mask)] = (uint32_t)v;
            __syncwarp();
            const uint64_t key = cand_keys(A, W, __popc(M), 1u, phase, lane);
            merge_batch<2>(W.pool, key, CAND, lane);
            __syncwarp();
        }
        A.c1[(size_t)u * CAND + lane] = W.pool[lane];
        A.c1[(size_t)u * CAND + lane + 32] = W.pool[lane + 32];
        __syncwarp();
    }
}

// ---- inner layer: own nearest list + greedy search in the sibling's graph (Alg. 1) ---------------
template <int EPL>
__global__ void __launch_bounds__(BWARPS * 32)
sibling_search_kernel(const BuildArgs A) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int SPOOL = 32 * EPL;
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    const BWarp W = bwarp_carve(smem_raw + bwarp_bytes(A.d_pad, SPOOL) * warp, A.d_pad, SPOOL);
    if (lane == 0) mbar_init(W.bar, 1u);
    __syncwarp();
    uint32_t phase = 0;
    const uint32_t lt_mask = (1u << lane) - 1u;
    uint32_t* bitmap = A.bitmap + (size_t)(blockIdx.x * BWARPS + warp) * A.bitmap_words;
    const int nwarps = gridDim.x * BWARPS;
    for (int u = blockIdx.x * BWARPS + warp; u < A.n; u += nwarps) {
        int L, R;
        segment_of(A.n, A.h, u, L, R);
        const int mid = L + ((R - L) >> 1);
        const int sL = u <= mid ? mid + 1 : L, sR = u <= mid ? R : mid;      // sibling child segment
        load_query(A, W, u, lane);
        W.pool[lane] = KEY_EMPTY;
        W.pool[lane + 32] = KEY_EMPTY;
        for (int i = lane; i < SPOOL; i += 32) W.spool[i] = KEY_EMPTY;
        __syncwarp();
        {   // the m nearest of the own child segment, found one layer below
            uint64_t key = KEY_EMPTY;
            if (lane < A.m) {
                const uint32_t id = A.ann_cur[(size_t)u * A.m + lane];
                if (id != BOT) key = make_key(A.pd_cur[(size_t)u * A.m + lane], id, 1u);
            }
            merge_batch<2>(W.pool, key, CAND, lane);
            __syncwarp();
        }
        if (sL <= sR) {
            for (int i = (sL >> 5) + lane; i <= (sR >> 5); i += 32) bitmap[i] = 0u;
            __syncwarp();
            const uint32_t ep = (uint32_t)(sL + ((sR - sL) >> 1));            // entry point: middle rank
            if (lane == 0) {
                atomicOr(bitmap + (ep >> 5), 1u << (ep & 31));
                W.cand[0] = ep;
            }
            __syncwarp();
            uint64_t key = cand_keys(A, W, 1, 0u, phase, lane);
            int first = (int)(merge_batch<EPL>(W.spool, key, A.ef_c, lane) & 0xFFFF);
            int pat = A.patience;
            for (int it = 0; first < A.ef_c && it < 4 * A.ef_c; ++it) {
                const uint32_t x = key_rank(W.spool[first]);
                const uint64_t mth = W.spool[A.m - 1];                         // m-th best before this expansion
                __syncwarp();
                if (lane == 0) W.spool[first] |= 1ull;
                uint32_t v = BOT;
                if (lane < A.m) v = __ldg(A.pg_cur + (size_t)x * A.m + lane);
                bool keep = false;
                if (v != BOT) {
                    const uint32_t bit = 1u << (v & 31);
                    keep = (atomicOr(bitmap + (v >> 5), bit) & bit) == 0;
                }
                const uint32_t M = __ballot_sync(FULL, keep);
                if (keep) W.cand[__popc(M & lt_mask)] = v;
                __syncwarp();
                key = cand_keys(A, W, __popc(M), 0u, phase, lane);
                const uint64_t best = warp_min_key(key);
                const bool improved = (best | 1ull) < (mth | 1ull);            // something enters the top m
                first = (int)(merge_batch<EPL>(W.spool, key, A.ef_c, lane) & 0xFFFF);
                if (improved) pat = A.patience;
                else if (--pat <= 0) break;
            }
            __syncwarp();
            key = KEY_EMPTY;
            if (lane < A.m) {
                key = W.spool[lane];
                if (key != KEY_EMPTY) key |= 1ull;
            }
            merge_batch<2>(W.pool, key, CAND, lane);
            __syncwarp();
        }
        A.c1[(size_t)u * CAND + lane] = W.pool[lane];
        A.c1[(size_t)u * CAND + lane + 32] = W.pool[lane + 32];
        __syncwarp();
    }
}

// ---- reverse edges of the forward graph ---------------------------------------------------------
__global__ void rev_count_kernel(const uint32_t* __restrict__ fwd, size_t edges, uint32_t* cnt) {
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < edges) {
        const uint32_t v = fwd[e];
        if (v != BOT) atomicAdd(cnt + v, 1u);
    }
}
__global__ void rev_fill_kernel(const uint32_t* __restrict__ fwd, size_t edges, int m, const uint32_t* __restrict__ off,
                                uint32_t* cur, uint32_t* src) {
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < edges) {
        const uint32_t v = fwd[e];
        if (v != BOT) src[off[v] + atomicAdd(cur + v, 1u)] = (uint32_t)(e / (size_t)m);
    }
}

// ---- candidates + sources of incoming edges, nearest CAND -----------------------------------------
__global__ void __launch_bounds__(BWARPS * 32)
pool_kernel(const BuildArgs A) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    const BWarp W = bwarp_carve(smem_raw + bwarp_bytes(A.d_pad, 0) * warp, A.d_pad, 0);
    if (lane == 0) mbar_init(W.bar, 1u);
    __syncwarp();
    uint32_t phase = 0;
    const int nwarps = gridDim.x * BWARPS;
    for (int u = blockIdx.x * BWARPS + warp; u < A.n; u += nwarps) {
        load_query(A, W, u, lane);
        W.pool[lane] = A.c1[(size_t)u * CAND + lane];
        W.pool[lane + 32] = A.c1[(size_t)u * CAND + lane + 32];
        __syncwarp();
        const uint32_t e1 = A.rev_off[u + 1];
        for (uint32_t e0 = A.rev_off[u]; e0 < e1; e0 += 32) {
            const int ns = (int)min(32u, e1 - e0);
            if (lane < ns) W.cand[lane] = A.rev_src[e0 + lane];
            __syncwarp();
            const uint64_t key = cand_keys(A, W, ns, 1u, phase, lane);
            merge_batch<2>(W.pool, key, CAND, lane);          // a source that is already a candidate is dropped
            __syncwarp();
        }
        A.c2[(size_t)u * CAND + lane] = W.pool[lane];
        A.c2[(size_t)u * CAND + lane + 32] = W.pool[lane + 32];
        __syncwarp();
    }
}

// ---- selection: pair distances among the candidates in shared memory, then the RNG rule ------------
struct SelSmem {
    uint64_t* keys;     // CAND
    float* D;           // CAND x CAND, upper triangle used
    float4* stage;      // CAND rows x STAGE_CHUNK bytes
    uint64_t* bar;
    int* ord;           // CAND: candidate indices in the visiting order
    int* kept;          // CAND
    int* pruned;        // CAND
    double* fus;        // CAND fusion distances
};
constexpr size_t SEL_BYTES = CAND * 8 + CAND * CAND * 4 + (size_t)CAND * STAGE_CHUNK + 16 + 3 * CAND * 4 + CAND * 8;

// visits ord[0..K) in order, keeps c iff d(u,c) < d(c,p) for every kept p, stops at m, back-fills
__device__ __forceinline__ int rng_rule(const SelSmem& S, int K, int m, int lane) {
    int nk = 0, np = 0;
    for (int t = 0; t < K && nk < m; ++t) {
        const int ci = S.ord[t];
        const float dc = key_dist2(S.keys[ci]);
        bool bad = false;
        if (lane < nk) {
            const int p = S.kept[lane];
            const float dcp = S.D[min(ci, p) * CAND + max(ci, p)];
            bad = !(dc < dcp);
        }
        const bool reject = __any_sync(FULL, bad);
        if (lane == 0) {
            if (reject) S.pruned[np] = ci; else S.kept[nk] = ci;
        }
        if (reject) ++np; else ++nk;
        __syncwarp();
    }
    for (int t = 0; t < np && nk < m; ++t) {
        if (lane == 0) S.kept[nk] = S.pruned[t];
        ++nk;
    }
    __syncwarp();
    return nk;
}

template <bool FINAL>
__global__ void __launch_bounds__(32)
select_kernel(const BuildArgs A) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SelSmem S;
    S.keys = reinterpret_cast<uint64_t*>(smem_raw);
    S.D = reinterpret_cast<float*>(S.keys + CAND);
    S.stage = reinterpret_cast<float4*>(S.D + CAND * CAND);
    S.bar = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(S.stage) + (size_t)CAND * STAGE_CHUNK);
    S.ord = reinterpret_cast<int*>(S.bar + 2);
    S.kept = S.ord + CAND;
    S.pruned = S.kept + CAND;
    S.fus = reinterpret_cast<double*>(S.pruned + CAND);
    const int lane = lane_id();
    const int team = lane >> 3, sub = lane & 7;
    if (lane == 0) mbar_init(S.bar, 1u);
    __syncwarp();
    uint32_t phase = 0;
    const uint64_t* cin = FINAL ? A.c2 : A.c1;
    const int row_bytes = A.d_pad * 4;
    for (int u = blockIdx.x; u < A.n; u += gridDim.x) {
        const uint64_t k0 = cin[(size_t)u * CAND + lane], k1 = cin[(size_t)u * CAND + lane + 32];
        S.keys[lane] = k0;
        S.keys[lane + 32] = k1;
        const int K = __popc(__ballot_sync(FULL, k0 != KEY_EMPTY)) + __popc(__ballot_sync(FULL, k1 != KEY_EMPTY));
        for (int i = lane; i < CAND * CAND; i += 32) S.D[i] = 0.f;
        __syncwarp();
        // pair distances, accumulated over column chunks of the rows
        for (int c0 = 0; c0 < row_bytes; c0 += STAGE_CHUNK) {
            const int cbytes = min(STAGE_CHUNK, row_bytes - c0);
            __syncwarp();
            if (lane == 0 && !A.skip_copies) mbar_expect_tx(S.bar, (uint32_t)(K * cbytes));
            __syncwarp();
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                const int r = lane + 32 * rr;
                if (r < K && !A.skip_copies)
                    tma_load_1d(reinterpret_cast<char*>(S.stage) + (size_t)r * STAGE_CHUNK,
                                reinterpret_cast<const char*>(A.V) + (size_t)key_rank(S.keys[r]) * row_bytes + c0,
                                (uint32_t)cbytes, S.bar);
            }
            wait_copies(A, S.bar, phase);
            phase ^= 1u;
            const int g_n = cbytes >> 4;
            for (int i = 0; i + 1 < K; ++i) {
                const float4* xi = S.stage + i * (STAGE_CHUNK / 16);
                for (int j0 = i + 1; j0 < K; j0 += 4) {
                    const int j = j0 + team;
                    float acc = 0.f;
                    if (j < K) {
                        const float4* xj = S.stage + j * (STAGE_CHUNK / 16);
                        for (int g = sub; g < g_n; g += 8) {
                            const float4 a = xi[g], b = xj[g];
                            float t;
                            t = a.x - b.x; acc = fmaf(t, t, acc);
                            t = a.y - b.y; acc = fmaf(t, t, acc);
                            t = a.z - b.z; acc = fmaf(t, t, acc);
                            t = a.w - b.w; acc = fmaf(t, t, acc);
                        }
                    }
                    acc += __shfl_xor_sync(FULL, acc, 4);
                    acc += __shfl_xor_sync(FULL, acc, 2);
                    acc += __shfl_xor_sync(FULL, acc, 1);
                    if (j < K && sub == 0) S.D[i * CAND + j] += acc;
                }
            }
        }
        __syncwarp();
        // temporary graph row: RNG rule in vector-distance order (the keys are already ascending)
        S.ord[lane] = lane;
        S.ord[lane + 32] = lane + 32;
        __syncwarp();
        int nk = rng_rule(S, K, A.m, lane);
        uint32_t* grow = (FINAL ? A.pg_nxt : A.fwd) + (size_t)u * A.m;
        if (lane < A.m) grow[lane] = lane < nk ? key_rank(S.keys[S.kept[lane]]) : BOT;
        if (FINAL) {
            if (lane < A.m) {
                const bool has = lane < K;
                A.ann_nxt[(size_t)u * A.m + lane] = has ? key_rank(S.keys[lane]) : BOT;
                A.pd_nxt[(size_t)u * A.m + lane] = has ? key_dist2(S.keys[lane]) : 0.f;
            }
            // ENC row: the same rule with the candidates in ascending fusion distance (Eq. 3)
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                const int i = lane + 32 * rr;
                if (i < K) {
                    const double dv = sqrt((double)key_dist2(S.keys[i]));
                    const double da = fabs((double)u - (double)key_rank(S.keys[i])) * A.inv_span;
                    const double za = A.gamma == 0.5 ? sqrt(da) : pow(da, A.gamma);   // sqrt is exact on both builders
                    S.fus[i] = dv * (1.0 - A.beta * (1.0 - za));
                }
            }
            __syncwarp();
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                const int i = lane + 32 * rr;
                if (i < K) {
                    const double fi = S.fus[i];
                    const uint32_t ri = key_rank(S.keys[i]);
                    int pos = 0;
                    for (int j = 0; j < K; ++j) {
                        const double fj = S.fus[j];
                        pos += (fj < fi || (fj == fi && key_rank(S.keys[j]) < ri)) ? 1 : 0;
                    }
                    S.ord[pos] = i;
                }
            }
            __syncwarp();
            if (A.fusion_nearest) {
                nk = min(K, A.m);                              // the paper's rule: the m fusion-nearest
                if (lane < nk) S.kept[lane] = S.ord[lane];
                __syncwarp();
            } else {
                nk = rng_rule(S, K, A.m, lane);
            }
            // store the kept candidates in ascending fusion distance (their position in ord)
            uint32_t* erow = A.enc + ((size_t)u * A.H + A.h) * A.m;
            int kpos = 0x7FFFFFFF;
            uint32_t krank = BOT;
            if (lane < nk) {
                const int ci = S.kept[lane];
                krank = key_rank(S.keys[ci]);
                for (int t = 0; t < K; ++t) if (S.ord[t] == ci) { kpos = t; break; }
            }
            int slot = 0;
            for (int j = 0; j < nk; ++j) {
                const int pj = __shfl_sync(FULL, kpos, j);
                slot += (pj < kpos) ? 1 : 0;
            }
            if (lane < A.m) erow[lane] = BOT;
            __syncwarp();
            if (lane < nk) erow[slot] = krank;
        }
        __syncwarp();
    }
}

// ---- host side ------------------------------------------------------------------------------------
bool write_all(FILE* f, const void* p, size_t bytes) {
    const char* c = static_cast<const char*>(p);
    while (bytes) {
        const size_t chunk = std::min<size_t>(bytes, (size_t)1 << 30);
        if (fwrite(c, 1, chunk, f) != chunk) return false;
        c += chunk;
        bytes -= chunk;
    }
    return true;
}
bool pad_to(FILE* f, uint64_t& pos, uint64_t target) {
    static const char zeros[128] = {0};
    while (pos < target) {
        const size_t c = (size_t)std::min<uint64_t>(target - pos, sizeof(zeros));
        if (fwrite(zeros, 1, c, f) != c) return false;
        pos += c;
    }
    return true;
}
inline uint64_t align128(uint64_t x) { return (x + 127) & ~(uint64_t)127; }

struct DeviceBuffers {
    std::vector<void*> ptrs;
    ~DeviceBuffers() { for (void* p : ptrs) cudaFree(p); }
    template <typename T> int alloc(T** out, size_t count) {
        void* p = nullptr;
        cudaError_t e = cudaMalloc(&p, count * sizeof(T));
        if (e != cudaSuccess) {
            cudaGetLastError();
            froghost::set_cuda_error(e);
            return FROG_ERR_NOMEM;
        }
        ptrs.push_back(p);
        *out = static_cast<T*>(p);
        return FROG_OK;
    }
};

int ceil_log2_i64(int64_t n) {
    int b = 0;
    while (((int64_t)1 << b) < n) ++b;
    return b;
}

}  // namespace

extern "C" int frog_index_build_gpu(const float* vectors, const int32_t* attrs, int64_t n64, int32_t d,
                                    const frog_build_params_t* params, int device, const char* path) {
    if (!vectors || !attrs || !path || n64 < 1 || d < 1 || n64 >= ((int64_t)1 << 31) - 1 || device < 0)
        return FROG_ERR_INVALID_ARG;
    frog_build_params_t P{};
    if (params) P = *params;
    else { P.n_inv = -1; P.beta = -1.f; }
    if (P.m == 0) P.m = d <= 300 ? 16 : 32;
    if (P.ef_c == 0) P.ef_c = d <= 300 ? 128 : 256;
    if (P.n_inv < 0) P.n_inv = d <= 300 ? 7 : 6;
    if (P.patience == 0) P.patience = 30;
    if (P.beta < 0) P.beta = 0.2f;
    if (P.gamma <= 0) P.gamma = 0.5f;
    if (P.m < 1 || P.ef_c < P.m || P.patience < 1) return FROG_ERR_INVALID_ARG;
    if (P.m > 32 || P.ef_c > 256) return FROG_ERR_UNSUPPORTED;
    const int n = (int)n64, m = P.m;
    int H = ceil_log2_i64(n64) + 1 - P.n_inv;
    if (H < 1) H = 1;
    const int d_pad = (d + 3) / 4 * 4;

    int dev_count = 0;
    FROG_CUDA_TRY(cudaGetDeviceCount(&dev_count));
    if (device >= dev_count) return FROG_ERR_INVALID_ARG;
    FROG_CUDA_TRY(cudaSetDevice(device));
    cudaDeviceProp prop;
    FROG_CUDA_TRY(cudaGetDeviceProperties(&prop, device));

    // Sec. 4: rank domain (host)
    std::vector<int32_t> rank2id((size_t)n);
    std::iota(rank2id.begin(), rank2id.end(), 0);
    std::stable_sort(rank2id.begin(), rank2id.end(), [&](int32_t a, int32_t b) { return attrs[a] < attrs[b]; });
    std::vector<int32_t> sorted_attr((size_t)n);
    std::unique_ptr<float[]> Vh(new (std::nothrow) float[(size_t)n * d_pad]);
    if (!Vh) return FROG_ERR_NOMEM;
    for (int64_t r = 0; r < n; ++r) {
        sorted_attr[r] = attrs[rank2id[r]];
        std::memcpy(Vh.get() + r * d_pad, vectors + (int64_t)rank2id[r] * d, sizeof(float) * d);
        for (int j = d; j < d_pad; ++j) Vh[r * d_pad + j] = 0.f;
    }

    DeviceBuffers buf;
    BuildArgs A{};
    float* dV = nullptr;
    int rc;
    const size_t nm = (size_t)n * m;
    uint32_t *annA, *annB, *pgA, *pgB;
    float *pdA, *pdB;
    if ((rc = buf.alloc(&dV, (size_t)n * d_pad)) || (rc = buf.alloc(&A.c1, (size_t)n * CAND)) ||
        (rc = buf.alloc(&A.c2, (size_t)n * CAND)) || (rc = buf.alloc(&annA, nm)) || (rc = buf.alloc(&annB, nm)) ||
        (rc = buf.alloc(&pgA, nm)) || (rc = buf.alloc(&pgB, nm)) || (rc = buf.alloc(&pdA, nm)) ||
        (rc = buf.alloc(&pdB, nm)) || (rc = buf.alloc(&A.fwd, nm)) || (rc = buf.alloc(&A.enc, nm * H)) ||
        (rc = buf.alloc(&A.rev_cnt, (size_t)n + 1)) || (rc = buf.alloc(&A.rev_off, (size_t)n + 1)) ||
        (rc = buf.alloc(&A.rev_cur, (size_t)n)) || (rc = buf.alloc(&A.rev_src, nm)) || (rc = buf.alloc(&A.fail, 1)))
        return rc;
    FROG_CUDA_TRY(cudaMemset(A.fail, 0, sizeof(uint32_t)));
    const bool reverse_edges = !(P.reserved & FROG_BUILD_NO_REVERSE_EDGES);
    A.fusion_nearest = (P.reserved & FROG_BUILD_ENC_FUSION_NEAREST) ? 1 : 0;
    // test hook (bits 16..31 of `reserved`): a nonzero value v makes every wait give up after v polls
    // and neither arms the barriers nor issues a copy, so that the give-up path runs with nothing in flight
    A.wait_limit = (P.reserved >> 16) ? (P.reserved >> 16) : (1 << 22);
    A.skip_copies = (P.reserved >> 16) ? 1 : 0;
    FROG_CUDA_TRY(cudaMemcpy(dV, Vh.get(), (size_t)n * d_pad * 4, cudaMemcpyHostToDevice));
    A.V = dV;
    A.n = n; A.d_pad = d_pad; A.H = H; A.m = m; A.ef_c = P.ef_c; A.patience = P.patience;
    A.beta = P.beta; A.gamma = P.gamma; A.inv_span = n > 1 ? 1.0 / (double)(n - 1) : 0.0;
    A.ann_cur = annA; A.ann_nxt = annB; A.pg_cur = pgA; A.pg_nxt = pgB; A.pd_cur = pdA; A.pd_nxt = pdB;

    // launch shapes
    const int spool_slots = P.ef_c <= 32 ? 32 : P.ef_c <= 64 ? 64 : P.ef_c <= 128 ? 128 : 256;
    const size_t smem_plain = bwarp_bytes(d_pad, 0) * BWARPS, smem_search = bwarp_bytes(d_pad, spool_slots) * BWARPS;
    void (*search_fn)(const BuildArgs) = spool_slots == 32 ? sibling_search_kernel<1>
                                       : spool_slots == 64 ? sibling_search_kernel<2>
                                       : spool_slots == 128 ? sibling_search_kernel<4> : sibling_search_kernel<8>;
    if (smem_search > 227 * 1024 || SEL_BYTES > 227 * 1024) return FROG_ERR_UNSUPPORTED;
    FROG_CUDA_TRY(cudaFuncSetAttribute((const void*)leaf_cand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_plain));
    FROG_CUDA_TRY(cudaFuncSetAttribute((const void*)pool_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_plain));
    FROG_CUDA_TRY(cudaFuncSetAttribute((const void*)search_fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_search));
    FROG_CUDA_TRY(cudaFuncSetAttribute((const void*)select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SEL_BYTES));
    FROG_CUDA_TRY(cudaFuncSetAttribute((const void*)select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SEL_BYTES));
    auto grid_for = [&](const void* fn, int threads, size_t smem, int per_cta) {
        int per_sm = 1;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, threads, smem);
        if (per_sm < 1) per_sm = 1;
        long long g = (long long)per_sm * prop.multiProcessorCount;
        const long long need = ((long long)n + per_cta - 1) / per_cta;
        return (int)std::max<long long>(1, std::min(g, need));
    };
    const int g_plain = grid_for((const void*)leaf_cand_kernel, BWARPS * 32, smem_plain, BWARPS);
    const int g_pool = grid_for((const void*)pool_kernel, BWARPS * 32, smem_plain, BWARPS);
    const int g_search = grid_for((const void*)search_fn, BWARPS * 32, smem_search, BWARPS);
    const int g_sel0 = grid_for((const void*)select_kernel<false>, 32, SEL_BYTES, 1);
    const int g_sel1 = grid_for((const void*)select_kernel<true>, 32, SEL_BYTES, 1);
    A.bitmap_words = (((size_t)n + 31) / 32 + 31) & ~(size_t)31;
    if (H > 1 && (rc = buf.alloc(&A.bitmap, (size_t)g_search * BWARPS * A.bitmap_words))) return rc;

    const size_t edges = nm;
    const int eb = 256, eg = (int)((edges + eb - 1) / eb);
    for (int h = H - 1; h >= 0; --h) {
        A.h = h;
        if (h == H - 1) leaf_cand_kernel<<<g_plain, BWARPS * 32, smem_plain>>>(A);
        else search_fn<<<g_search, BWARPS * 32, smem_search>>>(A);
        select_kernel<false><<<g_sel0, 32, SEL_BYTES>>>(A);
        FROG_CUDA_TRY(cudaMemsetAsync(A.rev_cnt, 0, ((size_t)n + 1) * 4));
        FROG_CUDA_TRY(cudaMemsetAsync(A.rev_cur, 0, (size_t)n * 4));
        if (reverse_edges) {
            rev_count_kernel<<<eg, eb>>>(A.fwd, edges, A.rev_cnt);
            thrust::exclusive_scan(thrust::device, A.rev_cnt, A.rev_cnt + n + 1, A.rev_off);
            rev_fill_kernel<<<eg, eb>>>(A.fwd, edges, m, A.rev_off, A.rev_cur, A.rev_src);
        } else {
            FROG_CUDA_TRY(cudaMemsetAsync(A.rev_off, 0, ((size_t)n + 1) * 4));      // no incoming sources
        }
        pool_kernel<<<g_pool, BWARPS * 32, smem_plain>>>(A);
        select_kernel<true><<<g_sel1, 32, SEL_BYTES>>>(A);
        FROG_CUDA_TRY(cudaGetLastError());
        std::swap(A.ann_cur, A.ann_nxt);
        std::swap(A.pd_cur, A.pd_nxt);
        std::swap(A.pg_cur, A.pg_nxt);
    }
    FROG_CUDA_TRY(cudaDeviceSynchronize());
    {
        uint32_t failed = 0;
        FROG_CUDA_TRY(cudaMemcpy(&failed, A.fail, sizeof(failed), cudaMemcpyDeviceToHost));
        if (failed) return FROG_ERR_CUDA;      // a bulk copy never completed: no file is written
    }

    std::unique_ptr<uint32_t[]> ench(new (std::nothrow) uint32_t[nm * H]);
    if (!ench) return FROG_ERR_NOMEM;
    FROG_CUDA_TRY(cudaMemcpy(ench.get(), A.enc, nm * H * 4, cudaMemcpyDeviceToHost));

    // the index file (same layout as the host builder writes)
    unsigned char hdr[256];
    std::memset(hdr, 0, sizeof(hdr));
    std::memcpy(hdr, "FROGIDX1", 8);
    const uint32_t u32s[8] = {1u, (uint32_t)d, (uint32_t)d_pad, (uint32_t)H, (uint32_t)m,
                              (uint32_t)P.n_inv, (uint32_t)P.ef_c, (uint32_t)P.patience};
    std::memcpy(hdr + 8, u32s, sizeof(u32s));
    std::memcpy(hdr + 40, &P.beta, 4);
    std::memcpy(hdr + 44, &P.gamma, 4);
    const uint64_t nn = (uint64_t)n;
    std::memcpy(hdr + 48, &nn, 8);
    std::memcpy(hdr + 56, &P.seed, 8);
    const uint32_t bot = BOT;
    std::memcpy(hdr + 64, &bot, 4);
    const uint32_t flags = (uint32_t)P.reserved & (FROG_BUILD_NO_REVERSE_EDGES | FROG_BUILD_ENC_FUSION_NEAREST);
    std::memcpy(hdr + 68, &flags, 4);
    const uint64_t off_attr = 256, off_r2i = align128(off_attr + nn * 4), off_vec = align128(off_r2i + nn * 4),
                   off_enc = align128(off_vec + nn * d_pad * 4), total = off_enc + nn * H * m * 4;
    const uint64_t offs[5] = {off_attr, off_r2i, off_vec, off_enc, total};
    std::memcpy(hdr + 72, offs, sizeof(offs));
    FILE* f = fopen(path, "wb");
    if (!f) return FROG_ERR_IO;
    uint64_t pos = 256;
    bool ok = write_all(f, hdr, 256) && write_all(f, sorted_attr.data(), (size_t)n * 4);
    pos += nn * 4;
    ok = ok && pad_to(f, pos, off_r2i) && write_all(f, rank2id.data(), (size_t)n * 4);
    pos += nn * 4;
    ok = ok && pad_to(f, pos, off_vec) && write_all(f, Vh.get(), (size_t)n * d_pad * 4);
    pos += nn * d_pad * 4;
    ok = ok && pad_to(f, pos, off_enc) && write_all(f, ench.get(), nm * H * 4);
    if (fclose(f) != 0) ok = false;
    return ok ? FROG_OK : FROG_ERR_IO;
}
