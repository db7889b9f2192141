// Device-side building blocks of the FROG search kernels (sm_100a).  One warp owns one query;
// everything below is warp-synchronous and uses only that warp's slice of shared memory.
//
//   warp_count_below   attribute -> rank endpoint lookup (paper Sec. 4), 32-ary search
//   hotspot_layers     Alg. 3 HotspotLocalization with Eq. 6 evaluated in integers
//   en_identify        Alg. 4 ENIdentification: ballot/popc stream compaction under budget B
//   visited_insert     the hash check of Alg. 2 line 12 (lazy: applied to the compacted ENs)
//   batch_dist2        gather of <= 16 rows with 16-byte loads + fp32 squared L2, 8-lane teams
//   merge_batch        sort `new`, MergeTopEfS and "first unexpanded" of Alg. 2 lines 15-17
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace frogdev {

constexpr uint32_t FULL = 0xFFFFFFFFu;
constexpr uint64_t KEY_EMPTY = ~0ull;
constexpr uint32_t BOT = 0xFFFFFFFFu;         // empty ENC entry
constexpr uint32_t HASH_EMPTY = 0xFFFFFFFFu;
constexpr int HASH_MAX_PROBES = 24;
constexpr int NO_POS = 0x7FFFFFFF;

__device__ __forceinline__ int lane_id() { return (int)(threadIdx.x & 31); }

// Streaming 16-byte load: rows and ENC blocks are touched once per query, keep them out of L1.
__device__ __forceinline__ float4 ldg_stream_f4(const float4* p) {
    float4 v;
    asm("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
        : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint32_t ldg_stream_u32(const uint32_t* p) {
    uint32_t v;
    asm("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

// Pool key: (squared distance bits) << 32 | rank << 1 | expanded flag.  Distances are >= +0, so
// the fp32 bit pattern is monotone as an unsigned integer; ranks are unique, so comparing
// key >> 1 realises the total order (distance, rank) regardless of the flag.
__device__ __forceinline__ uint64_t make_key(float dist2, uint32_t rank, uint32_t flag) {
    return ((uint64_t)__float_as_uint(dist2) << 32) | ((uint64_t)rank << 1) | flag;
}
__device__ __forceinline__ uint32_t key_rank(uint64_t key) { return (uint32_t)(key & 0xFFFFFFFFull) >> 1; }
__device__ __forceinline__ float key_dist2(uint64_t key) { return __uint_as_float((uint32_t)(key >> 32)); }

// Number of elements of the ascending array a[0..n) that are < key (inclusive=false) or
// <= key (inclusive=true).  32-ary search: each round every lane probes the last element of one
// of 32 sub-blocks, a ballot finds the block holding the boundary.  ~log32(n) dependent loads.
__device__ __forceinline__ int warp_count_below(const int32_t* __restrict__ a, int n, int32_t key,
                                                bool inclusive, int lane) {
    int lo = 0, hi = n;
    while (hi > lo) {
        int len = hi - lo;
        int step = (len + 31) >> 5;
        int off = lane * step;
        bool pred = false;
        int last = lo + min(off + step, len) - 1;
        if (off < len) {
            int32_t v = __ldg(a + last);
            pred = inclusive ? (v <= key) : (v < key);
        }
        int c = __popc(__ballot_sync(FULL, pred));
        if ((long long)c * step >= len) {
            lo = hi;
        } else {
            hi = lo + min((c + 1) * step, len) - 1;
            lo = lo + c * step;
        }
    }
    return lo;
}

// Alg. 3.  Rule 1: descend while one child holds the whole range -> L_start.  Rule 2: extend
// L_end over consecutive layers h that satisfy Eq. 6,
//     (b_l - l_q) + (r_q - b_r) >= 2^-h (r_q - l_q),
// b_l = last rank of the layer-h segment holding l_q, b_r = (first rank of the one holding r_q) - 1.
__device__ __forceinline__ void hotspot_layers(int l_q, int r_q, int H, int N, int& L_start, int& L_end) {
    int L = 0, R = N - 1, d = 0;
    while (d < H - 1) {
        int mid = L + ((R - L) >> 1);
        if (r_q <= mid) R = mid;
        else if (l_q >= mid + 1) L = mid + 1;
        else break;
        ++d;
    }
    L_start = d;
    L_end = d;
    int Ll = L, Rl = R, Lr = L, Rr = R;
    for (int h = d + 1; h <= H - 1; ++h) {
        int mid = Ll + ((Rl - Ll) >> 1);
        if (l_q <= mid) Rl = mid; else Ll = mid + 1;
        mid = Lr + ((Rr - Lr) >> 1);
        if (r_q <= mid) Rr = mid; else Lr = mid + 1;
        long long lhs = (long long)(Rl - l_q) + (long long)(r_q - (Lr - 1));
        long long rhs = (long long)r_q - (long long)l_q;
        bool valid = h >= 31 ? (lhs > 0 || rhs == 0) : ((lhs << h) >= rhs);
        if (!valid) break;
        L_end = h;
    }
}

// Alg. 4.  The warp scans rows L_start..L_end of ENC(u) (contiguous: `total` entries at `hot`)
// in 32-entry chunks, two chunks fetched per round trip.  Predicate: entry != BOT and
// l_q <= entry <= r_q, evaluated as one unsigned compare (BOT - l_q exceeds any span since
// ranks are < 2^31).  Passing lanes get dense slots from ballot + popc; the budget admits a
// prefix.  Output: en[0..count) in shared memory (caller syncs), returns count; entries_scanned
// = end of the last chunk the scan needed.
__device__ __forceinline__ int en_identify(const uint32_t* __restrict__ hot, int total, uint32_t l_q,
                                           uint32_t span, int B, uint32_t* en, int lane,
                                           int& entries_scanned) {
    int cnt = 0;
    int scanned = 0;
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int c0 = 0; c0 < total; c0 += 64) {
        uint32_t v0 = BOT, v1 = BOT;
        if (c0 + lane < total) v0 = ldg_stream_u32(hot + c0 + lane);
        if (c0 + 32 + lane < total) v1 = ldg_stream_u32(hot + c0 + 32 + lane);
        {
            bool pred = (v0 - l_q) <= span;
            uint32_t M = __ballot_sync(FULL, pred);
            int n = __popc(M);
            int rank = __popc(M & lt_mask);
            int a = min(n, B - cnt);
            if (pred && rank < a) en[cnt + rank] = v0;
            cnt += a;
            scanned = min(total, c0 + 32);
        }
        if (cnt == B || c0 + 32 >= total) { if (cnt == B) break; else continue; }
        {
            bool pred = (v1 - l_q) <= span;
            uint32_t M = __ballot_sync(FULL, pred);
            int n = __popc(M);
            int rank = __popc(M & lt_mask);
            int a = min(n, B - cnt);
            if (pred && rank < a) en[cnt + rank] = v1;
            cnt += a;
            scanned = min(total, c0 + 64);
        }
        if (cnt == B) break;
    }
    entries_scanned = scanned;
    return cnt;
}

// Visited set: open addressing in shared memory, linear probing, full ranks stored (no false
// positives).  Returns true iff `id` was not present (and is now).  If the probe sequence is
// exhausted the home slot is overwritten: an older entry is forgotten, which can only cause a
// repeated distance evaluation -- merge_batch drops a candidate that is already in the pool, and
// one that was evicted from a full pool can never re-enter, so results are unaffected.
__device__ __forceinline__ bool visited_insert(uint32_t* tab, int bits, uint32_t id, uint32_t& forgets) {
    const uint32_t mask = (1u << bits) - 1u;
    const uint32_t home = (id * 0x9E3779B1u) >> (32 - bits);
    uint32_t s = home;
#pragma unroll 1
    for (int p = 0; p < HASH_MAX_PROBES; ++p) {
        uint32_t old = atomicCAS(tab + s, HASH_EMPTY, id);
        if (old == HASH_EMPTY) return true;
        if (old == id) return false;
        s = (s + 1) & mask;
    }
    tab[home] = id;
    ++forgets;
    return true;
}

// Squared L2 distances of up to 16 rows to the query held in shared memory.  Lane j < ns holds
// the rank of row j in `my_rank`; on return lane j holds its distance.
// Fixed arithmetic order (the CPU oracle mirrors it bit for bit): a row is cut into 4-float
// groups; a team of 8 lanes shares one row, lane s taking groups g = s, s+8, s+16, ... in
// increasing g with acc = fma(x - q, x - q, acc) element by element; then the 8 partial sums are
// combined by xor-butterfly with partner distance 4, 2, 1.
// Memory: the four teams of a warp fetch four different rows per instruction, each team reading
// 128 contiguous bytes (8 x 16-byte loads) -- whole 32-byte sectors only.  Up to 8 such loads
// are in flight per lane.
__device__ __forceinline__ float batch_dist2(const float* __restrict__ vectors, int d_pad,
                                             const float4* qs, uint32_t my_rank, int ns, int lane) {
    const int team = lane >> 3, sub = lane & 7;
    const int G = d_pad >> 2;
    const float4* row[4];
    bool valid[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        int vi = r * 4 + team;
        uint32_t id = __shfl_sync(FULL, my_rank, vi);
        valid[r] = vi < ns;
        row[r] = reinterpret_cast<const float4*>(vectors + (size_t)id * (size_t)d_pad);
    }
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int g0 = sub; g0 < G; g0 += 16) {
        float4 x[4][2];
        const bool second = (g0 + 8) < G;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            if (valid[r]) {
                x[r][0] = ldg_stream_f4(row[r] + g0);
                if (second) x[r][1] = ldg_stream_f4(row[r] + g0 + 8);
            }
        }
        const float4 q0 = qs[g0];
        float4 q1 = q0;
        if (second) q1 = qs[g0 + 8];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            if (valid[r]) {
                float t;
                t = x[r][0].x - q0.x; acc[r] = fmaf(t, t, acc[r]);
                t = x[r][0].y - q0.y; acc[r] = fmaf(t, t, acc[r]);
                t = x[r][0].z - q0.z; acc[r] = fmaf(t, t, acc[r]);
                t = x[r][0].w - q0.w; acc[r] = fmaf(t, t, acc[r]);
                if (second) {
                    t = x[r][1].x - q1.x; acc[r] = fmaf(t, t, acc[r]);
                    t = x[r][1].y - q1.y; acc[r] = fmaf(t, t, acc[r]);
                    t = x[r][1].z - q1.z; acc[r] = fmaf(t, t, acc[r]);
                    t = x[r][1].w - q1.w; acc[r] = fmaf(t, t, acc[r]);
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        acc[r] = acc[r] + __shfl_xor_sync(FULL, acc[r], 4);
        acc[r] = acc[r] + __shfl_xor_sync(FULL, acc[r], 2);
        acc[r] = acc[r] + __shfl_xor_sync(FULL, acc[r], 1);
    }
    // row j was handled by team j & 3 in round j >> 2
    float out = 0.f;
    const int src = (lane & 3) << 3;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        float v = __shfl_sync(FULL, acc[r], src);
        if ((lane >> 2) == r) out = v;
    }
    return out;
}

// Alg. 2 lines 15-17 in one pass.  `pool` holds ef_s (<= 32*EPL) keys ascending by key >> 1,
// KEY_EMPTY at the tail; each lane brings at most one new key (KEY_EMPTY = none).  The final
// position of a new key is (#pool keys below it) + (#new keys below it); of a pool key, its
// index + (#new keys below it); everything landing at >= ef_s is dropped.  A new key equal to a
// pool key (a vertex the visited table forgot) is discarded first.  Returns the first position
// whose flag is 0, NO_POS if none.  nk: 32 x u64 scratch.
template <int EPL>
__device__ __forceinline__ int merge_batch(uint64_t* pool, uint64_t* nk, uint64_t my_key, int ef_s, int lane) {
    int cpool = 0;
    if (my_key != KEY_EMPTY) {
        const uint64_t mk = my_key >> 1;
        int lo = 0, hi = ef_s;
        while (lo < hi) {
            int mid = (lo + hi) >> 1;
            if ((pool[mid] >> 1) < mk) lo = mid + 1; else hi = mid;
        }
        cpool = lo;
        if (lo >= ef_s || (pool[lo] >> 1) == mk) my_key = KEY_EMPTY;   // beyond the beam, or duplicate
    }
    nk[lane] = my_key;
    uint32_t have = __ballot_sync(FULL, my_key != KEY_EMPTY);
    __syncwarp();
    uint64_t pk[EPL];
    int add[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
        pk[e] = pool[lane + 32 * e];
        add[e] = 0;
    }
    int rnew = 0;
    const uint64_t mk = my_key >> 1;
    for (uint32_t msk = have; msk; msk &= msk - 1) {
        int j = __ffs(msk) - 1;
        uint64_t x = nk[j] >> 1;
        rnew += (x < mk) ? 1 : 0;
#pragma unroll
        for (int e = 0; e < EPL; ++e) add[e] += (x < (pk[e] >> 1)) ? 1 : 0;
    }
    __syncwarp();
    int first = NO_POS;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
        if (pk[e] != KEY_EMPTY) {
            int p = lane + 32 * e + add[e];
            if (p < ef_s) {
                if (add[e]) pool[p] = pk[e];
                if (!(pk[e] & 1ull)) first = min(first, p);
            }
        }
    }
    if (my_key != KEY_EMPTY) {
        int p = cpool + rnew;
        if (p < ef_s) {
            pool[p] = my_key;
            if (!(my_key & 1ull)) first = min(first, p);
        }
    }
    __syncwarp();
    return (int)__reduce_min_sync(FULL, (unsigned)first);
}

}  // namespace frogdev
