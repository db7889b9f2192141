// Device-side building blocks of the FROG search kernels (sm_100a).  One warp owns one query;
// everything below is warp-synchronous and uses only that warp's slice of shared memory.
//
//   warp_rank_interval attribute -> rank endpoint lookup (paper Sec. 4), two 32-ary searches
//   hotspot_layers     Alg. 3 HotspotLocalization with Eq. 6 evaluated in integers
//   visited_insert     the hash check of Alg. 2 line 12
//   batch_dist2        gather of <= 16 rows with 16-byte loads + fp32 squared L2, 8-lane teams
//   staged_dist2       the same distances with the rows staged in shared memory by TMA bulk copies
//   merge_batch        sort `new`, MergeTopEfS and "first unexpanded" of Alg. 2 lines 15-17
#pragma once

#include <cstdint>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

namespace frogdev {

constexpr uint32_t FULL = 0xFFFFFFFFu;
constexpr uint64_t KEY_EMPTY = ~0ull;
constexpr uint32_t BOT = 0xFFFFFFFFu;         // empty ENC entry
constexpr uint32_t HASH_EMPTY = 0xFFFFFFFFu;
constexpr int HASH_MAX_PROBES = 16;
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
// L2 eviction policies for a whole access.  Short vector rows are read about once per batch and
// should leave L2 first (long rows are kept at normal priority: their popular rows are worth
// 4 % when they stay); the visited slab of a query is hit again and again and should stay.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_normal() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint32_t atomic_or_l2(uint32_t* p, uint32_t v, uint64_t policy) {
    uint32_t old;
    asm volatile("atom.global.or.b32.L2::cache_hint %0, [%1], %2, %3;" : "=r"(old) : "l"(p), "r"(v), "l"(policy) : "memory");
    return old;
}
__device__ __forceinline__ void st_u32_l2(uint32_t* p, uint32_t v, uint64_t policy) {
    asm volatile("st.global.L2::cache_hint.u32 [%0], %1, %2;" ::"l"(p), "r"(v), "l"(policy) : "memory");
}

// Pool key: (squared distance bits) << 32 | rank << 1 | expanded flag.  Distances are >= +0, so
// the fp32 bit pattern is monotone as an unsigned integer; ranks are unique, so comparing
// key | 1 realises the total order (distance, rank) regardless of the flag.
__device__ __forceinline__ uint64_t make_key(float dist2, uint32_t rank, uint32_t flag) {
    return ((uint64_t)__float_as_uint(dist2) << 32) | ((uint64_t)rank << 1) | flag;
}
__device__ __forceinline__ uint32_t key_rank(uint64_t key) { return (uint32_t)(key & 0xFFFFFFFFull) >> 1; }
__device__ __forceinline__ float key_dist2(uint64_t key) { return __uint_as_float((uint32_t)(key >> 32)); }

// Sec. 4: [lo, hi] -> [l_q, r_q] on the ascending attribute array: l_q = #{a < lo},
// r_q = #{a <= hi} - 1.  Both counts are found by 32-ary search: per round every lane probes the
// last element of one of 32 sub-blocks and a ballot locates the block holding the boundary; the
// two searches advance together so their loads overlap (~log32(n) dependent round trips).
__device__ __forceinline__ void warp_rank_interval(const int32_t* __restrict__ a, int n, int32_t lo_key,
                                                   int32_t hi_key, int lane, int& l_q, int& r_q) {
    int lo0 = 0, hi0 = n;      // search for #{a < lo_key}
    int lo1 = 0, hi1 = n;      // search for #{a <= hi_key}
    while (hi0 > lo0 || hi1 > lo1) {
        const int len0 = hi0 - lo0, len1 = hi1 - lo1;
        const int step0 = (len0 + 31) >> 5, step1 = (len1 + 31) >> 5;
        const int off0 = lane * step0, off1 = lane * step1;
        int32_t v0 = 0, v1 = 0;
        const bool in0 = off0 < len0, in1 = off1 < len1;
        if (in0) v0 = __ldg(a + lo0 + min(off0 + step0, len0) - 1);
        if (in1) v1 = __ldg(a + lo1 + min(off1 + step1, len1) - 1);
        const int c0 = __popc(__ballot_sync(FULL, in0 && v0 < lo_key));
        const int c1 = __popc(__ballot_sync(FULL, in1 && v1 <= hi_key));
        if (len0 > 0) {
            if ((long long)c0 * step0 >= len0) lo0 = hi0;
            else { hi0 = lo0 + min((c0 + 1) * step0, len0) - 1; lo0 = lo0 + c0 * step0; }
        }
        if (len1 > 0) {
            if ((long long)c1 * step1 >= len1) lo1 = hi1;
            else { hi1 = lo1 + min((c1 + 1) * step1, len1) - 1; lo1 = lo1 + c1 * step1; }
        }
    }
    l_q = lo0;
    r_q = lo1 - 1;
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

// Visited set: open addressing in shared memory, linear probing, full ranks stored (no false
// positives).  Returns true iff `id` was not present (and is now).  Lanes of one warp may insert
// concurrently: the compare-and-swap lets exactly one copy of a repeated id through.  If the
// probe sequence is exhausted the home slot is overwritten: an older entry is forgotten, which can
// only cause a repeated distance evaluation -- merge_batch drops a candidate that is already in the
// pool, and one that was evicted from a full pool can never re-enter, so results are unaffected.
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
// 128 contiguous bytes (8 x 16-byte loads) -- whole 32-byte sectors only.  Rows are taken two
// rounds (8 rows) at a time with NG groups of each in flight per lane: for d <= 32*NG all loads
// of up to 8 rows are issued before the first use, i.e. one memory round trip.
template <int NG>
__device__ __forceinline__ float batch_dist2(const float* __restrict__ vectors, int d_pad,
                                             const float4* qs, uint32_t my_rank, int ns, int lane) {
    const int team = lane >> 3, sub = lane & 7;
    const int G = d_pad >> 2;
    float out = 0.f;
    const int src = (lane & 3) << 3;
#pragma unroll 1
    for (int r0 = 0; r0 * 4 < ns; r0 += 2) {
        const int viA = r0 * 4 + team, viB = viA + 4;
        const bool vA = viA < ns, vB = viB < ns;
        const bool anyB = (r0 + 1) * 4 < ns;                    // warp-uniform
        const uint32_t idA = __shfl_sync(FULL, my_rank, viA & 31);
        const uint32_t idB = __shfl_sync(FULL, my_rank, viB & 31);
        const float4* rowA = reinterpret_cast<const float4*>(vectors + (size_t)idA * (size_t)d_pad) + sub;
        const float4* rowB = reinterpret_cast<const float4*>(vectors + (size_t)idB * (size_t)d_pad) + sub;
        float accA = 0.f, accB = 0.f;
#pragma unroll 1
        for (int g0 = sub; g0 < G; g0 += 8 * NG) {
            float4 xa[NG], xb[NG];
#pragma unroll
            for (int c = 0; c < NG; ++c) {
                if (g0 + 8 * c < G) {
                    if (vA) xa[c] = ldg_stream_f4(rowA + (g0 - sub) + 8 * c);
                    if (vB) xb[c] = ldg_stream_f4(rowB + (g0 - sub) + 8 * c);
                }
            }
#pragma unroll
            for (int c = 0; c < NG; ++c) {
                if (g0 + 8 * c < G) {
                    const float4 q = qs[g0 + 8 * c];
                    float t;
                    if (vA) {
                        t = xa[c].x - q.x; accA = fmaf(t, t, accA);
                        t = xa[c].y - q.y; accA = fmaf(t, t, accA);
                        t = xa[c].z - q.z; accA = fmaf(t, t, accA);
                        t = xa[c].w - q.w; accA = fmaf(t, t, accA);
                    }
                    if (vB) {
                        t = xb[c].x - q.x; accB = fmaf(t, t, accB);
                        t = xb[c].y - q.y; accB = fmaf(t, t, accB);
                        t = xb[c].z - q.z; accB = fmaf(t, t, accB);
                        t = xb[c].w - q.w; accB = fmaf(t, t, accB);
                    }
                }
            }
        }
        // row j was handled by team j & 3 in round j >> 2
        accA = accA + __shfl_xor_sync(FULL, accA, 4);
        accA = accA + __shfl_xor_sync(FULL, accA, 2);
        accA = accA + __shfl_xor_sync(FULL, accA, 1);
        const float va = __shfl_sync(FULL, accA, src);
        if ((lane >> 2) == r0) out = va;
        if (anyB) {
            accB = accB + __shfl_xor_sync(FULL, accB, 4);
            accB = accB + __shfl_xor_sync(FULL, accB, 2);
            accB = accB + __shfl_xor_sync(FULL, accB, 1);
            const float vb = __shfl_sync(FULL, accB, src);
            if ((lane >> 2) == r0 + 1) out = vb;
        }
    }
    return out;
}

// ---- TMA bulk copies (global -> shared) completing on an mbarrier ----------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// One thread asks the copy engine for `bytes` (multiple of 16, both addresses 16-byte aligned);
// the bytes are credited to the mbarrier when they have landed in shared memory.
__device__ __forceinline__ void tma_load_1d(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Four rows of a 2-D tensor (row-major rows of the vector store) in one request: the tensor map's
// box is one row (or one column chunk of it) wide and one row high, the instruction names the first
// column and four row indices, and the four pieces land back to back in shared memory (destination
// 128-byte aligned).  Rows beyond the tensor read as zeros and still count their bytes.
__device__ __forceinline__ void tma_gather4(void* dst_smem, const void* tensor_map, int col, int r0, int r1, int r2, int r3,
                                            uint64_t* bar, uint64_t l2_policy) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes.L2::cache_hint"
                 " [%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;"
                 ::"r"(smem_u32(dst_smem)), "l"(reinterpret_cast<uint64_t>(tensor_map)), "r"(smem_u32(bar)),
                   "r"(col), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "l"(l2_policy)
                 : "memory");
}
// tma_load_1d with an L2 eviction policy
__device__ __forceinline__ void tma_load_1d_l2(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar,
                                               uint64_t l2_policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)), "l"(l2_policy) : "memory");
}
// Wait for the phase of parity `phase`; bounded: gives up after 2^22 polls and reports false (the
// caller flags the query instead of hanging the GPU).  try_wait already parks the thread for a
// hardware-chosen interval per poll; passing an explicit suspend-time hint measured 7 % slower.
__device__ __forceinline__ bool mbar_wait_limit(uint64_t* bar, uint32_t phase, int limit) {
    const uint32_t addr = smem_u32(bar);
    for (int it = 0; it < limit; ++it) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(addr), "r"(phase) : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t phase) {
    const uint32_t addr = smem_u32(bar);
    for (int it = 0; it < (1 << 22); ++it) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(addr), "r"(phase) : "memory");
        if (done) return true;
    }
    return false;
}

// Squared L2 distances of up to 32 rows, rows staged in shared memory by the copy engine.
// Lane j < ns holds the rank of row j in `my_rank`; on return lane j holds its distance.
// The ranks of one call must be pairwise distinct (see evaluate_and_merge).
// Rows are taken STAGE_ROWS at a time and, for long rows, in column chunks of at most
// STAGE_CHUNK bytes: one elected lane per row issues a bulk copy of the chunk into the stage
// buffer, all copies of a pass complete on one mbarrier, then every 8-lane team reduces its rows
// from shared memory.  The arithmetic order is the one of batch_dist2 (lane s of a team takes the
// 4-float groups g = s, s+8, ... in increasing g, fused multiply-adds, butterfly 4-2-1), so both
// routines return identical bits.  `phase` is the running parity of the warp's mbarrier.
constexpr int STAGE_CHUNK = 512;     // bytes of one row in flight per pass
#ifndef FROG_STAGE_ROWS
#define FROG_STAGE_ROWS 8            // 512-byte row slots in the search kernel's stage buffer
#endif
template <int STAGE_ROWS>
__device__ __forceinline__ float staged_dist2(const float* __restrict__ vectors, int d_pad, const float4* qs,
                                              float4* stage, uint64_t* bar, uint32_t& phase, bool& ok,
                                              uint32_t my_rank, int ns, int lane, int wait_limit = 1 << 22,
                                              bool issue_copies = true) {
    static_assert(STAGE_ROWS == 8 || STAGE_ROWS == 12 || STAGE_ROWS == 16, "rows per pass");
    const int team = lane >> 3, sub = lane & 7;
    const int row_bytes = d_pad * 4;
    float out = 0.f;
#pragma unroll 1
    for (int r0 = 0; r0 < ns; r0 += STAGE_ROWS) {
        const int nrows = min(STAGE_ROWS, ns - r0);
        // rank of the row this lane would copy (lane r copies row r0 + r)
        const uint32_t copy_rank = __shfl_sync(FULL, my_rank, (r0 + lane) & 31);
        const char* src_row = reinterpret_cast<const char*>(vectors) + (size_t)copy_rank * (size_t)row_bytes;
        float acc[STAGE_ROWS / 4];
#pragma unroll
        for (int i = 0; i < STAGE_ROWS / 4; ++i) acc[i] = 0.f;
#pragma unroll 1
        for (int c0 = 0; c0 < row_bytes; c0 += STAGE_CHUNK) {
            const int cbytes = min(STAGE_CHUNK, row_bytes - c0);
            __syncwarp();                                   // every lane is done reading the stage buffer
            if (lane == 0 && issue_copies) mbar_expect_tx(bar, (uint32_t)(nrows * cbytes));
            __syncwarp();
            if (lane < nrows && issue_copies)
                tma_load_1d(reinterpret_cast<char*>(stage) + lane * STAGE_CHUNK, src_row + c0, (uint32_t)cbytes, bar);
            ok = mbar_wait_limit(bar, phase, wait_limit) && ok;
            phase ^= 1u;
            const int g_lo = c0 >> 4, g_n = cbytes >> 4;    // 4-float groups of this chunk
#pragma unroll
            for (int i = 0; i < STAGE_ROWS / 4; ++i) {
                const int r = i * 4 + team;
                if (r < nrows) {
                    const float4* xrow = stage + r * (STAGE_CHUNK / 16);
#pragma unroll 4
                    for (int g = sub; g < g_n; g += 8) {
                        const float4 x = xrow[g];
                        const float4 q = qs[g_lo + g];
                        float t;
                        t = x.x - q.x; acc[i] = fmaf(t, t, acc[i]);
                        t = x.y - q.y; acc[i] = fmaf(t, t, acc[i]);
                        t = x.z - q.z; acc[i] = fmaf(t, t, acc[i]);
                        t = x.w - q.w; acc[i] = fmaf(t, t, acc[i]);
                    }
                }
            }
        }
        // row r0 + j was reduced by team j & 3 as its (j >> 2)-th row
        const int src = (lane & 3) << 3;
#pragma unroll
        for (int i = 0; i < STAGE_ROWS / 4; ++i) {
            if (i * 4 < nrows) {
                float a = acc[i];
                a = a + __shfl_xor_sync(FULL, a, 4);
                a = a + __shfl_xor_sync(FULL, a, 2);
                a = a + __shfl_xor_sync(FULL, a, 1);
                // the result for row r0 + i*4 + t sits in team t; hand it to lane r0 + i*4 + t
                const float v = __shfl_sync(FULL, a, src);
                if (lane >= r0 && ((lane - r0) >> 2) == i && lane - r0 < nrows) out = v;
            }
        }
    }
    return out;
}

// The same gather + distance for the search kernel, with a run-time row geometry and optional
// half-precision storage.  `rows` points at row-major data of `row_bytes` per row (fp32, or fp16
// when F16); a row, or its STAGE_CHUNK-byte column chunk, occupies a slot of `slot_bytes`.  fp16
// elements are converted to fp32 on the way out of shared memory; products and sums are fp32 in
// the same fixed order, so the result equals the fp32 routine run on the rounded values bit for
// bit.  ROWB > 0 fixes the row size at compile time, which unrolls the inner loops for the common
// shape; ROWB == 0 takes the geometry from the arguments.
// The stage buffer is split into two halves, each with its own mbarrier: while the teams reduce the rows of one half, the copies of the next group of
// rows are already landing in the other, so the arithmetic hides behind the copy latency.  A
// group is up to 8 rows (4 for 512-byte slots: one row per team); a row longer than STAGE_CHUNK is
// taken in column chunks, one chunk of every row of the group per step.  bar[0], bar[1] are the
// two mbarriers; `phases` holds their parities in bits 0 and 1.
// HOOKABLE && hook (tests of the error path): no copy is armed or issued and a wait gives up after 64
// polls, so the routine reports a time-out with nothing in flight.
template <bool F16, int ROWB = 0, bool HOOKABLE = false>
__device__ __forceinline__ float staged_dist2_pipe(const void* __restrict__ rows, int row_bytes, int slot_bytes,
                                                   const float4* qs, float4* stage, uint64_t* bar,
                                                   uint32_t& phases, bool& ok, uint32_t my_rank, int ns, int lane,
                                                   const void* tmap = nullptr, const uint32_t* ranks = nullptr,
                                                   int n_rows_total = 0, bool hook = false) {
    if (ROWB > 0) {
        row_bytes = ROWB;
        slot_bytes = ROWB >= STAGE_CHUNK ? STAGE_CHUNK : ROWB;
    }
    constexpr int HALF = FROG_STAGE_ROWS * STAGE_CHUNK / 2;
    constexpr int GROUP_BYTES = F16 ? 8 : 16;             // 4 elements
    constexpr int UNROLL_G = ROWB > 0 ? 4 : 1;            // the run-time geometry is short of registers
    const int rph = (HALF / slot_bytes) >= 8 ? 8 : 4;     // rows per half: two rows or one row per team
    const int chunks = (row_bytes + STAGE_CHUNK - 1) / STAGE_CHUNK;
    const int steps = ((ns + rph - 1) / rph) * chunks;
    const int team = lane >> 3, sub = lane & 7;
    int ig = 0, ic = 0;                                   // group and chunk of the next step to issue
    // With a tensor map (`tmap`, `ranks` = the ns ranks in shared memory, 16-byte aligned) lane 0
    // requests the rows of a step four at a time; slots past the last row name rows beyond the
    // tensor (distinct ones), which arrive as zeros.  Otherwise one bulk copy per row.
    constexpr int ELEM = F16 ? 2 : 4;
    const int box_bytes = slot_bytes;                     // the box is one slot wide
    const uint64_t row_policy = row_bytes <= STAGE_CHUNK ? l2_policy_evict_first() : l2_policy_evict_normal();
    auto issue = [&](int s) {
        const int r0 = ig * rph, nrows = min(rph, ns - r0);
        const int c0 = ic * STAGE_CHUNK, cbytes = min(STAGE_CHUNK, row_bytes - c0);
        uint64_t* b = bar + (s & 1);
        if (HOOKABLE && hook) {
            // nothing is requested
        } else if (tmap) {
            if (lane == 0) {
                const int quads = (nrows + 3) >> 2;
                mbar_expect_tx(b, (uint32_t)(quads * 4 * box_bytes));
                char* dst = reinterpret_cast<char*>(stage) + (s & 1) * HALF;
#pragma unroll
                for (int qd = 0; qd < 2; ++qd) {
                    if (qd < quads) {
                        const uint4 rk = *reinterpret_cast<const uint4*>(ranks + r0 + 4 * qd);
                        const int left = nrows - 4 * qd;        // valid rows of this quad (1..4)
                        tma_gather4(dst + 4 * qd * slot_bytes, tmap, c0 / ELEM, (int)rk.x,
                                    left > 1 ? (int)rk.y : n_rows_total + 1, left > 2 ? (int)rk.z : n_rows_total + 2,
                                    left > 3 ? (int)rk.w : n_rows_total + 3, b, row_policy);
                    }
                }
            }
        } else {
            if (lane == 0) mbar_expect_tx(b, (uint32_t)(nrows * cbytes));
            __syncwarp();
            const uint32_t copy_rank = __shfl_sync(FULL, my_rank, (r0 + lane) & 31);
            if (lane < nrows)
                tma_load_1d_l2(reinterpret_cast<char*>(stage) + (s & 1) * HALF + lane * slot_bytes,
                               reinterpret_cast<const char*>(rows) + (size_t)copy_rank * (size_t)row_bytes + c0,
                               (uint32_t)cbytes, b, row_policy);
        }
        if (++ic == chunks) { ic = 0; ++ig; }
    };
    issue(0);
    if (steps > 1) issue(1);
    float out = 0.f, acc0 = 0.f, acc1 = 0.f;
    int g = 0, c = 0;
#pragma unroll 1
    for (int s = 0; s < steps; ++s) {
        const int h = s & 1;
        ok = ((HOOKABLE && hook) ? mbar_wait_limit(bar + h, (phases >> h) & 1u, 64) : mbar_wait(bar + h, (phases >> h) & 1u)) && ok;
        phases ^= 1u << h;
        const int r0 = g * rph, nrows = min(rph, ns - r0);
        const int c0 = c * STAGE_CHUNK, cbytes = min(STAGE_CHUNK, row_bytes - c0);
        const int g_lo = c0 / GROUP_BYTES, g_n = cbytes / GROUP_BYTES;
        const char* half = reinterpret_cast<const char*>(stage) + h * HALF;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int r = i * 4 + team;
            if ((i == 0 || rph > 4) && r < nrows) {
                const char* xrow = half + r * slot_bytes;
                float a = i == 0 ? acc0 : acc1;
#pragma unroll UNROLL_G
                for (int gg = sub; gg < g_n; gg += 8) {
                    float4 x;
                    if (F16) {
                        const uint2 raw = *reinterpret_cast<const uint2*>(xrow + gg * 8);
                        const float2 lo2 = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
                        const float2 hi2 = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
                        x = make_float4(lo2.x, lo2.y, hi2.x, hi2.y);
                    } else {
                        x = *reinterpret_cast<const float4*>(xrow + gg * 16);
                    }
                    const float4 q = qs[g_lo + gg];
                    float t;
                    t = x.x - q.x; a = fmaf(t, t, a);
                    t = x.y - q.y; a = fmaf(t, t, a);
                    t = x.z - q.z; a = fmaf(t, t, a);
                    t = x.w - q.w; a = fmaf(t, t, a);
                }
                if (i == 0) acc0 = a; else acc1 = a;
            }
        }
        if (c == chunks - 1) {
            const int src = ((lane - r0) & 3) << 3;         // team that summed this lane's row
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                if ((i == 0 || rph > 4) && i * 4 < nrows) {
                    float a = i == 0 ? acc0 : acc1;
                    a = a + __shfl_xor_sync(FULL, a, 4);
                    a = a + __shfl_xor_sync(FULL, a, 2);
                    a = a + __shfl_xor_sync(FULL, a, 1);
                    const float v = __shfl_sync(FULL, a, src);
                    if (lane >= r0 && ((lane - r0) >> 2) == i && lane - r0 < nrows) out = v;
                }
            }
            acc0 = acc1 = 0.f;
            c = 0;
            ++g;
        } else {
            ++c;
        }
        __syncwarp();                                       // every lane is done reading this half
        if (s + 2 < steps) issue(s + 2);
    }
    return out;
}

// warp-wide smallest of the per-lane positions (0xFFFF = none)
__device__ __forceinline__ uint32_t first_pos(int m1) {
    return __reduce_min_sync(FULL, min((unsigned)m1, 0xFFFFu));
}

// Alg. 2 lines 15-17 in one pass.  `pool` holds ef_s (<= 32*EPL) keys ascending by key | 1,
// KEY_EMPTY at the tail; each lane brings at most one new key (KEY_EMPTY = none).  The final
// position of a new key is (#pool keys below it) + (#new keys below it); of a pool key, its
// index + (#new keys below it); everything landing at >= ef_s is dropped.  All counts come from
// register compares and ballots: the new keys are broadcast one by one with shuffles, the lanes
// hold the pool keys (lane l owns positions l, l+32, ...).  A new key equal to a pool key (a vertex
// the visited table forgot) or to an earlier new key is discarded.  Returns the position of the
// first entry whose flag is 0 (0xFFFF = none).
template <int EPL, bool UNIQUE = false>
__device__ __forceinline__ uint32_t merge_batch(uint64_t* pool, uint64_t my_key, int ef_s, int lane) {
    uint64_t pk[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) pk[e] = pool[lane + 32 * e];
    // a full pool rejects what is not better than its worst entry (also drops a copy of it)
    const uint64_t worst = pool[ef_s - 1];
    if ((my_key | 1ull) >= (worst | 1ull)) my_key = KEY_EMPTY;
    uint32_t have = __ballot_sync(FULL, my_key != KEY_EMPTY);
    int m1 = NO_POS;
    if (have == 0) {
#pragma unroll
        for (int e = 0; e < EPL; ++e)
            if (pk[e] != KEY_EMPTY && !(pk[e] & 1ull)) m1 = min(m1, lane + 32 * e);
        return first_pos(m1);
    }
    int add[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) add[e] = 0;
    int rnew = 0, above = 0;
    bool dropped = false;
    const uint32_t my_lo = (uint32_t)my_key | 1u, my_hi = (uint32_t)(my_key >> 32);
    const uint64_t mk = my_key | 1ull;
    if (UNIQUE && EPL <= 4) {
        // no copies to look for: two entering keys per iteration, so that the shuffles and ballots
        // of one overlap those of the other (the chain of one key at a time is latency, not work)
#pragma unroll 1
        for (uint32_t msk = have; msk;) {
            const int j0 = __ffs(msk) - 1;
            msk &= msk - 1;
            const int j1 = msk ? __ffs(msk) - 1 : j0;
            const bool two = msk != 0;
            msk &= msk - 1;
            const uint64_t x0 = ((uint64_t)__shfl_sync(FULL, my_hi, j0) << 32) | __shfl_sync(FULL, my_lo, j0);
            uint64_t x1 = ((uint64_t)__shfl_sync(FULL, my_hi, j1) << 32) | __shfl_sync(FULL, my_lo, j1);
            if (!two) x1 = KEY_EMPTY;                       // compares below nothing
            int above0 = 0, above1 = 0;
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                const uint64_t p = pk[e] | 1ull;
                const bool lt0 = x0 < p, lt1 = x1 < p;
                above0 += __popc(__ballot_sync(FULL, lt0));
                above1 += __popc(__ballot_sync(FULL, lt1));
                add[e] += (lt0 ? 1 : 0) + (lt1 ? 1 : 0);
            }
            rnew += ((x0 < mk) ? 1 : 0) + ((x1 < mk) ? 1 : 0);
            if (lane == j0) above = above0;
            if (two && lane == j1) above = above1;
        }
    } else
#pragma unroll 1
    for (uint32_t msk = have; msk; msk &= msk - 1) {
        const int j = __ffs(msk) - 1;
        const uint64_t x = ((uint64_t)__shfl_sync(FULL, my_hi, j) << 32) | __shfl_sync(FULL, my_lo, j);
        // copies: of a pool key, or of a new key held by a lower lane (UNIQUE: the caller
        // guarantees there are none, e.g. an exact visited set)
        bool eq = !UNIQUE && (x == mk) && (lane < j);
        bool lt[EPL];
        int cnt_above = 0;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const uint64_t p = pk[e] | 1ull;
            lt[e] = x < p;
            if (!UNIQUE) eq = eq || (x == p);
            cnt_above += __popc(__ballot_sync(FULL, lt[e]));
        }
        if (!UNIQUE && __any_sync(FULL, eq)) {
            if (lane == j) dropped = true;
            continue;
        }
#pragma unroll
        for (int e = 0; e < EPL; ++e) add[e] += lt[e] ? 1 : 0;
        rnew += (x < mk) ? 1 : 0;
        if (lane == j) above = cnt_above;
    }
    __syncwarp();
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
        if (pk[e] != KEY_EMPTY) {
            const int p = lane + 32 * e + add[e];
            if (p < ef_s) {
                if (add[e]) pool[p] = pk[e];
                if (!(pk[e] & 1ull)) m1 = min(m1, p);
            }
        }
    }
    if (my_key != KEY_EMPTY && !dropped) {
        const int p = (32 * EPL - above) + rnew;
        if (p < ef_s) {
            pool[p] = my_key;
            if (!(my_key & 1ull)) m1 = min(m1, p);
        }
    }
    __syncwarp();
    return first_pos(m1);
}

// smallest key of the warp under the order key | 1 (KEY_EMPTY if no lane has one)
__device__ __forceinline__ uint64_t warp_min_key(uint64_t key) {
    const uint32_t hi = (uint32_t)(key >> 32), lo = (uint32_t)key | 1u;
    const uint32_t mhi = __reduce_min_sync(FULL, hi);
    const uint32_t mlo = __reduce_min_sync(FULL, hi == mhi ? lo : 0xFFFFFFFFu);
    return ((uint64_t)mhi << 32) | mlo;
}

// entry point j of a query range: stateless mixer of (seed, l_q, r_q, j), top 32 bits scaled
// into [0, w) by a multiply-high (Alg. 2 line 3: uniform sample from [l_q, r_q])
__device__ __forceinline__ uint32_t entry_point(unsigned long long seed, uint32_t l_q, uint32_t r_q, int j) {
    unsigned long long x = seed ^ ((unsigned long long)l_q * 0x9E3779B97F4A7C15ull)
                                ^ ((unsigned long long)r_q * 0xC2B2AE3D27D4EB4Full)
                                ^ ((unsigned long long)(j + 1) * 0x165667B19E3779F9ull);
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    unsigned long long w = (unsigned long long)(r_q - l_q) + 1ull;
    return l_q + (uint32_t)(((x >> 32) * w) >> 32);
}

// Ranges covering at least this many slab words (262,144 objects) log the ranks they evaluate and
// zero only those words afterwards; narrower ones zero the words of the range (<= 32 KB).
constexpr int SPARSE_MIN_WORDS = 8192;

// Append the ns <= 128 ranks of cand[] (the vertices whose visited bit this query has just set) to the
// warp's log.  Returns the new length, or -1 once the log is full: the query then falls back to zeroing
// the words of its whole range.
__device__ __forceinline__ int log_ranks(uint32_t* log, int cap, int n_logged, const uint32_t* cand, int ns, int lane) {
    if (n_logged + ns > cap) return -1;
    for (int i = lane; i < ns; i += 32) __stcg(log + n_logged + i, cand[i]);
    return n_logged + ns;
}

// ---- visited TABLE: an exact hash set in global memory, small enough to stay in L2 ---------------
// 4-slot buckets of ranks (16 bytes), 0xFFFFFFFF = empty, linear probing over buckets.  A key is
// looked up with one 16-byte load of its bucket and, if absent, claimed with a compare-and-swap on
// the first empty slot; losing the slot to another key means looking at the bucket again.  Slots
// never become empty while a query runs, so a key absent from a bucket with a free slot is absent
// from the table.  The caller keeps the table at most half full.
constexpr uint32_t TABLE_EMPTY = 0xFFFFFFFFu;
__device__ __forceinline__ uint4 ld_bucket_l2(const uint32_t* p, uint64_t policy) {
    uint4 v;
    asm volatile("ld.global.cg.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(policy) : "memory");
    return v;
}
// (the compare-and-swap form of atom takes no L2 cache hint; the bucket loads carry it)
__device__ __forceinline__ uint32_t atomic_cas_l2(uint32_t* p, uint32_t cmp, uint32_t val, uint64_t) {
    return atomicCAS(p, cmp, val);
}
__device__ __forceinline__ uint32_t table_bucket(uint32_t v, int table_bits) {
    return (v * 0x9E3779B1u) >> (34 - table_bits);           // table_bits - 2 bucket bits
}
// slot of the bucket that holds v (-1), the first empty slot (0..3), or 4 when the bucket is full of other keys
__device__ __forceinline__ int bucket_find(const uint4& b, uint32_t v) {
    if (b.x == v || b.y == v || b.z == v || b.w == v) return -1;
    return b.x == TABLE_EMPTY ? 0 : b.y == TABLE_EMPTY ? 1 : b.z == TABLE_EMPTY ? 2 : b.w == TABLE_EMPTY ? 3 : 4;
}
// Test-and-insert of up to two keys per lane (a lane's probes of both keys are in flight together).
// fa / fb: the key was not in the table and is now.  Returns false if a probe sequence ran into its limit.
__device__ __forceinline__ bool table_insert2(uint32_t* table, int table_bits, uint32_t va, bool ha, uint32_t vb, bool hb,
                                              bool& fa, bool& fb, uint64_t policy) {
    const uint32_t bmask = (1u << (table_bits - 2)) - 1u;
    uint32_t ka = table_bucket(va, table_bits), kb = table_bucket(vb, table_bits);
    bool pa = ha, pb = hb;
    fa = fb = false;
#pragma unroll 1
    for (int it = 0; it < 4096 && __any_sync(FULL, pa || pb); ++it) {
        uint4 ba = make_uint4(0, 0, 0, 0), bb = make_uint4(0, 0, 0, 0);
        if (pa) ba = ld_bucket_l2(table + 4 * ka, policy);
        if (pb) bb = ld_bucket_l2(table + 4 * kb, policy);
        const int ja = pa ? bucket_find(ba, va) : -1, jb = pb ? bucket_find(bb, vb) : -1;
        uint32_t oa = va, ob = vb;
        if (pa && ja >= 0 && ja < 4) oa = atomic_cas_l2(table + 4 * ka + ja, TABLE_EMPTY, va, policy);
        if (pb && jb >= 0 && jb < 4) ob = atomic_cas_l2(table + 4 * kb + jb, TABLE_EMPTY, vb, policy);
        if (pa) {
            if (ja == 4) ka = (ka + 1) & bmask;
            else if (ja < 0 || oa == va) pa = false;                // found, or another lane put it there just now
            else if (oa == TABLE_EMPTY) { fa = true; pa = false; }
        }
        if (pb) {
            if (jb == 4) kb = (kb + 1) & bmask;
            else if (jb < 0 || ob == vb) pb = false;
            else if (ob == TABLE_EMPTY) { fb = true; pb = false; }
        }
    }
    return !__any_sync(FULL, pa || pb);
}

}  // namespace frogdev
