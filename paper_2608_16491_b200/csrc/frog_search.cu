// frog_search / frog_search_ex: batched FROGSearch (paper Alg. 2) as one persistent kernel.
//
// Mapping.  Queries are independent (Sec. 7.1), so each WARP owns one query at a time and pulls
// the next one from a global work counter; a CTA is just a bundle of such warps, they never
// synchronise with each other.  Per-query state lives in that warp's slice of shared memory: the
// candidate pool (sorted u64 keys), the compacted candidate list and the query vector.  Global
// memory holds the ENC array and the vectors; per expansion the warp reads the hotspot rows of
// ENC(u) and the rows of the surviving ENs only.
//
// Visited set (the hashCheck of Alg. 2 line 12), two interchangeable forms:
//   * BITMAP: one bit per rank in a per-warp slab of global scratch memory, test-and-set with a
//     single atomicOr (exact, no probing, no shared memory; the slab stays L2-resident while the
//     query runs).  A slab is all-zero between queries: a query over a narrow range zeroes the words
//     covering [l_q, r_q] when it ends; a query over a wide range instead logs the ranks it evaluates
//     (a few hundred to a few thousand, next to the slab) and zeroes only their words, so that the
//     cost of the visited set follows the work of the query, not the width of its range;
//   * HASH: an open-addressing table in shared memory (no scratch besides the work counter; a
//     crowded table forgets entries, which costs repeated distance evaluations, never results).
#include <cstdio>
#include <cstring>
#include <mutex>

#include "frog_device.cuh"
#include "frog_internal.h"

using namespace frogdev;

namespace {

#ifndef FROG_WARPS_PER_CTA
#define FROG_WARPS_PER_CTA 2
#endif
constexpr int WARPS_PER_CTA = FROG_WARPS_PER_CTA;
#ifndef FROG_MINB
#define FROG_MINB 16          // resident CTAs per SM the register allocation aims at (EPL <= 4)
#endif

#ifndef FROG_MINB_8
#define FROG_MINB_8 12        // the same for pools of 256 entries (80 registers)
#endif
#ifndef FROG_MINB_16
#define FROG_MINB_16 10       // and of 512 entries (96 registers)
#endif
#ifndef FROG_GATHER4
#define FROG_GATHER4 1         // rows fetched four per tensor-copy instruction where a tensor map exists
#endif
constexpr int MODE_FAST = 0, MODE_TRACE = 1, MODE_PROFILE = 2, MODE_EAGER = 3, MODE_COUNT = 4;
// EAGER: FAST with the eager hash check; COUNT: FAST that also keeps the per-query counters (`stats`)

constexpr int STAGE_BYTES = FROG_STAGE_ROWS * STAGE_CHUNK;

// per-warp shared memory: stage | pool | candidate list | two mbarriers, their parities, a failure flag |
// query | hash, the whole rounded up to 128 bytes (the stage buffer is the target of tensor copies,
// which want 128-byte alignment)
struct WarpSmem {
    uint64_t* pool;
    uint32_t* cand;
    uint64_t* bar;       // bar[0], bar[1] = mbarriers of the two stage halves; the two words after them:
                         // their phase parities (bits 0, 1) and the copy-timeout flag; 32 bytes in all
    float4* q;
    float4* stage;
    uint32_t* hash;
};

__host__ __device__ inline size_t warp_smem_bytes(int pool_slots, int q_len, int hash_bits, bool bitmap) {
    const size_t b = (size_t)STAGE_BYTES + (size_t)pool_slots * 8 + FROG_MAX_BUDGET * 4 + 32 + (size_t)q_len * 4 +
                     (bitmap ? 0 : ((size_t)4 << hash_bits));
    return (b + 127) & ~(size_t)127;
}
inline int query_len(int d) { return (d + 7) / 8 * 8; }

// test-and-set of rank v in the visited set; true iff v had not been evaluated yet
template <bool BITMAP>
__device__ __forceinline__ bool visited_test_and_set(const WarpSmem& S, uint32_t* bitmap, int hash_bits,
                                                     uint32_t v, uint32_t& forgets) {
    if (BITMAP) {
        const uint32_t bit = 1u << (v & 31);
        return (atomicOr(bitmap + (v >> 5), bit) & bit) == 0;
    } else {
        return visited_insert(S.hash, hash_bits, v, forgets);
    }
}

// Distances of the ns <= 32 ranks listed in cand[0..ns) and their merge into the pool (Alg. 2
// lines 14-17).  Returns the first unexpanded pool position.  Kept out of line: it is called from
// several places of the kernel and inlining every copy costs registers and instruction cache.
// UNIQUE: the visited set is exact (bitmap form), so the ranks are distinct and none is in the pool.
template <int EPL, bool F16, int ROWB, bool UNIQUE, bool HOOKABLE = false>
__device__ __noinline__ int evaluate_and_merge(const void* __restrict__ rows, int row_bytes, int slot_bytes, int ef_s,
                                               uint64_t* pool, const uint32_t* cand, uint64_t* bar,
                                               const float4* qs, float4* stage, int ns, uint32_t new_flag,
                                               const void* tmap, int n, long long* t_dist, bool hook = false) {
    const int lane = lane_id();
    uint32_t id = (lane < ns) ? cand[lane] : 0u;
    if (!UNIQUE) {
        // The shared-memory visited table can let the same rank through twice in one batch once it
        // starts dropping entries.  Two bulk copies of one source row completing on the same
        // mbarrier were observed to leave the barrier incomplete (the wait ran into its polling
        // limit), so repeated ranks are squeezed out before the gather.  The bitmap form never
        // produces repeats.
        const uint32_t same = __match_any_sync(FULL, (lane < ns) ? id : (0x80000000u | (uint32_t)lane));
        const bool first_copy = (lane < ns) && ((__ffs(same) - 1) == lane);
        const uint32_t keep_mask = __ballot_sync(FULL, first_copy);
        const int src_lane = __fns(keep_mask, 0, lane + 1);          // lane holding the (lane+1)-th kept rank
        const uint32_t moved = __shfl_sync(FULL, id, src_lane & 31);
        ns = __popc(keep_mask);
        id = (lane < ns) ? moved : 0u;
    }
    float d2 = 0.f;
    if (ns > 0) {
        uint32_t* bar_words = reinterpret_cast<uint32_t*>(bar + 2);
        __syncwarp();                       // lane 0's update of the parity in the previous call
        uint32_t phase = bar_words[0];
        bool ok = true;
        d2 = staged_dist2_pipe<F16, ROWB, HOOKABLE>(rows, row_bytes, slot_bytes, qs, stage, bar, phase, ok, id, ns, lane,
                                                    UNIQUE ? tmap : nullptr, cand, n, hook);
        __syncwarp();                       // every lane has read the old parity
        if (lane == 0) {
            bar_words[0] = phase;
            if (!ok) bar_words[1] = 1u;
        }
    }
    const uint64_t key = (lane < ns) ? make_key(d2, id, new_flag) : KEY_EMPTY;
    if (t_dist) *t_dist = clock64();
    return (int)merge_batch<EPL, UNIQUE>(pool, key, ef_s, lane);
}

template <int EPL, int MODE, bool BITMAP, bool F16, int ROWB = 0>
__global__ void __launch_bounds__(WARPS_PER_CTA * 32,
                                  (MODE == MODE_FAST || MODE == MODE_EAGER || MODE == MODE_COUNT)
                                      ? (EPL <= 4 ? FROG_MINB : EPL == 8 ? FROG_MINB_8 : FROG_MINB_16) : 1)
frog_search_kernel(const __grid_constant__ FrogSearchArgs A) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int lane = lane_id();
    const int warp = threadIdx.x >> 5;
    constexpr int POOL = 32 * EPL;
    const int hash_slots = BITMAP ? 0 : (1 << A.hash_bits);
    unsigned char* base = smem_raw + warp_smem_bytes(POOL, A.q_len, A.hash_bits, BITMAP) * warp;
    WarpSmem S;
    S.stage = reinterpret_cast<float4*>(base);
    S.pool = reinterpret_cast<uint64_t*>(base + STAGE_BYTES);
    S.cand = reinterpret_cast<uint32_t*>(S.pool + POOL);
    S.bar = reinterpret_cast<uint64_t*>(S.cand + FROG_MAX_BUDGET);
    S.q = reinterpret_cast<float4*>(S.bar + 4);
    S.hash = reinterpret_cast<uint32_t*>(reinterpret_cast<float*>(S.q) + A.q_len);
    if (lane == 0) {
        mbar_init(S.bar, 1u);
        mbar_init(S.bar + 1, 1u);
        reinterpret_cast<uint32_t*>(S.bar + 2)[0] = 0u;   // phase parities (bit 0, bit 1)
        reinterpret_cast<uint32_t*>(S.bar + 2)[1] = 0u;   // copy-timeout flag
    }
    __syncwarp();
    uint32_t* bitmap = BITMAP ? A.bitmap + (size_t)(blockIdx.x * WARPS_PER_CTA + warp) * A.slab_stride : nullptr;
    const uint32_t lt_mask = (1u << lane) - 1u;
    const uint64_t keep_in_l2 = l2_policy_evict_last();      // for the visited slab of the running query

    for (;;) {
        int q = 0;
        if (lane == 0) {
            q = (int)atomicAdd(A.work_counter, 1u);
            if (q < A.nq && A.order) q = __ldg(A.order + q);
        }
        q = __shfl_sync(FULL, q, 0);
        if (q >= A.nq) break;

        long long t_ph[6] = {0, 0, 0, 0, 0, 0};   // set-up, ENC scan, visited check, gather+distance, output, merge
        long long t_mark = (MODE == MODE_PROFILE) ? clock64() : 0;
 #define FROG_PHASE(i)                                                        \
    do {                                                                     \
        if (MODE == MODE_PROFILE) {                                          \
            long long _n = clock64();                                        \
            t_ph[i] += _n - t_mark;                                          \
            t_mark = _n;                                                     \
        }                                                                    \
    } while (0)

        // distance + merge call; in profile builds the time is split at the end of the distances
        long long t_split = 0;
        auto EVAL = [&](int ns_, uint32_t flag_, int off_ = 0) {
            int f_ = evaluate_and_merge<EPL, F16, ROWB, BITMAP, MODE == MODE_COUNT>(
                A.rows, A.row_bytes, A.slot_bytes, A.ef_s, S.pool, S.cand + off_, S.bar, S.q, S.stage, ns_, flag_,
                A.gather4 ? &A.tmap : nullptr, A.n, MODE == MODE_PROFILE ? &t_split : nullptr,
                MODE == MODE_COUNT && A.no_copies != 0);
            if (MODE == MODE_PROFILE) {
                long long n_ = clock64();
                t_ph[3] += t_split - t_mark;
                t_ph[5] += n_ - t_split;
                t_mark = n_;
            }
            return f_;
        };

        // ---- per-query set-up ---------------------------------------------------------------
        {
            float* qf = reinterpret_cast<float*>(S.q);
            const float* src = A.queries + (size_t)q * A.d;
            for (int i = lane; i < A.q_len; i += 32) qf[i] = i < A.d ? __ldg(src + i) : 0.f;
            for (int i = lane; i < POOL; i += 32) S.pool[i] = KEY_EMPTY;
        }
        const int32_t lo = __ldg(A.lo + q), hi = __ldg(A.hi + q);
        int l_q, r_q;
        if (A.ranges) {
            const int2 lr = __ldg(A.ranges + q);
            l_q = lr.x;
            r_q = lr.y;
        } else {
            warp_rank_interval(A.sorted_attr, A.n, lo, hi, lane, l_q, r_q);    // Sec. 4
        }
        const int w = (lo > hi) ? 0 : (r_q - l_q + 1);
        constexpr bool COUNT = MODE != MODE_FAST;          // the plain kernel keeps no work counters
        uint32_t st = 0, n_exp = 0, n_rows = 0, n_en = 0, n_dist = 0, forgets = 0;
        uint32_t trace_len = 0;
        bool trace_ok = true;
        uint32_t* trace_row = (MODE == MODE_TRACE || MODE == MODE_PROFILE) ? A.trace + (size_t)q * A.trace_cap : nullptr;
        __syncwarp();

        if (w <= 0) {
            st |= FROG_ST_EMPTY;
        } else if (w <= A.exact_w) {
            // every valid object is evaluated, the pool keeps the ef_s nearest: exact answer
            st |= FROG_ST_EXACT;
            for (int b0 = 0; b0 < w; b0 += 32) {
                const int cnt = min(32, w - b0);
                if (lane < cnt) S.cand[lane] = (uint32_t)(l_q + b0 + lane);
                __syncwarp();
                EVAL(cnt, 1u);
                if (COUNT) n_dist += cnt;
                __syncwarp();
            }
        } else {
            // Visited slab.  With `slab_clean` it is all-zero here and this query restores that when it
            // ends: by zeroing the words of its range, or (wide ranges) only the words of the ranks it
            // logged.  Without it the words of the range are zeroed now.
            int n_logged = -1;                                      // >= 0: ranks logged so far
            if (BITMAP) {
                const int w0 = l_q >> 5, w1 = r_q >> 5;
                if (!A.slab_clean)
                    for (int i = w0 + lane; i <= w1; i += 32) st_u32_l2(bitmap + i, 0u, keep_in_l2);
                else if (A.log_cap > 0 && w1 - w0 >= SPARSE_MIN_WORDS)
                    n_logged = 0;
            } else {
                uint4* h4 = reinterpret_cast<uint4*>(S.hash);
                const uint4 e4 = make_uint4(HASH_EMPTY, HASH_EMPTY, HASH_EMPTY, HASH_EMPTY);
                for (int i = lane; i < (hash_slots >> 2); i += 32) h4[i] = e4;
            }
            int L_start, L_end;
            hotspot_layers(l_q, r_q, A.H, A.n, L_start, L_end);          // Alg. 2 line 1
            if (A.no_hotspot) { L_start = 0; L_end = A.H - 1; }
            const int total = (L_end - L_start + 1) * A.m;
            const uint32_t span = (uint32_t)(r_q - l_q);
            __syncwarp();
            // lines 2-5: entry points, passed through the visited set
            int ns;
            {
                const uint32_t ep = entry_point(A.seed, (uint32_t)l_q, (uint32_t)r_q, lane);
                bool keep = lane < A.epn;
                if (keep) keep = visited_test_and_set<BITMAP>(S, bitmap, A.hash_bits, ep, forgets);
                const uint32_t M = __ballot_sync(FULL, keep);
                if (keep) S.cand[__popc(M & lt_mask)] = ep;
                ns = __popc(M);
                __syncwarp();
            }
            FROG_PHASE(0);
            if (COUNT) n_dist += ns;
            if (BITMAP && n_logged >= 0) n_logged = log_ranks(bitmap + A.bitmap_words, A.log_cap, n_logged, S.cand, ns, lane);
            int first = EVAL(ns, 0u);
            // lines 7-17
            while (first < A.ef_s) {
                if ((int)n_exp >= A.max_iters) { st |= FROG_ST_ITER_CAP; break; }
                const uint32_t u = key_rank(S.pool[first]);               // line 8
                __syncwarp();
                if (lane == 0) S.pool[first] |= 1ull;                     // line 9
                // line 10, Alg. 4: scan rows L_start..L_end of ENC(u) in 32-entry chunks (four
                // fetched per round trip); predicate "not empty and l_q <= v <= r_q" as one
                // unsigned compare (the empty entry 0xFFFFFFFF minus l_q exceeds any span);
                // ballot + popc give the admitted prefix under budget B.  Lines 12-13: each
                // admitted lane applies the visited check where it stands (it stays lazy: entries
                // already evaluated still consume budget); survivors are compacted into S.cand.
                const uint32_t* hot = A.enc + ((size_t)u * A.H + L_start) * A.m;
                // a trace record is appended only while a full one (header + max(64, B) entries) fits
                const bool rec_ok = (MODE == MODE_TRACE) && trace_ok && (trace_len + 2 + (uint32_t)max(64, A.B) <= (uint32_t)A.trace_cap - 1);
                int cnt = 0, scanned = 0;
                ns = 0;
                if (MODE == MODE_EAGER) {
                    // Ablation: the visited test is part of the predicate.  One 32-entry chunk at a
                    // time: every lane tests against the bitmap as the previous chunk left it, the
                    // admitted prefix sets its bits (a second copy of an id inside the chunk is
                    // admitted, finds the bit set and is dropped).
                    for (int c0 = 0; c0 < total && cnt < A.B; c0 += 32) {
                        uint32_t v = BOT;
                        if (c0 + lane < total) v = ldg_stream_u32(hot + c0 + lane);
                        const bool in_range = (v - (uint32_t)l_q) <= span;
                        const uint32_t bit = 1u << (v & 31);
                        uint32_t word = 0xFFFFFFFFu;
                        if (in_range) word = __ldcg(bitmap + (v >> 5));
                        const bool pred = (word & bit) == 0;
                        const uint32_t M = __ballot_sync(FULL, pred);
                        const int a = min(__popc(M), A.B - cnt);
                        const bool adm = pred && __popc(M & lt_mask) < a;
                        uint32_t old = 0xFFFFFFFFu;
                        if (adm) old = atomicOr(bitmap + (v >> 5), bit);
                        const bool keep = (old & bit) == 0;
                        const uint32_t K = __ballot_sync(FULL, keep);
                        if (keep) S.cand[ns + __popc(K & lt_mask)] = v;
                        ns += __popc(K);
                        cnt += a;
                        scanned = min(total, c0 + 32);
                    }
                } else
                // Four 32-entry chunks are fetched per round trip and their visited atomics are in
                // flight together; the admission under budget B runs over them in order, so the EN
                // list is the one a chunk-by-chunk scan yields.  A chunk counts as scanned only if it
                // exists and budget is left after the chunks before it.
                for (int c0 = 0; c0 < total && cnt < A.B; c0 += 128) {
                    uint32_t v0 = BOT, v1 = BOT, v2 = BOT, v3 = BOT;
                    if (c0 + lane < total) v0 = ldg_stream_u32(hot + c0 + lane);
                    if (c0 + 32 + lane < total) v1 = ldg_stream_u32(hot + c0 + 32 + lane);
                    if (c0 + 64 + lane < total) v2 = ldg_stream_u32(hot + c0 + 64 + lane);
                    if (c0 + 96 + lane < total) v3 = ldg_stream_u32(hot + c0 + 96 + lane);
                    const bool pred0 = (v0 - (uint32_t)l_q) <= span;
                    const uint32_t M0 = __ballot_sync(FULL, pred0);
                    const int a0 = min(__popc(M0), A.B - cnt);
                    const int rank0 = __popc(M0 & lt_mask);
                    const bool adm0 = pred0 && rank0 < a0;
                    const int rem1 = A.B - cnt - a0;
                    const bool has1 = (c0 + 32 < total) && rem1 > 0;
                    const bool pred1 = has1 && ((v1 - (uint32_t)l_q) <= span);
                    const uint32_t M1 = __ballot_sync(FULL, pred1);
                    const int a1 = min(__popc(M1), rem1);
                    const int rank1 = __popc(M1 & lt_mask);
                    const bool adm1 = pred1 && rank1 < a1;
                    const int rem2 = rem1 - a1;
                    const bool has2 = (c0 + 64 < total) && rem2 > 0;
                    const bool pred2 = has2 && ((v2 - (uint32_t)l_q) <= span);
                    const uint32_t M2 = __ballot_sync(FULL, pred2);
                    const int a2 = min(__popc(M2), rem2);
                    const int rank2 = __popc(M2 & lt_mask);
                    const bool adm2 = pred2 && rank2 < a2;
                    const int rem3 = rem2 - a2;
                    const bool has3 = (c0 + 96 < total) && rem3 > 0;
                    const bool pred3 = has3 && ((v3 - (uint32_t)l_q) <= span);
                    const uint32_t M3 = __ballot_sync(FULL, pred3);
                    const int a3 = min(__popc(M3), rem3);
                    const int rank3 = __popc(M3 & lt_mask);
                    const bool adm3 = pred3 && rank3 < a3;
                    if (MODE == MODE_TRACE && rec_ok) {
                        if (adm0) trace_row[3 + trace_len + cnt + rank0] = v0;
                        if (adm1) trace_row[3 + trace_len + cnt + a0 + rank1] = v1;
                        if (adm2) trace_row[3 + trace_len + cnt + a0 + a1 + rank2] = v2;
                        if (adm3) trace_row[3 + trace_len + cnt + a0 + a1 + a2 + rank3] = v3;
                    }
                    FROG_PHASE(1);
                    bool keep0, keep1, keep2, keep3;
                    if (BITMAP) {
                        const uint32_t bit0 = 1u << (v0 & 31), bit1 = 1u << (v1 & 31);
                        const uint32_t bit2 = 1u << (v2 & 31), bit3 = 1u << (v3 & 31);
                        uint32_t old0 = 0xFFFFFFFFu, old1 = 0xFFFFFFFFu, old2 = 0xFFFFFFFFu, old3 = 0xFFFFFFFFu;
                        if (adm0) old0 = atomic_or_l2(bitmap + (v0 >> 5), bit0, keep_in_l2);
                        if (adm1) old1 = atomic_or_l2(bitmap + (v1 >> 5), bit1, keep_in_l2);
                        if (adm2) old2 = atomic_or_l2(bitmap + (v2 >> 5), bit2, keep_in_l2);
                        if (adm3) old3 = atomic_or_l2(bitmap + (v3 >> 5), bit3, keep_in_l2);
                        keep0 = (old0 & bit0) == 0;
                        keep1 = (old1 & bit1) == 0;
                        keep2 = (old2 & bit2) == 0;
                        keep3 = (old3 & bit3) == 0;
                    } else {
                        keep0 = adm0 && visited_insert(S.hash, A.hash_bits, v0, forgets);
                        keep1 = adm1 && visited_insert(S.hash, A.hash_bits, v1, forgets);
                        keep2 = adm2 && visited_insert(S.hash, A.hash_bits, v2, forgets);
                        keep3 = adm3 && visited_insert(S.hash, A.hash_bits, v3, forgets);
                    }
                    const uint32_t K0 = __ballot_sync(FULL, keep0);
                    const uint32_t K1 = __ballot_sync(FULL, keep1);
                    const uint32_t K2 = __ballot_sync(FULL, keep2);
                    const uint32_t K3 = __ballot_sync(FULL, keep3);
                    const int n0 = __popc(K0), n1 = __popc(K1), n2 = __popc(K2);
                    if (keep0) S.cand[ns + __popc(K0 & lt_mask)] = v0;
                    if (keep1) S.cand[ns + n0 + __popc(K1 & lt_mask)] = v1;
                    if (keep2) S.cand[ns + n0 + n1 + __popc(K2 & lt_mask)] = v2;
                    if (keep3) S.cand[ns + n0 + n1 + n2 + __popc(K3 & lt_mask)] = v3;
                    ns += n0 + n1 + n2 + __popc(K3);
                    cnt += a0 + a1 + a2 + a3;
                    if (COUNT) scanned = min(total, c0 + (has3 ? 128 : has2 ? 96 : has1 ? 64 : 32));
                    FROG_PHASE(2);
                }
                __syncwarp();
                ++n_exp;
                if (COUNT) {
                    n_rows += (scanned + A.m - 1) / A.m;
                    n_en += cnt;
                    n_dist += ns;
                }
                if (MODE == MODE_TRACE) {
                    if (rec_ok) {
                        if (lane == 0) { trace_row[1 + trace_len] = u; trace_row[2 + trace_len] = (uint32_t)cnt; }
                        trace_len += 2 + cnt;
                    } else {
                        trace_ok = false;
                    }
                }
                if (BITMAP && n_logged >= 0) n_logged = log_ranks(bitmap + A.bitmap_words, A.log_cap, n_logged, S.cand, ns, lane);
                // lines 14-17; a budget above 32 can leave up to B survivors: batches of 32, the pool
                // after all of them is the same as after one merge of everything
                first = EVAL(min(ns, 32), 0u);
                for (int off = 32; off < ns; off += 32) first = EVAL(min(ns - off, 32), 0u, off);
            }
            if (BITMAP && A.slab_clean) {
                // leave the slab all-zero: the words of the logged ranks, or of the whole range
                if (n_logged >= 0) {
                    const uint32_t* log = bitmap + A.bitmap_words;
                    for (int i = lane; i < n_logged; i += 32) st_u32_l2(bitmap + (__ldcg(log + i) >> 5), 0u, keep_in_l2);
                } else {
                    const int w0 = l_q >> 5, w1 = r_q >> 5;
                    for (int i = w0 + lane; i <= w1; i += 32) bitmap[i] = 0u;
                }
            }
        }

        // ---- line 18: first k of the pool ---------------------------------------------------
        __syncwarp();
        const bool bad = reinterpret_cast<uint32_t*>(S.bar + 2)[1] != 0u;   // a copy never completed: not valid
        int got = 0;
        for (int j = lane; j < A.k; j += 32) {
            uint64_t key = S.pool[j];
            int32_t oid = -1;
            float dist = __int_as_float(0x7F800000);
            if (key != KEY_EMPTY && !bad) {
                oid = __ldg(A.rank2id + key_rank(key));
                dist = __fsqrt_rn(key_dist2(key));
                ++got;
            }
            A.out_ids[(size_t)q * A.k + j] = oid;
            A.out_dists[(size_t)q * A.k + j] = dist;
        }
        got = __reduce_add_sync(FULL, got);
        if (got < A.k) st |= FROG_ST_SHORT;
        if (__any_sync(FULL, forgets != 0)) st |= FROG_ST_FORGOT;   // counted per lane
        if (bad) st |= FROG_ST_COPY_TIMEOUT;
        if (bad && lane == 0) atomicOr(A.work_counter + 1, FROG_ST_COPY_TIMEOUT);   // sticky word of this launch
        FROG_PHASE(4);
        if (lane == 0) {
            if (A.status) A.status[q] = st;
            if (COUNT && A.stats) {
                uint32_t* srow = A.stats + 4 * (size_t)q;
                srow[0] = n_exp; srow[1] = n_rows; srow[2] = n_en; srow[3] = n_dist;
            }
            if (MODE == MODE_TRACE) trace_row[0] = trace_len;
            if (MODE == MODE_PROFILE) {
                trace_row[0] = 6;
                for (int i = 0; i < 6; ++i) trace_row[1 + i] = (uint32_t)min(t_ph[i], 0xFFFFFFFFll);
            }
        }
        __syncwarp();
#undef FROG_PHASE
    }
}

// ---- planning pass: endpoint conversion for the whole batch and a heaviest-first order ---------
// Queries differ in cost by the width of their range (wider ranges survive the filter more often
// and evaluate more distances).  With only a few queries per resident warp, the batch ends when the
// last long query does, so long queries are started first: queries are bucketed by floor(log2 w)
// and processed bucket by bucket in descending order.
constexpr int PLAN_HIST = 64, PLAN_CURSOR = 128;   // word offsets in the index's 1 KB work area

__global__ void __launch_bounds__(256)
frog_plan_kernel(const int32_t* __restrict__ sorted_attr, int n, const int32_t* __restrict__ lo,
                 const int32_t* __restrict__ hi, int nq, int2* __restrict__ ranges, unsigned int* work) {
    const int q = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = lane_id();
    if (q >= nq) return;
    const int32_t lo_q = __ldg(lo + q), hi_q = __ldg(hi + q);
    int l_q, r_q;
    warp_rank_interval(sorted_attr, n, lo_q, hi_q, lane, l_q, r_q);        // Sec. 4
    if (lane == 0) {
        ranges[q] = make_int2(l_q, r_q);
        const int w = (lo_q > hi_q) ? 0 : (r_q - l_q + 1);
        const int bucket = w <= 0 ? 0 : 32 - __clz(w);
        atomicAdd(work + PLAN_HIST + bucket, 1u);
    }
}

__global__ void __launch_bounds__(256)
frog_order_kernel(const int32_t* __restrict__ lo, const int32_t* __restrict__ hi, int nq,
                  const int2* __restrict__ ranges, int32_t* __restrict__ order, unsigned int* work) {
    const int q = (int)(blockIdx.x * blockDim.x + threadIdx.x);
    if (q >= nq) return;
    const int2 lr = ranges[q];
    const int w = (__ldg(lo + q) > __ldg(hi + q)) ? 0 : (lr.y - lr.x + 1);
    const int bucket = w <= 0 ? 0 : 32 - __clz(w);
    unsigned int base = 0;
    for (int b = bucket + 1; b <= 32; ++b) base += work[PLAN_HIST + b];   // queries in heavier buckets
    const unsigned int pos = base + atomicAdd(work + PLAN_CURSOR + bucket, 1u);
    order[pos] = q;
}

typedef frog_kernel_fn kernel_fn;

template <int MODE, bool BITMAP, bool F16>
kernel_fn pick_kernel(int ef_s, int* pool_slots) {
    if (ef_s <= 32) { *pool_slots = 32; return frog_search_kernel<1, MODE, BITMAP, F16>; }
    if (ef_s <= 64) { *pool_slots = 64; return frog_search_kernel<2, MODE, BITMAP, F16>; }
    if (ef_s <= 128) { *pool_slots = 128; return frog_search_kernel<4, MODE, BITMAP, F16>; }
    if (ef_s <= 256) { *pool_slots = 256; return frog_search_kernel<8, MODE, BITMAP, F16>; }
    *pool_slots = 512;
    return frog_search_kernel<16, MODE, BITMAP, F16>;
}

template <int ROWB, int MODE = MODE_FAST>
kernel_fn pick_rowb(int ef_s) {
    if (ef_s <= 32) return frog_search_kernel<1, MODE, true, false, ROWB>;
    if (ef_s <= 64) return frog_search_kernel<2, MODE, true, false, ROWB>;
    if (ef_s <= 128) return frog_search_kernel<4, MODE, true, false, ROWB>;
    if (ef_s <= 256) return frog_search_kernel<8, MODE, true, false, ROWB>;
    return frog_search_kernel<16, MODE, true, false, ROWB>;
}

size_t bitmap_words_per_slot(const frog_index* ix);
constexpr int TABLE_MIN_SLAB_WORDS = 1 << 17;     // 512 KB of visited bits per warp

struct LaunchPlan {
    kernel_fn fn;
    int grid, block, ctas_per_sm;
    size_t smem;
    bool table;        // the kernel keeps its visited sets in the L2-resident hash tables
};

int plan_launch(const frog_index* ix, int beam_width, const frog_params_t& P, int mode, bool bitmap, int nq,
                LaunchPlan* out, bool allow_table = true) {
    int pool_slots = 0;
    kernel_fn fn;
    const bool f16 = P.storage == FROG_STORAGE_F16;
    if (f16 && !bitmap) return FROG_ERR_UNSUPPORTED;       // fp16 rows are read by the bitmap kernels only
    if (f16)
        fn = mode == MODE_TRACE ? pick_kernel<MODE_TRACE, true, true>(beam_width, &pool_slots)
           : mode == MODE_PROFILE ? pick_kernel<MODE_PROFILE, true, true>(beam_width, &pool_slots)
           : mode == MODE_COUNT ? pick_kernel<MODE_COUNT, true, true>(beam_width, &pool_slots)
                                : pick_kernel<MODE_FAST, true, true>(beam_width, &pool_slots);
    else if (bitmap)
        fn = mode == MODE_TRACE ? pick_kernel<MODE_TRACE, true, false>(beam_width, &pool_slots)
           : mode == MODE_PROFILE ? pick_kernel<MODE_PROFILE, true, false>(beam_width, &pool_slots)
           : mode == MODE_COUNT ? pick_kernel<MODE_COUNT, true, false>(beam_width, &pool_slots)
                                : pick_kernel<MODE_FAST, true, false>(beam_width, &pool_slots);
    else
        fn = mode == MODE_TRACE ? pick_kernel<MODE_TRACE, false, false>(beam_width, &pool_slots)
           : mode == MODE_PROFILE ? pick_kernel<MODE_PROFILE, false, false>(beam_width, &pool_slots)
           : mode == MODE_COUNT ? pick_kernel<MODE_COUNT, false, false>(beam_width, &pool_slots)
                                : pick_kernel<MODE_FAST, false, false>(beam_width, &pool_slots);
    if (P.eager_hash) {
        if (!bitmap || f16 || (mode != MODE_FAST && mode != MODE_COUNT)) return FROG_ERR_UNSUPPORTED;
        fn = pick_kernel<MODE_EAGER, true, false>(beam_width, &pool_slots);
        if (ix->info.d_pad * 4 == 512) fn = pick_rowb<512, MODE_EAGER>(beam_width);
    }
    // common shapes with the row geometry fixed at compile time (fp32 rows of 384, 512 and 3072 bytes:
    // d = 96, 128, 768)
    if (mode == MODE_FAST && bitmap && !f16 && !P.eager_hash) {
        const int rb = ix->info.d_pad * 4;
        if (rb == 512) fn = pick_rowb<512>(beam_width);
        else if (rb == 384) fn = pick_rowb<384>(beam_width);
        else if (rb == 3072) fn = pick_rowb<3072>(beam_width);
    }
    size_t smem = warp_smem_bytes(pool_slots, query_len(ix->info.d), P.hash_bits, bitmap) * WARPS_PER_CTA;
    bool table = false;
    // the trimmed kernel for short fp32 rows (needs the row tensor map); debug_flags bit 2 keeps the generic one
    if (mode == MODE_FAST && bitmap && !f16 && !P.eager_hash && FROG_GATHER4 && ix->has_tmap_f32 && !(P.debug_flags & 4)) {
        size_t per_warp = 0;
        int wpc = 0;
        // visited hash table instead of the bitmap: where the slabs are far too large for L2 (indexes of
        // 4,194,304 objects and more: measured 1.26x faster at 10M objects, 0.85x at 1M, where the bits a
        // query touches still fit L2) and the pool is small enough for a query to fit the table as a rule;
        // FROG_VISITED_BITMAP keeps the bitmap
        const bool hook = (P.debug_flags & 32) != 0;
        table = allow_table && !hook && P.visited == FROG_VISITED_AUTO && beam_width <= 128 &&
                (bitmap_words_per_slot(ix) >= (size_t)TABLE_MIN_SLAB_WORDS || (P.debug_flags & 8));
        kernel_fn lean = froghost::lean_kernel(beam_width, P.budget, ix->info.d_pad * 4, table, hook, &per_warp, &wpc);
        if (!lean && table) {
            table = false;
            lean = froghost::lean_kernel(beam_width, P.budget, ix->info.d_pad * 4, false, hook, &per_warp, &wpc);
        }
        if (lean && wpc == WARPS_PER_CTA) {
            fn = lean;
            smem = per_warp * WARPS_PER_CTA;
        } else {
            table = false;
        }
    }
    if (smem > 227 * 1024) return FROG_ERR_UNSUPPORTED;
    FROG_CUDA_TRY(cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 0;
    FROG_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, (const void*)fn, WARPS_PER_CTA * 32, smem));
    if (per_sm < 1) return FROG_ERR_UNSUPPORTED;
    int grid = per_sm * ix->sm_count;
    if (nq > 0) {
        int need = (nq + WARPS_PER_CTA - 1) / WARPS_PER_CTA;
        if (grid > need) grid = need;
    }
    out->fn = fn;
    out->grid = grid < 1 ? 1 : grid;
    out->block = WARPS_PER_CTA * 32;
    out->ctas_per_sm = per_sm;
    out->smem = smem;
    out->table = table;
    return FROG_OK;
}

// gather source and stage geometry: a row slot is the row, or its 512-byte chunk
void set_gather(const frog_index* ix, bool f16, FrogSearchArgs* A) {
    const int d_pad_h = query_len(ix->info.d);
    A->rows = f16 ? ix->d_vectors_h : (const void*)ix->d_vectors;
    A->row_bytes = f16 ? d_pad_h * 2 : ix->info.d_pad * 4;
    A->slot_bytes = A->row_bytes < STAGE_CHUNK ? A->row_bytes : STAGE_CHUNK;   // rows are 16-byte multiples
    A->q_len = d_pad_h;
    A->no_copies = 0;
    A->gather4 = FROG_GATHER4 && (f16 ? ix->has_tmap_f16 : ix->has_tmap_f32);
    if (A->gather4) A->tmap = f16 ? ix->tmap_f16 : ix->tmap_f32;
    else std::memset(&A->tmap, 0, sizeof(A->tmap));
}

// per-warp visited slab: one bit per rank, padded to 128 bytes
size_t bitmap_words_per_slot(const frog_index* ix) {
    size_t words = ((size_t)ix->info.n + 31) / 32;
    return (words + 31) & ~(size_t)31;
}
// entries of the log of evaluated ranks that follows the bits of a slab in the index's own scratch
// (indexes whose slab never reaches SPARSE_MIN_WORDS have none)
constexpr int SLAB_LOG_ENTRIES = 8192;
int slab_log_entries(const frog_index* ix) {
    return bitmap_words_per_slot(ix) > (size_t)SPARSE_MIN_WORDS ? SLAB_LOG_ENTRIES : 0;
}

}  // namespace

namespace froghost {

int resolve_params(const frog_index* ix, int beam_width, const frog_params_t* in, frog_params_t* out) {
    frog_params_t P;
    std::memset(&P, 0, sizeof(P));
    if (in) P = *in;
    if (P.epn == 0) P.epn = 16;
    if (P.budget == 0) P.budget = 16;
    if (P.max_iters == 0) P.max_iters = 16 * beam_width;
    if (P.epn < 1 || P.epn > FROG_MAX_EPN || P.budget < 1 || P.budget > FROG_MAX_BUDGET || P.max_iters < 1)
        return FROG_ERR_INVALID_ARG;
    if (P.hash_bits == 0) {
        // about 16 evaluated vertices per beam slot, at most half full
        int want = 16 * beam_width;
        int bits = 9;
        while ((1 << bits) < want && bits < 13) ++bits;
        P.hash_bits = bits;
    }
    if (P.hash_bits < 6 || P.hash_bits > 15) return FROG_ERR_INVALID_ARG;
    if (P.visited != FROG_VISITED_AUTO && P.visited != FROG_VISITED_BITMAP && P.visited != FROG_VISITED_HASH)
        return FROG_ERR_INVALID_ARG;
    if (P.storage != FROG_STORAGE_F32 && P.storage != FROG_STORAGE_F16) return FROG_ERR_INVALID_ARG;
    if (P.exact_below < 0) return FROG_ERR_INVALID_ARG;
    if (P.storage == FROG_STORAGE_F16 && !ix->d_vectors_h) return FROG_ERR_INVALID_ARG;   // not enabled on this index
    (void)ix;
    *out = P;
    return FROG_OK;
}

// Tensor map over a row store (n rows of row_elems elements, row_bytes apart) whose box is one row
// high and one stage slot wide: what the 4-row gather of the copy engine needs.  Returns false
// (rows are then copied one by one) if the driver entry point cannot be had, the shape does not
// qualify (two quads per stage half need 4 slots to be a multiple of 128 bytes) or encoding fails.
bool make_row_tensor_map(const void* base, bool f16, int row_elems, size_t row_bytes, size_t n, CUtensorMap* out) {
    typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static encode_fn encode = nullptr;
    static bool looked_up = false;
    if (!looked_up) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            encode = reinterpret_cast<encode_fn>(fn);
        else
            cudaGetLastError();
        looked_up = true;
    }
    const int elem = f16 ? 2 : 4;
    const size_t slot = row_bytes < (size_t)STAGE_CHUNK ? row_bytes : (size_t)STAGE_CHUNK;
    if (!encode || !base || n == 0 || n > 0x7FFFFFF0ull) return false;
    if (row_bytes % 16 != 0 || slot % 16 != 0 || (reinterpret_cast<uintptr_t>(base) & 15) != 0) return false;
    if (slot <= 256 && slot % 32 != 0) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)row_elems, (cuuint64_t)n};
    cuuint64_t gstride[1] = {(cuuint64_t)row_bytes};
    cuuint32_t box[2] = {(cuuint32_t)(slot / elem), 1u};
    cuuint32_t estride[2] = {1u, 1u};
    const CUresult r = encode(out, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                              const_cast<void*>(base), gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Scratch set for a launch on stream s.  Launches of one stream are ordered by the stream, so a
// stream keeps the set it used last.  Otherwise an idle set (its last launch has finished) is
// taken, or a new one is created while fewer than FROG_SCRATCH_SETS exist, or the stream is made
// to wait for the set that has been unused the longest.  Called with ix->mu held.
int acquire_scratch(frog_index* ix, cudaStream_t s, FrogScratch** out) {
    FrogScratch* pick = nullptr;
    for (int i = 0; i < ix->n_scratch && !pick; ++i)
        if (ix->scratch[i].tick && ix->scratch[i].stream == s) pick = &ix->scratch[i];
    for (int i = 0; i < ix->n_scratch && !pick; ++i) {
        FrogScratch& sc = ix->scratch[i];
        if (!sc.tick) { pick = &sc; break; }
        const cudaError_t q = cudaEventQuery(sc.done);
        if (q == cudaSuccess) pick = &sc;
        else if (q == cudaErrorNotReady) cudaGetLastError();
        else { set_cuda_error(q); return FROG_ERR_CUDA; }
    }
    if (!pick && ix->n_scratch < FROG_SCRATCH_SETS) {
        FrogScratch& sc = ix->scratch[ix->n_scratch];
        cudaError_t e = cudaMalloc(&sc.d_work, 1024);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&sc.done, cudaEventDisableTiming);
        if (e != cudaSuccess) {
            cudaGetLastError();
            if (sc.d_work) cudaFree(sc.d_work);
            sc.d_work = nullptr;
            if (ix->n_scratch == 0) { set_cuda_error(e); return e == cudaErrorMemoryAllocation ? FROG_ERR_NOMEM : FROG_ERR_CUDA; }
        } else {
            ++ix->n_scratch;
            pick = &sc;
        }
    }
    if (!pick) {
        pick = &ix->scratch[0];
        for (int i = 1; i < ix->n_scratch; ++i)
            if (ix->scratch[i].tick < pick->tick) pick = &ix->scratch[i];
        FROG_CUDA_TRY(cudaStreamWaitEvent(s, pick->done, 0));
    }
    *out = pick;
    return FROG_OK;
}

// Make sure the set owns a visited slab for `slots` resident warps.  Grows (cudaFree + cudaMalloc,
// after synchronising the device) only when a launch needs more slots than any launch before it.
int ensure_bitmap(const frog_index* ix, FrogScratch* sc, size_t slots) {
    const size_t words = bitmap_words_per_slot(ix) + (size_t)slab_log_entries(ix);
    if (sc->d_bitmap && sc->bitmap_slots >= slots) return FROG_OK;
    FROG_CUDA_TRY(cudaDeviceSynchronize());
    if (sc->d_bitmap) FROG_CUDA_TRY(cudaFree(sc->d_bitmap));
    sc->d_bitmap = nullptr;
    sc->bitmap_slots = 0;
    cudaError_t e = cudaMalloc(&sc->d_bitmap, slots * words * sizeof(uint32_t));
    if (e != cudaSuccess) {
        cudaGetLastError();
        set_cuda_error(e);
        return FROG_ERR_NOMEM;
    }
    // the search kernel keeps every slab all-zero between queries; start it that way
    FROG_CUDA_TRY(cudaMemset(sc->d_bitmap, 0, slots * words * sizeof(uint32_t)));
    FROG_CUDA_TRY(cudaDeviceSynchronize());               // before a launch on any (non-blocking) stream
    sc->bitmap_slots = slots;
    return FROG_OK;
}

// Visited hash tables for `slots` resident warps, all entries empty (the kernel leaves them so).
int ensure_table(FrogScratch* sc, size_t slots, int bits) {
    // the tables are all-empty at rest, so an allocation can be re-cut into tables of another size
    const size_t bytes = (slots << bits) * sizeof(uint32_t);
    if (sc->d_table && sc->table_bytes >= bytes) {
        sc->table_bits = bits;
        sc->table_slots = sc->table_bytes / sizeof(uint32_t) >> bits;
        return FROG_OK;
    }
    FROG_CUDA_TRY(cudaDeviceSynchronize());
    if (sc->d_table) FROG_CUDA_TRY(cudaFree(sc->d_table));
    sc->d_table = nullptr;
    sc->table_slots = 0;
    sc->table_bytes = 0;
    cudaError_t e = cudaMalloc(&sc->d_table, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        set_cuda_error(e);
        return FROG_ERR_NOMEM;
    }
    FROG_CUDA_TRY(cudaMemset(sc->d_table, 0xFF, bytes));
    FROG_CUDA_TRY(cudaDeviceSynchronize());
    sc->table_bytes = bytes;
    sc->table_bits = bits;
    sc->table_slots = slots;
    return FROG_OK;
}

// Per-query planning scratch: 3 ints per query, grown when a batch is larger than any before.
int ensure_plan(FrogScratch* sc, size_t nq) {
    if (sc->d_plan && sc->plan_queries >= nq) return FROG_OK;
    FROG_CUDA_TRY(cudaDeviceSynchronize());
    if (sc->d_plan) FROG_CUDA_TRY(cudaFree(sc->d_plan));
    sc->d_plan = nullptr;
    sc->plan_queries = 0;
    cudaError_t e = cudaMalloc(&sc->d_plan, nq * 3 * sizeof(int32_t));
    if (e != cudaSuccess) {
        cudaGetLastError();
        set_cuda_error(e);
        return FROG_ERR_NOMEM;
    }
    sc->plan_queries = nq;
    return FROG_OK;
}

}  // namespace froghost

extern "C" int frog_search_launch_info(const frog_index_t* index, int beam_width, const frog_params_t* params,
                                       int* grid, int* block, int* smem_bytes, int* queries_per_sm) {
    if (!index || beam_width < 1 || beam_width > FROG_MAX_BEAM_WIDTH) return FROG_ERR_INVALID_ARG;
    frog_params_t P;
    int rc = froghost::resolve_params(index, beam_width, params, &P);
    if (rc) return rc;
    FROG_CUDA_TRY(cudaSetDevice(index->info.device));
    LaunchPlan plan;
    rc = plan_launch(index, beam_width, P, MODE_FAST, P.visited != FROG_VISITED_HASH, 0, &plan);
    if (rc) return rc;
    if (grid) *grid = plan.grid;
    if (block) *block = plan.block;
    if (smem_bytes) *smem_bytes = (int)plan.smem;
    if (queries_per_sm) *queries_per_sm = plan.ctas_per_sm * WARPS_PER_CTA;
    return FROG_OK;
}

extern "C" int frog_search_ex(const frog_index_t* index, const float* queries, const int32_t* lo, const int32_t* hi,
                              int nq, int k, int beam_width, const frog_params_t* params,
                              int32_t* out_ids, float* out_dists, uint32_t* status, uint32_t* stats,
                              uint32_t* trace, int trace_cap, void* stream) {
    if (!index || nq < 0) return FROG_ERR_INVALID_ARG;
    if (k < 1 || beam_width < 1 || beam_width > FROG_MAX_BEAM_WIDTH || k > beam_width) return FROG_ERR_INVALID_ARG;
    if (trace && trace_cap < 8) return FROG_ERR_INVALID_ARG;
    if (nq == 0) return FROG_OK;
    if (!queries || !lo || !hi || !out_ids || !out_dists) return FROG_ERR_INVALID_ARG;
    frog_params_t P;
    int rc = froghost::resolve_params(index, beam_width, params, &P);
    if (rc) return rc;
    FROG_CUDA_TRY(cudaSetDevice(index->info.device));
    const int mode = trace ? ((P.debug_flags & 1) ? MODE_PROFILE : MODE_TRACE) : stats ? MODE_COUNT : MODE_FAST;
    bool bitmap = P.visited != FROG_VISITED_HASH;
    LaunchPlan plan;
    rc = plan_launch(index, beam_width, P, mode, bitmap, nq, &plan);
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    frog_index* mix = const_cast<frog_index*>(index);      // the scratch sets are the index's only mutable part
    std::lock_guard<std::mutex> lock(mix->mu);
    FrogScratch* sc = nullptr;
    rc = froghost::acquire_scratch(mix, s, &sc);
    if (rc) return rc;
    if (bitmap) {
        rc = froghost::ensure_bitmap(index, sc, (size_t)plan.grid * WARPS_PER_CTA);
        if (rc == FROG_ERR_NOMEM && P.visited == FROG_VISITED_AUTO) {
            // no room for the slabs: fall back to the shared-memory table
            bitmap = false;
            rc = plan_launch(index, beam_width, P, mode, false, nq, &plan);
        }
        if (rc) return rc;
    }
    const int table_bits = beam_width <= 64 ? FROG_TABLE_BITS : FROG_TABLE_BITS_WIDE;
    if (plan.table && froghost::ensure_table(sc, (size_t)plan.grid * WARPS_PER_CTA, table_bits) != FROG_OK) {
        rc = plan_launch(index, beam_width, P, mode, bitmap, nq, &plan, false);     // no room: bitmap only
        if (rc) return rc;
    }

    FrogSearchArgs A;
    A.sorted_attr = index->d_sorted_attr;
    A.rank2id = index->d_rank2id;
    A.vectors = index->d_vectors;
    A.enc = index->d_enc;
    A.n = (int)index->info.n;
    A.d = index->info.d;
    A.d_pad = index->info.d_pad;
    A.H = index->info.H;
    A.m = index->info.m;
    A.queries = queries;
    A.lo = lo;
    A.hi = hi;
    A.nq = nq;
    A.k = k;
    A.ef_s = beam_width;
    A.epn = P.epn;
    A.B = P.budget;
    A.max_iters = P.max_iters;
    A.no_hotspot = P.no_hotspot;
    A.exact_w = P.exact_below > beam_width ? P.exact_below : beam_width;
    A.hash_bits = P.hash_bits;
    A.seed = P.seed;
    A.out_ids = out_ids;
    A.out_dists = out_dists;
    A.status = status;
    A.stats = stats;
    A.trace = trace;
    A.trace_cap = trace_cap;
    A.work_counter = sc->d_work;
    A.bitmap = bitmap ? sc->d_bitmap : nullptr;
    A.bitmap_words = bitmap_words_per_slot(index);
    A.log_cap = slab_log_entries(index);
    A.slab_stride = A.bitmap_words + (size_t)A.log_cap;
    A.slab_clean = 1;
    A.table = plan.table ? sc->d_table : nullptr;
    A.table_bits = table_bits;
    if (((P.debug_flags >> 8) & 15) >= 6 && ((P.debug_flags >> 8) & 15) <= table_bits)
        A.table_bits = (P.debug_flags >> 8) & 15;           // tests: a small table, so that queries outgrow it
    A.ranges = nullptr;
    A.order = nullptr;
    set_gather(index, P.storage == FROG_STORAGE_F16, &A);
    A.no_copies = (P.debug_flags & 32) ? 1 : 0;             // tests of the error path (see frog.h)

    FROG_CUDA_TRY(cudaMemsetAsync(sc->d_work, 0, 1024, s));
    // planning pass (skipped for tiny batches and when its scratch cannot be had)
    const bool planned = !(P.debug_flags & 2) && nq >= 64 && froghost::ensure_plan(sc, (size_t)nq) == FROG_OK;
    if (planned) {
        int2* ranges = reinterpret_cast<int2*>(sc->d_plan);
        int32_t* order = sc->d_plan + 2 * sc->plan_queries;
        frog_plan_kernel<<<(nq * 32 + 255) / 256, 256, 0, s>>>(index->d_sorted_attr, A.n, lo, hi, nq, ranges, sc->d_work);
        frog_order_kernel<<<(nq + 255) / 256, 256, 0, s>>>(lo, hi, nq, ranges, order, sc->d_work);
        A.ranges = ranges;
        A.order = order;
    }
    const bool timed = (P.debug_flags & 16) != 0;          // events around the search kernel alone
    if (timed) {
        if (!sc->k_begin) FROG_CUDA_TRY(cudaEventCreate(&sc->k_begin));
        if (!sc->k_end) FROG_CUDA_TRY(cudaEventCreate(&sc->k_end));
        FROG_CUDA_TRY(cudaEventRecord(sc->k_begin, s));
    }
    plan.fn<<<plan.grid, plan.block, plan.smem, s>>>(A);
    FROG_CUDA_TRY(cudaGetLastError());
    if (timed) FROG_CUDA_TRY(cudaEventRecord(sc->k_end, s));
    sc->k_timed = timed;
    FROG_CUDA_TRY(cudaEventRecord(sc->done, s));
    sc->stream = s;
    sc->tick = ++mix->tick;
    return FROG_OK;
}

extern "C" int frog_search_last_status(const frog_index_t* index, void* stream, uint32_t* flags) {
    if (!index || !flags) return FROG_ERR_INVALID_ARG;
    frog_index* mix = const_cast<frog_index*>(index);
    std::lock_guard<std::mutex> lock(mix->mu);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (int i = 0; i < mix->n_scratch; ++i) {
        FrogScratch& sc = mix->scratch[i];
        if (sc.tick && sc.stream == s) {
            FROG_CUDA_TRY(cudaEventSynchronize(sc.done));
            unsigned int word = 0;
            FROG_CUDA_TRY(cudaMemcpy(&word, sc.d_work + 1, sizeof(word), cudaMemcpyDeviceToHost));
            *flags = word;
            return FROG_OK;
        }
    }
    return FROG_ERR_INVALID_ARG;           // no launch on this stream
}

extern "C" int frog_search_kernel_ms(const frog_index_t* index, void* stream, float* ms) {
    if (!index || !ms) return FROG_ERR_INVALID_ARG;
    frog_index* mix = const_cast<frog_index*>(index);
    std::lock_guard<std::mutex> lock(mix->mu);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (int i = 0; i < mix->n_scratch; ++i) {
        FrogScratch& sc = mix->scratch[i];
        if (sc.tick && sc.stream == s && sc.k_timed) {
            FROG_CUDA_TRY(cudaEventSynchronize(sc.k_end));
            FROG_CUDA_TRY(cudaEventElapsedTime(ms, sc.k_begin, sc.k_end));
            return FROG_OK;
        }
    }
    return FROG_ERR_INVALID_ARG;           // no timed launch on this stream
}

extern "C" int frog_search(const frog_index_t* index, const float* queries, const int32_t* lo, const int32_t* hi,
                           int nq, int k, int beam_width, int32_t* out_ids, float* out_dists, void* stream) {
    return frog_search_ex(index, queries, lo, hi, nq, k, beam_width, nullptr, out_ids, out_dists,
                          nullptr, nullptr, nullptr, 0, stream);
}

// ---------------------------------------------------------------------------------------------
// frog_search_static: the same search with every byte of scratch in a fixed device array.
//
// Some callers must not allocate device memory while they search: code running under a stream
// capture or inside a latency-critical serving loop where cudaMalloc's implicit synchronisation
// is not acceptable, plug-ins whose host hands them a fixed memory budget, and processes that
// run next to another framework's caching allocator which already owns the free memory.  For them
// the work counter and the per-warp visited slabs live in the array below.  Its size is fixed at
// compile time (16 MiB + 256 B, held by every GPU that loads this library until the process
// exits), so the call limits the number of resident warps to the slabs that fit and refuses
// indexes whose slab is too large for at least FROG_STATIC_MIN_SLOTS warps.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr size_t STATIC_HEADER_WORDS = 64;                          // work counter + spare
constexpr size_t STATIC_SLAB_WORDS = (size_t)4 << 20;               // 4 Mi words = 16 MiB of visited bits
static __device__ __align__(256) uint32_t g_static_scratch[STATIC_HEADER_WORDS + STATIC_SLAB_WORDS];

constexpr int STATIC_MAX_DEVICES = 64;
uint32_t* g_static_ptr[STATIC_MAX_DEVICES] = {};                    // device address of the array, per device
std::mutex g_static_mutex;

// The array's name is only a host-side handle in host code; the device address must be asked
// for, once per device, with that device current.
int static_scratch_for_device(int device, uint32_t** out) {
    if (device < 0 || device >= STATIC_MAX_DEVICES) return FROG_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) {
            froghost::set_cuda_error(e);
            return FROG_ERR_CUDA;
        }
        g_static_ptr[device] = static_cast<uint32_t*>(p);
    }
    *out = g_static_ptr[device];
    return FROG_OK;
}

}  // namespace

extern "C" int frog_search_static(const frog_index_t* index, const float* queries, const int32_t* lo,
                                  const int32_t* hi, int nq, int k, int beam_width, const frog_params_t* params,
                                  int32_t* out_ids, float* out_dists, void* stream) {
    if (!index || nq < 0) return FROG_ERR_INVALID_ARG;
    if (k < 1 || beam_width < 1 || beam_width > FROG_MAX_BEAM_WIDTH || k > beam_width) return FROG_ERR_INVALID_ARG;
    if (nq == 0) return FROG_OK;
    if (!queries || !lo || !hi || !out_ids || !out_dists) return FROG_ERR_INVALID_ARG;
    frog_params_t P;
    int rc = froghost::resolve_params(index, beam_width, params, &P);
    if (rc) return rc;
    // the slab of one warp must fit FROG_STATIC_MIN_SLOTS times: n <= FROG_STATIC_MAX_N
    if (index->info.n > FROG_STATIC_MAX_N) return FROG_ERR_TOO_LARGE;
    const size_t words = bitmap_words_per_slot(index);
    const size_t fit = STATIC_SLAB_WORDS / words;
    if (fit < FROG_STATIC_MIN_SLOTS) return FROG_ERR_TOO_LARGE;
    FROG_CUDA_TRY(cudaSetDevice(index->info.device));
    uint32_t* scratch = nullptr;
    rc = static_scratch_for_device(index->info.device, &scratch);
    if (rc) return rc;
    LaunchPlan plan;
    rc = plan_launch(index, beam_width, P, MODE_FAST, true, nq, &plan, false);
    if (rc) return rc;
    const int max_ctas = (int)(fit / WARPS_PER_CTA);
    if (plan.grid > max_ctas) plan.grid = max_ctas;

    FrogSearchArgs A;
    A.sorted_attr = index->d_sorted_attr;
    A.rank2id = index->d_rank2id;
    A.vectors = index->d_vectors;
    A.enc = index->d_enc;
    A.n = (int)index->info.n;
    A.d = index->info.d;
    A.d_pad = index->info.d_pad;
    A.H = index->info.H;
    A.m = index->info.m;
    A.queries = queries;
    A.lo = lo;
    A.hi = hi;
    A.nq = nq;
    A.k = k;
    A.ef_s = beam_width;
    A.epn = P.epn;
    A.B = P.budget;
    A.max_iters = P.max_iters;
    A.no_hotspot = P.no_hotspot;
    A.exact_w = P.exact_below > beam_width ? P.exact_below : beam_width;
    A.hash_bits = P.hash_bits;
    A.seed = P.seed;
    A.out_ids = out_ids;
    A.out_dists = out_dists;
    A.status = nullptr;
    A.stats = nullptr;
    A.trace = nullptr;
    A.trace_cap = 0;
    A.work_counter = scratch;                               // word 0 of the header
    A.bitmap = scratch + STATIC_HEADER_WORDS;
    A.bitmap_words = words;
    A.slab_stride = words;
    A.log_cap = 0;
    A.slab_clean = 0;                                       // the array may hold anything: clear before use
    A.table = nullptr;
    A.table_bits = 0;
    A.ranges = nullptr;                                     // endpoints and order are computed in the kernel
    A.order = nullptr;
    set_gather(index, P.storage == FROG_STORAGE_F16, &A);

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the array keeps what the previous call left: the counter must restart at zero; every warp
    // clears the slab words of a query's range itself before using them
    FROG_CUDA_TRY(cudaMemsetAsync(scratch, 0, sizeof(unsigned int), s));
    plan.fn<<<plan.grid, plan.block, plan.smem, s>>>(A);
    FROG_CUDA_TRY(cudaGetLastError());
    return FROG_OK;
}


// ---- optional fp16 copy of the vectors (paper Sec. 8.1.4: its GPU programs compute distances from
// float16 data with float32 accumulation) ---------------------------------------------------------
namespace {
__global__ void to_half_kernel(const float* __restrict__ src, int d_pad, __half* __restrict__ dst, int d_pad_h, size_t n) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n * (size_t)d_pad_h) return;
    const size_t r = i / d_pad_h;
    const int c = (int)(i - r * d_pad_h);
    dst[i] = __float2half_rn(c < d_pad ? src[r * d_pad + c] : 0.f);
}
}  // namespace

extern "C" int frog_index_enable_f16(frog_index_t* ix) {
    if (!ix) return FROG_ERR_INVALID_ARG;
    if (ix->d_vectors_h) return FROG_OK;
    FROG_CUDA_TRY(cudaSetDevice(ix->info.device));
    const int d_pad_h = query_len(ix->info.d);
    const size_t elems = (size_t)ix->info.n * d_pad_h;
    cudaError_t e = cudaMalloc(&ix->d_vectors_h, elems * sizeof(__half));
    if (e != cudaSuccess) {
        cudaGetLastError();
        froghost::set_cuda_error(e);
        ix->d_vectors_h = nullptr;
        return FROG_ERR_NOMEM;
    }
    to_half_kernel<<<(unsigned)((elems + 255) / 256), 256>>>(ix->d_vectors, ix->info.d_pad,
                                                             static_cast<__half*>(ix->d_vectors_h), d_pad_h,
                                                             (size_t)ix->info.n);
    FROG_CUDA_TRY(cudaGetLastError());
    FROG_CUDA_TRY(cudaDeviceSynchronize());
    ix->info.device_bytes += (int64_t)(elems * sizeof(__half));
    ix->has_tmap_f16 = froghost::make_row_tensor_map(ix->d_vectors_h, true, d_pad_h, (size_t)d_pad_h * 2,
                                                     (size_t)ix->info.n, &ix->tmap_f16);
    return FROG_OK;
}
