// The search kernel for the common case: fp32 rows of 384 or 512 bytes (d = 96, 128), an exact
// visited set in global scratch (bitmap slab, or for large indexes a hash table of ranks), rows
// fetched four at a time by the copy engine's tile::gather4, no counters and no trace.  It
// computes exactly what frog_search_kernel computes (paper Alg. 2 with Alg. 3 once per query and
// Alg. 4 + the lazy hash check per expansion; same distance order, same merge), and the tests
// compare the two bit for bit.
//
// Why a second kernel: with short rows the general kernel spends 1,000-1,400 warp instructions per
// expansion for 10-20 distance evaluations and keeps 60-70 % of the issue slots busy -- it is bound
// by instruction issue and dependent latency, not by bytes.  Here
//   * the stage buffer is a ring of two quads (4 rows each, one mbarrier per quad) and lane 0
//     issues the copies from one short block (the rank list is padded to a whole quad with rows
//     beyond the tensor, which arrive as zeros, so a copy needs no per-row selects); deeper rings
//     were measured slower;
//   * a team's leader stores its row's squared distance to shared memory, every lane picks up
//     "its" distance with one load (no shuffle/compare chain to route results to lanes);
//   * all survivors of one expansion (up to B: 64, or 128 in the instantiations for large budgets)
//     go through one gather loop;
//   * everything in the expansion loop is inlined (no call, no argument shuffling), the row
//     geometry and the shared-memory layout are compile-time constants;
//   * on indexes of 4M objects and more the visited set is a 16 KB hash table per warp that stays
//     in L2 instead of a bitmap slab of n/8 bytes per warp that does not.
#include "frog_device.cuh"
#include "frog_internal.h"

using namespace frogdev;

namespace {

constexpr int LEAN_WARPS = 2;      // warps per CTA; they never synchronise with each other
// Tuning constants (overridable for scratch builds).  NSLOT: quads (4 rows each) in the stage ring.
// MINB: resident CTAs per SM that the register allocation aims at, per row size and pool size; the
// values are the measured optima.  More than about 100 KB of tensor copies in flight per SM makes
// the copy engine's throughput fall off, which is why 512-byte rows want fewer warps than 384-byte
// rows once the registers of a larger pool cost occupancy anyway.
#ifndef FROG_LEAN_NSLOT_384
#define FROG_LEAN_NSLOT_384 2
#endif
#ifndef FROG_LEAN_NSLOT_512
#define FROG_LEAN_NSLOT_512 2
#endif
#ifndef FROG_LEAN_MINB_384
#define FROG_LEAN_MINB_384 18       // 384-byte rows, pools of 32 and 64 keys: 36 warps at 56 registers (+3 % over 32)
#endif
#ifndef FROG_LEAN_MINB_384_P128
#define FROG_LEAN_MINB_384_P128 16  // ... 128 keys: 32 warps (56 registers spill there; 28 and 24 warps: 5-12 % slower)
#endif
#ifndef FROG_LEAN_MINB_POOL192
#define FROG_LEAN_MINB_POOL192 16   // ... 192 keys (beams 129-192): 32 warps at 64 registers (28: -2 %, 24: -5 %)
#endif
#ifndef FROG_LEAN_MINB_POOL256
#define FROG_LEAN_MINB_POOL256 14   // ... 256 keys: 28 warps at 72 registers (the merge holds 8 keys per lane;
#endif                              // +3-4 % over 24 warps at 80 registers, 32 warps at 64: +1-2 %)
#ifndef FROG_LEAN_MINB_POOL512
#define FROG_LEAN_MINB_POOL512 10   // pools of 512 keys, both row sizes: 20 warps at 96 registers (16 and 24: slower)
#endif
#ifndef FROG_LEAN_MINB_512
#define FROG_LEAN_MINB_512 16       // 512-byte rows, pools of 32 and 64 keys: 32 warps (36: 8 % slower, 28 and 24: 1-2 % slower)
#endif
#ifndef FROG_LEAN_MINB_512_P128
#define FROG_LEAN_MINB_512_P128 12  // ... 128 keys: 24 warps (+12 % over 32)
#endif
#ifndef FROG_LEAN_MINB_512_P192
#define FROG_LEAN_MINB_512_P192 12  // ... 192 keys: 24 warps (28 and 20: 11 % slower)
#endif
#ifndef FROG_LEAN_MINB_512_P256
#define FROG_LEAN_MINB_512_P256 12  // ... 256 keys: 24 warps (+12 % over 28)
#endif
__host__ __device__ constexpr int lean_min_ctas(int epl, int rowb) {
    return rowb <= 384 ? (epl <= 2 ? FROG_LEAN_MINB_384 : epl == 4 ? FROG_LEAN_MINB_384_P128 : epl == 6 ? FROG_LEAN_MINB_POOL192
                          : epl == 8 ? FROG_LEAN_MINB_POOL256 : FROG_LEAN_MINB_POOL512)
                       : (epl <= 2 ? FROG_LEAN_MINB_512 : epl == 4 ? FROG_LEAN_MINB_512_P128 : epl == 6 ? FROG_LEAN_MINB_512_P192
                          : epl == 8 ? FROG_LEAN_MINB_512_P256 : FROG_LEAN_MINB_POOL512);
}

// Scratch builds with -DFROG_LEAN_PROFILE add per-phase cycle counters (summed over all warps into
// g_lean_prof, read back through frog_debug_lean_profile); the shipped library has none of this.
#ifdef FROG_LEAN_PROFILE
__device__ unsigned long long g_lean_prof[8];
#define LEAN_T(i) do { const long long _n = clock64(); t_ph[i] += _n - t_mark; t_mark = _n; } while (0)
#else
#define LEAN_T(i) do { } while (0)
#endif

template <int EPL, int ROWB, int CAP>
struct Lean {
    static constexpr int NSLOT = ROWB <= 384 ? FROG_LEAN_NSLOT_384 : FROG_LEAN_NSLOT_512;   // quads in the ring
    static constexpr int QUAD = 4 * ROWB;                       // bytes of one quad
    static constexpr int POOL = 32 * EPL;
    static constexpr int OFF_POOL = NSLOT * QUAD;
    static constexpr int OFF_CAND = OFF_POOL + POOL * 8;        // <= CAP (64 or 128) ranks + 3 of padding (+ 5 spare)
    static constexpr int OFF_D2 = OFF_CAND + (CAP + 8) * 4;     // squared distances of the <= CAP rows
    static constexpr int OFF_Q = OFF_D2 + CAP * 4;              // query vector, ROWB bytes
    static constexpr int OFF_BAR = OFF_Q + ROWB;                // NSLOT mbarriers, then the time-out flag
    static constexpr int BYTES = (OFF_BAR + 40 + 127) / 128 * 128;
    static_assert(OFF_CAND % 16 == 0 && OFF_Q % 16 == 0 && OFF_BAR % 8 == 0 && QUAD % 128 == 0, "alignment");
};

template <int EPL, int ROWB, int CAP>
struct LeanSmem {
    char* stage;
    uint64_t* pool;
    uint32_t* cand;
    float* d2;
    const float4* q;
    uint64_t* bar;
    uint32_t* timeout;
    __device__ __forceinline__ explicit LeanSmem(unsigned char* base) {
        using L = Lean<EPL, ROWB, CAP>;
        stage = reinterpret_cast<char*>(base);
        pool = reinterpret_cast<uint64_t*>(base + L::OFF_POOL);
        cand = reinterpret_cast<uint32_t*>(base + L::OFF_CAND);
        d2 = reinterpret_cast<float*>(base + L::OFF_D2);
        q = reinterpret_cast<const float4*>(base + L::OFF_Q);
        bar = reinterpret_cast<uint64_t*>(base + L::OFF_BAR);
        timeout = reinterpret_cast<uint32_t*>(base + L::OFF_BAR + L::NSLOT * 8);
    }
};

// Squared distances of the ns <= 128 ranks in cand[0..ns) into d2[0..ns) (Alg. 2 line 14).  `ph`
// holds the parities of the ring's mbarriers.  Arithmetic order: lane s of an 8-lane team takes
// the 4-float groups s, s+8, s+16, ... of its row in increasing order with fused multiply-adds,
// then the partial sums are combined by a butterfly with partner distance 4, 2, 1.
// HOOK (an instantiation of its own, for the test of the error path): no copy is armed or issued and a
// wait gives up after 64 polls, so every gather ends in the time-out branch without anything in flight.
template <int EPL, int ROWB, int CAP, bool HOOK = false>
__device__ __forceinline__ void lean_gather(const FrogSearchArgs& A, const LeanSmem<EPL, ROWB, CAP>& S, int ns,
                                            uint32_t& ph, int lane) {
    using L = Lean<EPL, ROWB, CAP>;
    const int groups = (ns + 3) >> 2;
    if (lane < 3) S.cand[ns + lane] = (uint32_t)A.n + 1u + (uint32_t)lane;    // rows beyond the tensor: zeros
    __syncwarp();
    const uint64_t policy = l2_policy_evict_first();                           // rows are read about once per batch
    auto issue = [&](int g, int slot) {
        if (HOOK) return;
        uint64_t* b = S.bar + slot;
        mbar_expect_tx(b, (uint32_t)L::QUAD);
        const uint4 rk = *reinterpret_cast<const uint4*>(S.cand + 4 * g);
        tma_gather4(S.stage + slot * L::QUAD, &A.tmap, 0, (int)rk.x, (int)rk.y, (int)rk.z, (int)rk.w, b, policy);
    };
    if (lane == 0) {
#pragma unroll
        for (int g = 0; g < L::NSLOT; ++g)
            if (g < groups) issue(g, g);
    }
    const int team = lane >> 3, sub = lane & 7;
    const char* mine = S.stage + team * ROWB + sub * 16;
    int slot = 0;
#pragma unroll 1
    for (int g = 0; g < groups; ++g) {
        if (!(HOOK ? mbar_wait_limit(S.bar + slot, (ph >> slot) & 1u, 64) : mbar_wait(S.bar + slot, (ph >> slot) & 1u))) *S.timeout = 1u;
        ph ^= 1u << slot;
        const char* x = mine + slot * L::QUAD;
        float a = 0.f;
#pragma unroll
        for (int c = 0; c < ROWB / 128; ++c) {
            const float4 xv = *reinterpret_cast<const float4*>(x + c * 128);
            const float4 qv = S.q[sub + 8 * c];
            float t;
            t = xv.x - qv.x; a = fmaf(t, t, a);
            t = xv.y - qv.y; a = fmaf(t, t, a);
            t = xv.z - qv.z; a = fmaf(t, t, a);
            t = xv.w - qv.w; a = fmaf(t, t, a);
        }
        a = a + __shfl_xor_sync(FULL, a, 4);
        a = a + __shfl_xor_sync(FULL, a, 2);
        a = a + __shfl_xor_sync(FULL, a, 1);
        if (sub == 0) S.d2[4 * g + team] = a;
        __syncwarp();                                       // every lane is done reading this quad
        if (lane == 0 && g + L::NSLOT < groups) issue(g + L::NSLOT, slot);
        slot = (slot + 1 == L::NSLOT) ? 0 : slot + 1;
    }
    __syncwarp();
}

// MergeTopEfS of 32 of the ns <= 128 evaluated candidates, those from `off` on (lines 15-17: merging
// them batch by batch leaves the pool that one merge of all would); returns the first unexpanded position.
template <int EPL, int ROWB, int CAP>
__device__ __forceinline__ int lean_merge(const LeanSmem<EPL, ROWB, CAP>& S, int ns, int ef_s, uint32_t new_flag, int off, int lane) {
    const int j = off + lane;
    const uint64_t key = (j < ns) ? make_key(S.d2[j], S.cand[j], new_flag) : KEY_EMPTY;
    return (int)merge_batch<EPL, true>(S.pool, key, ef_s, lane);
}

// gather + merge out of line, for the places that run once per query (entry points, exact scan) and
// the rare second batch of an expansion; returns first | parities << 16
template <int EPL, int ROWB, int CAP, bool HOOK = false>
__device__ __noinline__ uint32_t lean_eval_cold(const FrogSearchArgs& A, unsigned char* base, int ns, uint32_t new_flag,
                                                uint32_t ph) {
    const LeanSmem<EPL, ROWB, CAP> S(base);
    const int lane = lane_id();
    lean_gather<EPL, ROWB, CAP, HOOK>(A, S, ns, ph, lane);
    int first = lean_merge<EPL, ROWB, CAP>(S, ns, A.ef_s, new_flag, 0, lane);
    for (int off = 32; off < ns; off += 32) first = lean_merge<EPL, ROWB, CAP>(S, ns, A.ef_s, new_flag, off, lane);
    return (uint32_t)first | (ph << 16);
}
template <int EPL, int ROWB, int CAP>
__device__ __noinline__ int lean_merge_cold(unsigned char* base, int ns, int ef_s, uint32_t new_flag, int off) {
    const LeanSmem<EPL, ROWB, CAP> S(base);
    return lean_merge<EPL, ROWB, CAP>(S, ns, ef_s, new_flag, off, lane_id());
}

// Visited check of the cnt <= 64 ranks in en[] (EN order; a longer list is passed in two parts): survivors are compacted, in order, into
// cand[]; returns their number.  Lane l looks after en[l] and en[l + 32].  With `table` the set is the
// warp's hash table (L2-resident), otherwise its bitmap slab.
__device__ __forceinline__ int lean_visit_list(const uint32_t* en, int cnt, uint32_t* cand, uint32_t* table, int table_bits,
                                               uint32_t* bitmap, uint64_t policy, uint32_t* timeout, int lane) {
    const uint32_t lt_mask = (1u << lane) - 1u;
    const bool ha = lane < cnt, hb = lane + 32 < cnt;
    const uint32_t va = ha ? en[lane] : 0u, vb = hb ? en[lane + 32] : 0u;
    bool fa, fb;
    if (table) {
        if (!table_insert2(table, table_bits, va, ha, vb, hb, fa, fb, policy)) *timeout = 1u;
    } else {
        const uint32_t bit_a = 1u << (va & 31), bit_b = 1u << (vb & 31);
        uint32_t old_a = 0xFFFFFFFFu, old_b = 0xFFFFFFFFu;
        if (ha) old_a = atomic_or_l2(bitmap + (va >> 5), bit_a, policy);
        if (hb) old_b = atomic_or_l2(bitmap + (vb >> 5), bit_b, policy);
        fa = (old_a & bit_a) == 0;
        fb = (old_b & bit_b) == 0;
    }
    const uint32_t Ka = __ballot_sync(FULL, fa), Kb = __ballot_sync(FULL, fb);
    const int na = __popc(Ka);
    if (fa) cand[__popc(Ka & lt_mask)] = va;
    if (fb) cand[na + __popc(Kb & lt_mask)] = vb;
    __syncwarp();
    return na + __popc(Kb);
}

// TABLE: the visited set of a query is a hash table of ranks in global scratch (A.table, 1 << table_bits
// slots per warp: 16 KB, so that the tables of all resident warps stay in L2 and the test-and-set of a
// candidate costs no DRAM access; the bitmap's scattered read-modify-writes are what keeps DRAM from the
// row gathers on large indexes).  The table is exact; a query that fills it half way moves its entries
// to the warp's bitmap slab and carries on there.
template <int EPL, int ROWB, bool TABLE, int CAP = 64, bool HOOK = false>
__global__ void __launch_bounds__(LEAN_WARPS * 32, lean_min_ctas(EPL, ROWB))
frog_search_lean_kernel(const __grid_constant__ FrogSearchArgs A) {
    using L = Lean<EPL, ROWB, CAP>;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int lane = lane_id();
    const int warp = threadIdx.x >> 5;
    unsigned char* base = smem_raw + L::BYTES * warp;
    const LeanSmem<EPL, ROWB, CAP> S(base);
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < L::NSLOT; ++i) mbar_init(S.bar + i, 1u);
        *S.timeout = 0u;
    }
    __syncwarp();
    uint32_t ph = 0;                                         // parities of the ring's mbarriers
#ifdef FROG_LEAN_PROFILE
    long long t_ph[8] = {0, 0, 0, 0, 0, 0, 0, 0};           // set-up, ENC+visited, gather, merge, output, idle, expansions
    long long t_mark = clock64();
#endif
    const size_t warp_id = (size_t)(blockIdx.x * LEAN_WARPS + warp);
    uint32_t* bitmap = A.bitmap + warp_id * A.slab_stride;
    uint32_t* const my_table = TABLE ? A.table + (warp_id << A.table_bits) : nullptr;
    uint32_t* en = reinterpret_cast<uint32_t*>(S.d2);        // admitted ENs of an expansion (the distances come later)
    const uint32_t lt_mask = (1u << lane) - 1u;
    const uint64_t keep_in_l2 = l2_policy_evict_last();      // for the visited set of the running query

    for (;;) {
        int q = 0;
        if (lane == 0) {
            q = (int)atomicAdd(A.work_counter, 1u);
            if (q < A.nq && A.order) q = __ldg(A.order + q);
        }
        q = __shfl_sync(FULL, q, 0);
        if (q >= A.nq) break;
        LEAN_T(5);

        // ---- per-query set-up ---------------------------------------------------------------
        {
            float* qf = reinterpret_cast<float*>(base + L::OFF_Q);
            const float* src = A.queries + (size_t)q * A.d;
            for (int i = lane; i < ROWB / 4; i += 32) qf[i] = i < A.d ? __ldg(src + i) : 0.f;
            for (int i = lane; i < L::POOL; i += 32) S.pool[i] = KEY_EMPTY;
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
        uint32_t st = 0;
        __syncwarp();

        if (w <= 0) {
            st |= FROG_ST_EMPTY;
        } else if (w <= A.exact_w) {
            // every valid object is evaluated, the pool keeps the ef_s nearest: exact answer
            st |= FROG_ST_EXACT;
            for (int b0 = 0; b0 < w; b0 += 64) {
                const int cnt = min(64, w - b0);
                if (lane < cnt) S.cand[lane] = (uint32_t)(l_q + b0 + lane);
                if (lane + 32 < cnt) S.cand[lane + 32] = (uint32_t)(l_q + b0 + lane + 32);
                __syncwarp();
                ph = lean_eval_cold<EPL, ROWB, CAP, HOOK>(A, base, cnt, 1u, ph) >> 16;
                __syncwarp();
            }
        } else {
            // Visited set.  TABLE: the warp's hash table (empty here), until the query outgrows it.
            // Otherwise the bitmap slab: all-zero here (slab_clean) or zeroed now; see frog_search.cu.
            uint32_t* table = my_table;
            int n_seen = 0;                                         // ranks in the table
            int n_logged = -1;
            if (!TABLE) {
                const int w0 = l_q >> 5, w1 = r_q >> 5;
                if (!A.slab_clean)
                    for (int i = w0 + lane; i <= w1; i += 32) st_u32_l2(bitmap + i, 0u, keep_in_l2);
                else if (A.log_cap > 0 && w1 - w0 >= SPARSE_MIN_WORDS)
                    n_logged = 0;
            }
            int L_start, L_end;
            hotspot_layers(l_q, r_q, A.H, A.n, L_start, L_end);          // Alg. 2 line 1
            if (A.no_hotspot) { L_start = 0; L_end = A.H - 1; }
            const int total = (L_end - L_start + 1) * A.m;
            const uint32_t span = (uint32_t)(r_q - l_q);
            __syncwarp();
            // lines 2-5: entry points, passed through the visited set
            int ns;
            if (TABLE) {
                if (lane < A.epn) en[lane] = entry_point(A.seed, (uint32_t)l_q, (uint32_t)r_q, lane);
                __syncwarp();
                ns = lean_visit_list(en, A.epn, S.cand, table, A.table_bits, bitmap, keep_in_l2, S.timeout, lane);
                n_seen = ns;
            } else {
                const uint32_t ep = entry_point(A.seed, (uint32_t)l_q, (uint32_t)r_q, lane);
                bool keep = lane < A.epn;
                if (keep) {
                    const uint32_t bit = 1u << (ep & 31);
                    keep = (atomicOr(bitmap + (ep >> 5), bit) & bit) == 0;
                }
                const uint32_t M = __ballot_sync(FULL, keep);
                if (keep) S.cand[__popc(M & lt_mask)] = ep;
                ns = __popc(M);
                __syncwarp();
            }
            if (n_logged >= 0) n_logged = log_ranks(bitmap + A.bitmap_words, A.log_cap, n_logged, S.cand, ns, lane);
            int first;
            {
                const uint32_t r = lean_eval_cold<EPL, ROWB, CAP, HOOK>(A, base, ns, 0u, ph);
                first = (int)(r & 0xFFFFu);
                ph = r >> 16;
            }
            int n_exp = 0;
            LEAN_T(0);
            // lines 7-17
            while (first < A.ef_s) {
                if (n_exp >= A.max_iters) { st |= FROG_ST_ITER_CAP; break; }
                const uint32_t u = key_rank(S.pool[first]);               // line 8
                __syncwarp();
                if (lane == 0) S.pool[first] |= 1ull;                     // line 9
                if (TABLE && table && n_seen + A.B > (1 << (A.table_bits - 1))) {
                    // the next expansion could take the table past half full: move every rank to the
                    // bitmap slab (all-zero until now) and carry on there; the slab is zeroed by range at the end
                    for (int i = lane; i < (1 << A.table_bits); i += 32) {
                        const uint32_t v = __ldcg(table + i);
                        if (v != TABLE_EMPTY) atomicOr(bitmap + (v >> 5), 1u << (v & 31));
                    }
                    __syncwarp();
                    table = nullptr;
                }
                // line 10, Alg. 4 over rows L_start..L_end of ENC(u), four 32-entry chunks per round
                // trip, admission under budget B across the chunks in order
                const uint32_t* hot = A.enc + ((size_t)u * A.H + L_start) * A.m;
                int cnt = 0;
                ns = 0;
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
                    const bool pred1 = rem1 > 0 && ((v1 - (uint32_t)l_q) <= span);
                    const uint32_t M1 = __ballot_sync(FULL, pred1);
                    const int a1 = min(__popc(M1), rem1);
                    const int rank1 = __popc(M1 & lt_mask);
                    const bool adm1 = pred1 && rank1 < a1;
                    const int rem2 = rem1 - a1;
                    const bool pred2 = rem2 > 0 && ((v2 - (uint32_t)l_q) <= span);
                    const uint32_t M2 = __ballot_sync(FULL, pred2);
                    const int a2 = min(__popc(M2), rem2);
                    const int rank2 = __popc(M2 & lt_mask);
                    const bool adm2 = pred2 && rank2 < a2;
                    const int rem3 = rem2 - a2;
                    const bool pred3 = rem3 > 0 && ((v3 - (uint32_t)l_q) <= span);
                    const uint32_t M3 = __ballot_sync(FULL, pred3);
                    const int a3 = min(__popc(M3), rem3);
                    const int rank3 = __popc(M3 & lt_mask);
                    const bool adm3 = pred3 && rank3 < a3;
                    if (TABLE) {
                        // lines 12-13 come after the scan: the admitted ENs are listed in order first
                        if (adm0) en[cnt + rank0] = v0;
                        if (adm1) en[cnt + a0 + rank1] = v1;
                        if (adm2) en[cnt + a0 + a1 + rank2] = v2;
                        if (adm3) en[cnt + a0 + a1 + a2 + rank3] = v3;
                    } else {
                        // lines 12-13: the admitted lanes test-and-set their visited bits in place,
                        // survivors are compacted into cand[]
                        const uint32_t bit0 = 1u << (v0 & 31), bit1 = 1u << (v1 & 31);
                        const uint32_t bit2 = 1u << (v2 & 31), bit3 = 1u << (v3 & 31);
                        uint32_t old0 = 0xFFFFFFFFu, old1 = 0xFFFFFFFFu, old2 = 0xFFFFFFFFu, old3 = 0xFFFFFFFFu;
                        if (adm0) old0 = atomic_or_l2(bitmap + (v0 >> 5), bit0, keep_in_l2);
                        if (adm1) old1 = atomic_or_l2(bitmap + (v1 >> 5), bit1, keep_in_l2);
                        if (adm2) old2 = atomic_or_l2(bitmap + (v2 >> 5), bit2, keep_in_l2);
                        if (adm3) old3 = atomic_or_l2(bitmap + (v3 >> 5), bit3, keep_in_l2);
                        const bool keep0 = (old0 & bit0) == 0, keep1 = (old1 & bit1) == 0;
                        const bool keep2 = (old2 & bit2) == 0, keep3 = (old3 & bit3) == 0;
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
                    }
                    cnt += a0 + a1 + a2 + a3;
                }
                __syncwarp();
                if (TABLE) {
                    ns = lean_visit_list(en, min(cnt, 64), S.cand, table, A.table_bits, bitmap, keep_in_l2, S.timeout, lane);
                    if (cnt > 64)
                        ns += lean_visit_list(en + 64, cnt - 64, S.cand + ns, table, A.table_bits, bitmap, keep_in_l2,
                                              S.timeout, lane);
                    n_seen += ns;
                }
                ++n_exp;
                if (n_logged >= 0) n_logged = log_ranks(bitmap + A.bitmap_words, A.log_cap, n_logged, S.cand, ns, lane);
                // lines 14-17
                LEAN_T(1);
                lean_gather<EPL, ROWB, CAP, HOOK>(A, S, ns, ph, lane);
                LEAN_T(2);
                first = lean_merge<EPL, ROWB, CAP>(S, ns, A.ef_s, 0u, 0, lane);
                for (int off = 32; off < ns; off += 32) first = lean_merge_cold<EPL, ROWB, CAP>(base, ns, A.ef_s, 0u, off);
                LEAN_T(3);
#ifdef FROG_LEAN_PROFILE
                t_ph[6] += 1;
                t_ph[7] += ns;
#endif
            }
            if (TABLE) {
                // empty the table again; a query that moved to the slab zeroes the words of its range
                const uint4 e4 = make_uint4(TABLE_EMPTY, TABLE_EMPTY, TABLE_EMPTY, TABLE_EMPTY);
                uint4* t4 = reinterpret_cast<uint4*>(my_table);
                for (int i = lane; i < (1 << (A.table_bits - 2)); i += 32) __stcg(t4 + i, e4);
                if (!table) {
                    const int w0 = l_q >> 5, w1 = r_q >> 5;
                    for (int i = w0 + lane; i <= w1; i += 32) bitmap[i] = 0u;
                }
            } else if (A.slab_clean) {
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
        const bool bad = *S.timeout != 0u;                  // a copy never completed: the row is not valid
        int got = 0;
        for (int j = lane; j < A.k; j += 32) {
            const uint64_t key = S.pool[j];
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
        if (bad && lane == 0) atomicOr(A.work_counter + 1, FROG_ST_COPY_TIMEOUT);   // sticky word of this launch
        if (A.status) {
            got = __reduce_add_sync(FULL, got);
            if (got < A.k) st |= FROG_ST_SHORT;
            if (bad) st |= FROG_ST_COPY_TIMEOUT;
            if (lane == 0) A.status[q] = st;
        }
        __syncwarp();
        LEAN_T(4);
    }
#ifdef FROG_LEAN_PROFILE
    if (lane == 0)
        for (int i = 0; i < 8; ++i) atomicAdd(g_lean_prof + i, (unsigned long long)t_ph[i]);
#endif
}

// Budgets up to 64 get the compact shared-memory layout (CAP = 64: what keeps 32-36 warps resident
// inside the 196 KB carve-out, so that L1 keeps 60 KB; the larger layout was measured 4-9 % slower at
// B <= 64); budgets up to 128 are instantiated for the pools of 128-256 keys, where they pay (hard,
// narrow-range batches); other combinations go to the general kernel.
template <int ROWB>
frog_kernel_fn lean_pick(int ef_s, int budget, bool table, bool hook, size_t* smem_per_warp) {
    if (hook) {
        if (table || budget > 64 || ef_s > 32) return nullptr;
        *smem_per_warp = Lean<1, ROWB, 64>::BYTES;
        return frog_search_lean_kernel<1, ROWB, false, 64, true>;
    }
    if (budget > 64) {
        if (ef_s <= 64 || ef_s > 256 || (table && ef_s > 128)) return nullptr;
        if (ef_s <= 128) { *smem_per_warp = Lean<4, ROWB, 128>::BYTES; return table ? frog_search_lean_kernel<4, ROWB, true, 128> : frog_search_lean_kernel<4, ROWB, false, 128>; }
        if (ef_s <= 192) { *smem_per_warp = Lean<6, ROWB, 128>::BYTES; return frog_search_lean_kernel<6, ROWB, false, 128>; }
        *smem_per_warp = Lean<8, ROWB, 128>::BYTES;
        return frog_search_lean_kernel<8, ROWB, false, 128>;
    }
    if (ef_s <= 32) { *smem_per_warp = Lean<1, ROWB, 64>::BYTES; return table ? frog_search_lean_kernel<1, ROWB, true> : frog_search_lean_kernel<1, ROWB, false>; }
    if (ef_s <= 64) { *smem_per_warp = Lean<2, ROWB, 64>::BYTES; return table ? frog_search_lean_kernel<2, ROWB, true> : frog_search_lean_kernel<2, ROWB, false>; }
    if (ef_s <= 128) { *smem_per_warp = Lean<4, ROWB, 64>::BYTES; return table ? frog_search_lean_kernel<4, ROWB, true> : frog_search_lean_kernel<4, ROWB, false>; }
    if (table) return nullptr;
    if (ef_s <= 192) { *smem_per_warp = Lean<6, ROWB, 64>::BYTES; return frog_search_lean_kernel<6, ROWB, false>; }
    if (ef_s <= 256) { *smem_per_warp = Lean<8, ROWB, 64>::BYTES; return frog_search_lean_kernel<8, ROWB, false>; }
    *smem_per_warp = Lean<16, ROWB, 64>::BYTES;
    return frog_search_lean_kernel<16, ROWB, false>;
}

}  // namespace

namespace froghost {

// The lean kernel for this beam width and row size, or null if the shape is not covered (the caller
// then uses the generic kernel).  Needs the row tensor map and the bitmap visited set.  `table`: the
// variant whose visited set is the L2-resident hash table (pools of up to 128 keys only); `hook`: the
// instantiation whose gathers time out by construction (bitmap form, beams up to 32, budgets up to 64).
frog_kernel_fn lean_kernel(int ef_s, int budget, int row_bytes, bool table, bool hook, size_t* smem_per_warp,
                           int* warps_per_cta) {
    *warps_per_cta = LEAN_WARPS;
    if (row_bytes == 384) return lean_pick<384>(ef_s, budget, table, hook, smem_per_warp);
    if (row_bytes == 512) return lean_pick<512>(ef_s, budget, table, hook, smem_per_warp);
    return nullptr;
}

}  // namespace froghost

#ifdef FROG_LEAN_PROFILE
extern "C" int frog_debug_lean_profile(unsigned long long* out8, int reset) {
    if (cudaMemcpyFromSymbol(out8, g_lean_prof, sizeof(unsigned long long) * 8) != cudaSuccess) return 5;
    if (reset) {
        unsigned long long z[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (cudaMemcpyToSymbol(g_lean_prof, z, sizeof(z)) != cudaSuccess) return 5;
    }
    return 0;
}
#endif
