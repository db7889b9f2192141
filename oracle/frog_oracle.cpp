// CPU oracle for FROG query processing -- TEST INFRASTRUCTURE, not part of the product.
//
// A plain, slow, sequential restatement of what the search path computes, written from the
// paper (FROG: range-filtering approximate nearest neighbour search on GPUs) and sharing no
// code with the CUDA library.  Only the tests, the smoke check and the benchmark's CPU-baseline
// leg may call it.  Every function names the passage it follows.
//
// Two kinds of function live here:
//   (G) the plain definition: exact filtered k-nearest neighbours (Def. 2, Sec. 2.1);
//   (O) the search algorithm step by step: Alg. 2 (FROGSearch), Alg. 3 (HotspotLocalization),
//       Alg. 4 (ENIdentification), the lazy hash check of Sec. 7.3.2, and the attribute ->
//       rank endpoint conversion of Sec. 4.
//
// Readings taken where the paper is silent (each one is also listed in the design notes):
//   * vertex id == attribute rank; ENC entries are ranks; the empty entry is 0xFFFFFFFF.
//   * H = max(1, ceil(log2 n) + 1 - n_inv) (stored in the index, never recomputed here).
//   * BoundaryRefinementInvalid (Alg. 3 line 18, body not printed): Eq. 6 evaluated in integers
//     with a boundary represented, as in Alg. 3, by the last rank of the segment on its left.
//   * entry points: a stateless 64-bit mixer of (seed, l_q, r_q, j); duplicates are removed by
//     the visited set.
//   * distances: squared L2 in fp32 with a fixed summation order (8 interleaved partial sums
//     over 4-float groups, fused multiply-add, then a 3-level pairwise butterfly); order and
//     ties are decided on the squared value, ties broken by rank; reported distance =
//     sqrtf(squared).
//   * visited set: exact, never erased.  Hard cap on expansions (max_iters).
//   * a range holding at most ef_s objects is answered exactly (every object enters the pool);
//     the option exact_below = T extends this to ranges of at most max(ef_s, T) objects.
//   * ablation options: no_hotspot (scan all H layers), eager_hash (visited test inside the
//     predicate of Alg. 4 instead of after selection and budget).
//
// Parity unpinned by the paper: the +-1 convention of Eq. 6 (pinned only by the reading
// above), and recall levels (the paper's curves are figures on datasets not available here).
//
// Build: g++ -O2 -ffp-contract=off -fopenmp -shared -fPIC (no fast-math; fmaf is explicit).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <set>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

constexpr uint32_t BOT = 0xFFFFFFFFu;   // empty ENC entry

// ---------------------------------------------------------------------------------------------
// Sec. 4: attribute -> rank.  Objects are sorted ascending by attribute and numbered 0..n-1;
// a query's [lo, hi] becomes the rank interval holding exactly the valid objects, found by
// lower- and upper-bound lookup.
// ---------------------------------------------------------------------------------------------
void rank_interval(const int32_t* sorted_attr, int64_t n, int32_t lo, int32_t hi,
                   int64_t* l_q, int64_t* r_q) {
    const int32_t* b = sorted_attr;
    const int32_t* e = sorted_attr + n;
    *l_q = std::lower_bound(b, e, lo) - b;          // first rank with attr >= lo
    *r_q = (std::upper_bound(b, e, hi) - b) - 1;    // last rank with attr <= hi
}

// ---------------------------------------------------------------------------------------------
// Sec. 4 / Alg. 3 lines 1-12: the implicit segment tree.  The root covers [0, N-1]; a node
// [L, R] splits at mid = L + floor((R-L)/2) into [L, mid] and [mid+1, R].  Returns the layer-h
// segment that contains rank x.
// ---------------------------------------------------------------------------------------------
void segment_at(int64_t N, int h, int64_t x, int64_t* L_out, int64_t* R_out) {
    int64_t L = 0, R = N - 1;
    for (int depth = 0; depth < h; ++depth) {
        int64_t mid = L + (R - L) / 2;
        if (x <= mid) R = mid; else L = mid + 1;
    }
    *L_out = L;
    *R_out = R;
}

// Eq. 6 (Rule 2 of Sec. 7.2).  b_l / b_r are the leftmost / rightmost layer-h segment
// boundaries inside [l_q, r_q]; a boundary is the last rank of the segment on its left and is
// inside the range iff l_q <= b < r_q.  Layer h is valid iff
//     (b_l - l_q) + (r_q - b_r) >= 2^-h (r_q - l_q),
// evaluated exactly as ((b_l - l_q) + (r_q - b_r)) * 2^h >= (r_q - l_q) in 64-bit integers.
bool boundary_refinement_invalid(int64_t l_q, int64_t r_q, int h, int64_t N) {
    int64_t Ll, Rl, Lr, Rr;
    segment_at(N, h, l_q, &Ll, &Rl);
    segment_at(N, h, r_q, &Lr, &Rr);
    (void)Ll; (void)Rr;
    int64_t b_l = Rl;        // last rank of the segment holding l_q
    int64_t b_r = Lr - 1;    // boundary just left of the segment holding r_q
    int64_t lhs = (b_l - l_q) + (r_q - b_r);
    int64_t rhs = r_q - l_q;
    // lhs * 2^h >= rhs, with h < 63 and lhs, rhs < 2^31 in practice; guard the shift anyway
    if (h >= 31) return !(lhs > 0 || rhs == 0);
    return !((lhs << h) >= rhs);
}

// ---------------------------------------------------------------------------------------------
// Alg. 3: HotspotLocalization(l_q, r_q, H, N) -> (L_start, L_end).
// Rule 1 (the descent of Alg. 3 lines 1-12), stated by what it finds rather than how: the walk
// from the root follows the child that holds the whole range and stops where the range is cut,
// so L_start is the deepest retained layer at which l_q and r_q still lie in the same segment.
// Rule 2 (lines 13-22): L_end grows over the following layers while Eq. 6 holds.
// ---------------------------------------------------------------------------------------------
void hotspot_localization(int64_t l_q, int64_t r_q, int H, int64_t N, int* L_start, int* L_end) {
    int deepest_shared = 0;                       // layer 0 is one segment: it always holds both ends
    for (int h = 1; h <= H - 1; ++h) {
        int64_t La, Ra, Lb, Rb;
        segment_at(N, h, l_q, &La, &Ra);
        segment_at(N, h, r_q, &Lb, &Rb);
        if (La != Lb) break;                      // the layer-h segmentation cuts [l_q, r_q]
        (void)Ra; (void)Rb;
        deepest_shared = h;
    }
    *L_start = deepest_shared;
    *L_end = deepest_shared;
    for (int h = deepest_shared + 1; h <= H - 1; ++h) {
        if (boundary_refinement_invalid(l_q, r_q, h, N)) break;
        *L_end = h;
    }
}

// ---------------------------------------------------------------------------------------------
// Alg. 4: ENIdentification.  One warp of `warp` lanes scans the hotspot rows of ENC(u) in
// warp-sized chunks; each lane holds one candidate, the ballot mask M and its population counts
// give every passing lane a dense output slot, and the budget B admits a prefix.
// enc_u points at the H x m block of vertex u.  Returns |EN(u)|; *rows_read = number of m-wide
// layer rows the scan touched (for the traffic model).
// ---------------------------------------------------------------------------------------------
int en_identification(const uint32_t* enc_u, int m, int64_t l_q, int64_t r_q,
                      int L_start, int L_end, int B, int warp, uint32_t* EN, int* rows_read) {
    int size_EN = 0;
    int rows = 0;
    if (B <= 0) { if (rows_read) *rows_read = 0; return 0; }
    // The rows L_start..L_end are contiguous in memory; a chunk is `warp` consecutive entries.
    const uint32_t* hot = enc_u + (int64_t)L_start * m;
    int total = (L_end - L_start + 1) * m;
    for (int c0 = 0; c0 < total; c0 += warp) {
        int c1 = std::min(total, c0 + warp);
        rows = (c1 + m - 1) / m;
        // each lane loads one candidate and evaluates the predicate
        uint64_t M = 0;
        for (int lane = 0; lane < c1 - c0; ++lane) {
            uint32_t v = hot[c0 + lane];
            bool pred = (v != BOT) && (l_q <= (int64_t)v) && ((int64_t)v <= r_q);
            if (pred) M |= (uint64_t)1 << lane;
        }
        int n = __builtin_popcountll(M);
        int base = size_EN;
        int a = std::min(n, B - base);
        for (int lane = 0; lane < c1 - c0; ++lane) {
            bool pred = (M >> lane) & 1;
            int rank = __builtin_popcountll(M & (((uint64_t)1 << lane) - 1));
            if (pred && rank < a) EN[base + rank] = hot[c0 + lane];
        }
        size_EN = base + a;
        if (size_EN == B) break;
    }
    if (rows_read) *rows_read = rows;
    return size_EN;
}

// ---------------------------------------------------------------------------------------------
// Ablation of the lazy hash check (Sec. 6.2): the EAGER form puts the visited test into the
// predicate of Alg. 4, so an id that was already evaluated neither occupies a slot nor consumes
// budget.  Chunk semantics as in Alg. 4: all lanes of a chunk test against the visited set as it
// stood when the chunk was loaded; the admitted prefix is then inserted, in order (a second copy
// of an id inside the same chunk is admitted, fails the insertion and is not evaluated).
// `fresh` receives the admitted ids that were inserted, in order.
// ---------------------------------------------------------------------------------------------
int en_identification_eager(const uint32_t* enc_u, int m, int64_t l_q, int64_t r_q,
                            int L_start, int L_end, int B, int warp, std::set<uint32_t>& visited,
                            uint32_t* EN, std::vector<uint32_t>& fresh, int* rows_read) {
    int size_EN = 0;
    int rows = 0;
    fresh.clear();
    if (B <= 0) { if (rows_read) *rows_read = 0; return 0; }
    const uint32_t* hot = enc_u + (int64_t)L_start * m;
    int total = (L_end - L_start + 1) * m;
    for (int c0 = 0; c0 < total; c0 += warp) {
        int c1 = std::min(total, c0 + warp);
        rows = (c1 + m - 1) / m;
        std::vector<uint32_t> pass;
        for (int lane = 0; lane < c1 - c0; ++lane) {
            uint32_t v = hot[c0 + lane];
            bool pred = (v != BOT) && (l_q <= (int64_t)v) && ((int64_t)v <= r_q) && !visited.count(v);
            if (pred) pass.push_back(v);
        }
        int a = std::min<int>((int)pass.size(), B - size_EN);
        for (int j = 0; j < a; ++j) {
            EN[size_EN++] = pass[j];
            if (visited.insert(pass[j]).second) fresh.push_back(pass[j]);
        }
        if (size_EN == B) break;
    }
    if (rows_read) *rows_read = rows;
    return size_EN;
}

// ---------------------------------------------------------------------------------------------
// Squared L2 distance in fp32, fixed order.  The d floats are cut into 4-float groups; group g
// goes to partial sum g mod 8; each partial sum takes its groups in increasing g, elements in
// increasing index, acc = fma(x - q, x - q, acc); then the 8 partial sums are combined by a
// butterfly with partner distances 4, 2, 1 (a[t] += a[t ^ off], all t at once).
// d must be a multiple of 4 (rows are zero-padded to that by the index format).
// ---------------------------------------------------------------------------------------------
float dist2_canonical(const float* q, const float* x, int d) {
    float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    int groups = d / 4;
    for (int g = 0; g < groups; ++g) {
        int t = g & 7;
        for (int e = 0; e < 4; ++e) {
            float diff = x[4 * g + e] - q[4 * g + e];
            a[t] = fmaf(diff, diff, a[t]);
        }
    }
    for (int off = 4; off >= 1; off >>= 1) {
        float b[8];
        for (int t = 0; t < 8; ++t) b[t] = a[t] + a[t ^ off];
        for (int t = 0; t < 8; ++t) a[t] = b[t];
    }
    return a[0];
}

// Sec. 2.1 definition in double precision (used by (G) in its reference mode).
double dist2_f64(const float* q, const float* x, int d) {
    double s = 0.0;
    for (int i = 0; i < d; ++i) {
        double diff = (double)x[i] - (double)q[i];
        s += diff * diff;
    }
    return s;
}

// ---------------------------------------------------------------------------------------------
// Alg. 2 line 3: "uniformly sample ep_j from [l_q, r_q]".  Stateless generator so that the
// result depends on the range only: x = seed ^ l*K1 ^ r*K2 ^ j*K3, the splitmix64 finaliser,
// then the top 32 bits scaled into [0, w) by a multiply-high.
// ---------------------------------------------------------------------------------------------
uint64_t mix64(uint64_t x) {
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

int64_t entry_point(uint64_t seed, int64_t l_q, int64_t r_q, int j) {
    uint64_t x = seed ^ ((uint64_t)l_q * 0x9E3779B97F4A7C15ull)
                      ^ ((uint64_t)r_q * 0xC2B2AE3D27D4EB4Full)
                      ^ ((uint64_t)(j + 1) * 0x165667B19E3779F9ull);
    x = mix64(x);
    uint64_t w = (uint64_t)(r_q - l_q + 1);
    return l_q + (int64_t)(((x >> 32) * w) >> 32);
}

struct Cand {            // (id, dist, flag) triple of Alg. 2; id is a rank
    float dist2;
    uint32_t id;
    int flag;
};

// total order of the pool: squared distance ascending, then rank ascending
bool cand_less(const Cand& a, const Cand& b) {
    if (a.dist2 != b.dist2) return a.dist2 < b.dist2;
    return a.id < b.id;
}

struct Index {
    const int32_t* sorted_attr;
    const int32_t* rank2id;
    const float* vectors;     // n x d_pad, rank order
    const uint32_t* enc;      // n x H x m
    int64_t n;
    int d_pad;
    int H;
    int m;
};

struct Params {
    int epn;
    int B;
    int max_iters;
    uint64_t seed;
    int warp;        // chunk width of Alg. 4 (32; any value gives the same EN list)
    int no_hotspot;  // ablation: scan all H layers
    int exact_below; // ranges of at most this many objects are answered by the exact scan too (0: off)
    int eager_hash;  // ablation: visited test inside the predicate of Alg. 4 instead of after it
};

// status bits
constexpr uint32_t ST_EMPTY = 1u, ST_EXACT = 2u, ST_ITER_CAP = 4u, ST_SHORT = 8u;

// ---------------------------------------------------------------------------------------------
// Alg. 2: FROGSearch for one query.  trace (optional) receives, per expansion, the record
// [u, |EN(u)|, EN(u)...]; stats = {expansions, ENC rows read, ENs admitted, distances}.
// ---------------------------------------------------------------------------------------------
void search_one(const Index& ix, const float* v_q, int32_t lo, int32_t hi, int k, int ef_s,
                const Params& P, int32_t* out_ids, float* out_dists, uint32_t* status,
                uint32_t* stats, std::vector<uint32_t>* trace, int64_t trace_cap) {
    uint32_t st = 0;
    bool trace_ok = true;   // records are appended until the first one that does not fit
    uint32_t n_exp = 0, n_rows = 0, n_en = 0, n_dist = 0;
    for (int j = 0; j < k; ++j) { out_ids[j] = -1; out_dists[j] = std::numeric_limits<float>::infinity(); }

    int64_t l_q, r_q;
    rank_interval(ix.sorted_attr, ix.n, lo, hi, &l_q, &r_q);
    int64_t w = r_q - l_q + 1;
    std::vector<Cand> pool;
    if (lo > hi || w <= 0) {
        st |= ST_EMPTY;
    } else if (w <= ef_s || w <= P.exact_below) {
        // every valid object is evaluated and the pool keeps the ef_s nearest: the answer is exact
        // (Def. 2 over the contiguous rank slab of Sec. 4)
        st |= ST_EXACT;
        for (int64_t r = l_q; r <= r_q; ++r) {
            pool.push_back(Cand{dist2_canonical(v_q, ix.vectors + r * ix.d_pad, ix.d_pad), (uint32_t)r, 1});
            ++n_dist;
        }
        std::sort(pool.begin(), pool.end(), cand_less);
        if ((int)pool.size() > ef_s) pool.resize(ef_s);
    } else {
        int L_start, L_end;
        hotspot_localization(l_q, r_q, ix.H, ix.n, &L_start, &L_end);        // line 1
        if (P.no_hotspot) { L_start = 0; L_end = ix.H - 1; }
        std::set<uint32_t> visited;                                           // hashCheck state
        for (int j = 0; j < P.epn; ++j) {                                     // lines 2-4
            uint32_t ep = (uint32_t)entry_point(P.seed, l_q, r_q, j);
            if (visited.insert(ep).second) {
                pool.push_back(Cand{dist2_canonical(v_q, ix.vectors + (int64_t)ep * ix.d_pad, ix.d_pad), ep, 0});
                ++n_dist;
            }
        }
        std::sort(pool.begin(), pool.end(), cand_less);                       // line 5
        if ((int)pool.size() > ef_s) pool.resize(ef_s);
        std::vector<uint32_t> EN(P.B > 0 ? P.B : 1);
        std::vector<Cand> fresh;
        std::vector<uint32_t> fresh_ids;
        for (;;) {                                                            // line 7
            // line 17 (and line 6): first pool position whose flag is 0
            int i = 0;
            while (i < (int)pool.size() && pool[i].flag) ++i;
            if (i >= (int)pool.size() || i >= ef_s) break;
            if ((int)n_exp >= P.max_iters) { st |= ST_ITER_CAP; break; }
            uint32_t u = pool[i].id;                                          // line 8
            pool[i].flag = 1;                                                 // line 9
            int rows = 0;
            int cnt = P.eager_hash
                ? en_identification_eager(ix.enc + (int64_t)u * ix.H * ix.m, ix.m, l_q, r_q, L_start, L_end,
                                          P.B, P.warp, visited, EN.data(), fresh_ids, &rows)
                : en_identification(ix.enc + (int64_t)u * ix.H * ix.m, ix.m, l_q, r_q,
                                    L_start, L_end, P.B, P.warp, EN.data(), &rows);       // line 10
            ++n_exp; n_rows += rows; n_en += cnt;
            if (trace && trace_ok && (int64_t)trace->size() + 2 + std::max(64, P.B) > trace_cap - 1) trace_ok = false;   // room for a full record
            if (trace && trace_ok) {
                trace->push_back(u);
                trace->push_back((uint32_t)cnt);
                for (int j = 0; j < cnt; ++j) trace->push_back(EN[j]);
            }
            fresh.clear();                                                    // line 11
            for (int j = 0; j < (P.eager_hash ? (int)fresh_ids.size() : cnt); ++j) {   // line 12
                uint32_t v = P.eager_hash ? fresh_ids[j] : EN[j];
                if (P.eager_hash || visited.insert(v).second) {               // line 13
                    fresh.push_back(Cand{dist2_canonical(v_q, ix.vectors + (int64_t)v * ix.d_pad, ix.d_pad), v, 0});
                    ++n_dist;                                                 // line 14
                }
            }
            std::sort(fresh.begin(), fresh.end(), cand_less);                 // line 15
            std::vector<Cand> merged(pool.size() + fresh.size());             // line 16
            std::merge(pool.begin(), pool.end(), fresh.begin(), fresh.end(), merged.begin(), cand_less);
            if ((int)merged.size() > ef_s) merged.resize(ef_s);
            pool.swap(merged);
        }
    }
    int got = std::min<int>(k, (int)pool.size());                            // line 18
    for (int j = 0; j < got; ++j) {
        out_ids[j] = ix.rank2id[pool[j].id];
        out_dists[j] = sqrtf(pool[j].dist2);
    }
    if (got < k) st |= ST_SHORT;
    if (status) *status = st;
    if (stats) { stats[0] = n_exp; stats[1] = n_rows; stats[2] = n_en; stats[3] = n_dist; }
}

}  // namespace

extern "C" {

void frog_oracle_rank_interval(const int32_t* sorted_attr, int64_t n, int32_t lo, int32_t hi,
                               int64_t* l_q, int64_t* r_q) {
    rank_interval(sorted_attr, n, lo, hi, l_q, r_q);
}

void frog_oracle_segment_at(int64_t N, int h, int64_t x, int64_t* L, int64_t* R) {
    segment_at(N, h, x, L, R);
}

void frog_oracle_hotspot(int64_t l_q, int64_t r_q, int H, int64_t N, int* L_start, int* L_end) {
    hotspot_localization(l_q, r_q, H, N, L_start, L_end);
}

int frog_oracle_en_identification(const uint32_t* enc_u, int m, int64_t l_q, int64_t r_q,
                                  int L_start, int L_end, int B, int warp, uint32_t* EN, int* rows_read) {
    return en_identification(enc_u, m, l_q, r_q, L_start, L_end, B, warp, EN, rows_read);
}

float frog_oracle_dist2(const float* q, const float* x, int d) { return dist2_canonical(q, x, d); }

int64_t frog_oracle_entry_point(uint64_t seed, int64_t l_q, int64_t r_q, int j) {
    return entry_point(seed, l_q, r_q, j);
}

// (O) batched search over an index given as raw arrays (vectors in rank order, rows of d_pad
// floats).  trace_out (optional): nq x trace_cap uint32, row q = [len, records...].
// Parallel over queries only.  Returns the number of threads used.
int frog_oracle_search(const int32_t* sorted_attr, const int32_t* rank2id, const float* vectors,
                       const uint32_t* enc, int64_t n, int d_pad, int H, int m,
                       const float* queries, const int32_t* lo, const int32_t* hi, int64_t nq,
                       int k, int ef_s, int epn, int B, int max_iters, uint64_t seed, int warp,
                       int no_hotspot, int exact_below, int eager_hash,
                       int32_t* out_ids, float* out_dists, uint32_t* status, uint32_t* stats,
                       uint32_t* trace_out, int64_t trace_cap, int threads) {
    Index ix{sorted_attr, rank2id, vectors, enc, n, d_pad, H, m};
    Params P{epn, B, max_iters, seed, warp, no_hotspot, exact_below, eager_hash};
    int used = 1;
#ifdef _OPENMP
    omp_set_num_threads(threads > 0 ? threads : omp_get_num_procs());   // <= 0: all cores
    used = omp_get_max_threads();
#endif
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t q = 0; q < nq; ++q) {
        std::vector<uint32_t> tr;
        search_one(ix, queries + q * d_pad, lo[q], hi[q], k, ef_s, P,
                   out_ids + q * k, out_dists + q * k,
                   status ? status + q : nullptr, stats ? stats + 4 * q : nullptr,
                   trace_out ? &tr : nullptr, trace_cap);
        if (trace_out) {
            uint32_t* row = trace_out + q * trace_cap;
            int64_t len = std::min<int64_t>((int64_t)tr.size(), trace_cap - 1);
            row[0] = (uint32_t)len;
            std::memcpy(row + 1, tr.data(), (size_t)len * sizeof(uint32_t));
        }
    }
    return used;
}

// (G) exact filtered kNN by the definition: scan ALL objects, test the attribute, rank by
// (distance, original id).  vectors/attrs are in original object order (row i = object i).
// mode 0: distances in double (the definition); mode 1: the fp32 fixed-order distance.
// out_dists holds the (non-squared) distance as float.
int frog_oracle_exact_scan(const float* vectors, const int32_t* attrs, int64_t n, int d,
                           const float* queries, const int32_t* lo, const int32_t* hi, int64_t nq,
                           int k, int mode, int32_t* out_ids, float* out_dists, int threads) {
    int used = 1;
#ifdef _OPENMP
    omp_set_num_threads(threads > 0 ? threads : omp_get_num_procs());   // <= 0: all cores
    used = omp_get_max_threads();
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t q = 0; q < nq; ++q) {
        std::vector<std::pair<double, int64_t>> best;   // (squared distance, id)
        const float* v_q = queries + q * d;
        for (int64_t i = 0; i < n; ++i) {
            if (attrs[i] < lo[q] || attrs[i] > hi[q]) continue;
            double dd = mode == 0 ? dist2_f64(v_q, vectors + i * d, d)
                                  : (double)dist2_canonical(v_q, vectors + i * d, d);
            best.emplace_back(dd, i);
        }
        std::sort(best.begin(), best.end());
        for (int j = 0; j < k; ++j) {
            if (j < (int)best.size()) {
                out_ids[q * k + j] = (int32_t)best[j].second;
                out_dists[q * k + j] = mode == 0 ? (float)std::sqrt(best[j].first) : sqrtf((float)best[j].first);
            } else {
                out_ids[q * k + j] = -1;
                out_dists[q * k + j] = std::numeric_limits<float>::infinity();
            }
        }
    }
    return used;
}

// (G) the same answer through the index: the valid objects are the contiguous rank slab
// [l_q, r_q] of the rank-ordered vector table.  Ties by original id, as above.
int frog_oracle_exact_slab(const int32_t* sorted_attr, const int32_t* rank2id, const float* vectors,
                           int64_t n, int d_pad,
                           const float* queries, const int32_t* lo, const int32_t* hi, int64_t nq,
                           int k, int mode, int32_t* out_ids, float* out_dists, int threads) {
    int used = 1;
#ifdef _OPENMP
    omp_set_num_threads(threads > 0 ? threads : omp_get_num_procs());   // <= 0: all cores
    used = omp_get_max_threads();
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t q = 0; q < nq; ++q) {
        int64_t l_q, r_q;
        rank_interval(sorted_attr, n, lo[q], hi[q], &l_q, &r_q);
        std::vector<std::pair<double, int64_t>> best;
        const float* v_q = queries + q * d_pad;
        if (lo[q] <= hi[q])
            for (int64_t r = l_q; r <= r_q; ++r) {
                double dd = mode == 0 ? dist2_f64(v_q, vectors + r * d_pad, d_pad)
                                      : (double)dist2_canonical(v_q, vectors + r * d_pad, d_pad);
                best.emplace_back(dd, (int64_t)rank2id[r]);
            }
        size_t keep = std::min<size_t>(best.size(), (size_t)k);
        std::partial_sort(best.begin(), best.begin() + keep, best.end());
        for (int j = 0; j < k; ++j) {
            if (j < (int)keep) {
                out_ids[q * k + j] = (int32_t)best[j].second;
                out_dists[q * k + j] = mode == 0 ? (float)std::sqrt(best[j].first) : sqrtf((float)best[j].first);
            } else {
                out_ids[q * k + j] = -1;
                out_dists[q * k + j] = std::numeric_limits<float>::infinity();
            }
        }
    }
    return used;
}

int frog_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // extern "C"
