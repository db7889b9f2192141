// FROG index builder (host, multi-threaded over objects).  Produces the index file read by the
// search library.  Structure per the paper: Sec. 4 (rank domain, implicit segment tree, dense
// n x H x m ENC array), Sec. 5.2 (fusion distance, Eq. 3), Sec. 6.1 (bottom-up construction:
// brute-force leaves, then per layer the own-child neighbours plus a greedy search, Alg. 1, in
// the sibling's temporary vector-distance graph), Sec. 6.2.2 (patience early termination).
// The CUDA builder (frog_build_gpu.cu) follows the same sentences and writes the same file, bit
// for bit; this program is its CPU counterpart and the two are compared element by element.
// Choices where the paper is silent, and two additions:
//   * ranks by (attribute, object id); H = max(1, ceil(log2 n) + 1 - n_inv);
//   * vector distance: squared L2 in fp32, rows cut into 4-float groups, group g to partial sum
//     g mod 8, fused multiply-adds in increasing index, partial sums combined pairwise at distance
//     4, 2, 1 (the order of the search path).  The distance BETWEEN TWO CANDIDATES used by the RNG
//     rule is that distance taken over column chunks of 128 floats and summed chunk by chunk (for
//     d <= 128 it is the same number);
//   * delta_a = |rank_i - rank_j| / (n - 1); delta_f evaluated in double from sqrt of the fp32
//     squared distance (delta_a^gamma is sqrt(delta_a) for the default gamma = 0.5, pow otherwise);
//     orders are (delta_v, rank) and (delta_f, rank); ENC rows stored in ascending delta_f,
//     empty entries at the tail;
//   * every object works on at most 64 candidates per layer.  Leaf layer: the 64 nearest other
//     objects of its leaf (all of them when the leaf has no more than 65).  Inner layers: the m
//     nearest it already has in its own child segment plus the m best of a greedy search (Alg. 1:
//     pool width ef_c, entry point = middle rank of the sibling, patience rule of Sec. 6.2.2 with
//     "improvement" = a new candidate enters the m best, at most 4 ef_c expansions) in the
//     sibling's temporary graph;
//   * RNG prune (rule not spelled out in the paper): visit candidates in ascending order, keep c
//     iff it is closer to u than to every neighbour kept so far, stop at m, back-fill with the
//     first rejected ones;
//   * ADDITION 1, reverse edges (switch FROG_BUILD_NO_REVERSE_EDGES turns it off): a forward graph
//     row is RNG-selected from the candidates, and the sources of an object's incoming forward
//     edges join its candidates (the 64 nearest of the union are kept).  Without them hubs absorb
//     the edges, about a third of the objects get no incoming edge at the upper layers, the
//     construction searches of the next layer cannot find them, and search recall saturates near
//     0.75 on clustered data;
//   * ADDITION 2, ENC selection (switch FROG_BUILD_ENC_FUSION_NEAREST turns it off): the m ENCs
//     are chosen by the same RNG rule applied in ascending FUSION distance; the paper keeps the m
//     fusion-nearest, which gives a k-NN-like graph that navigates poorly on low-intrinsic-
//     dimension mixtures.  With both switches set the builder is the paper's Sec. 6.1 as written;
//   * the parent graph is written to a second buffer and swapped (the paper overwrites in place);
//     the result does not depend on the thread count.
#include "frog_build.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <memory>
#include <new>
#include <numeric>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

constexpr uint32_t BOT = 0xFFFFFFFFu;

constexpr int CAND = 64;          // candidates an object works on per layer
constexpr int PAIR_CHUNK = 128;   // floats per column chunk of the candidate-to-candidate distance

// squared L2 over d floats (d a multiple of 4): 8 partial sums over 4-float groups, fused
// multiply-adds in increasing index, combined pairwise at distance 4, 2, 1
inline float sqdist(const float* a, const float* b, int d) {
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    const int groups = d >> 2;
    for (int g = 0; g < groups; ++g) {
        float s = acc[g & 7];
        for (int e = 0; e < 4; ++e) {
            const float t = a[4 * g + e] - b[4 * g + e];
            s = fmaf(t, t, s);
        }
        acc[g & 7] = s;
    }
    for (int off = 4; off >= 1; off >>= 1) {
        float nxt[8];
        for (int t = 0; t < 8; ++t) nxt[t] = acc[t] + acc[t ^ off];
        for (int t = 0; t < 8; ++t) acc[t] = nxt[t];
    }
    return acc[0];
}

// distance between two candidates (RNG rule): the same, chunk by chunk
inline float pair_sqdist(const float* a, const float* b, int d) {
    float s = 0.f;
    for (int c0 = 0; c0 < d; c0 += PAIR_CHUNK) s += sqdist(a + c0, b + c0, std::min(PAIR_CHUNK, d - c0));
    return s;
}

int ceil_log2(int64_t n) {
    int b = 0;
    while (((int64_t)1 << b) < n) ++b;
    return b;
}

struct Nb {
    float d2;
    uint32_t id;
};
inline bool nb_less(const Nb& a, const Nb& b) { return a.d2 != b.d2 ? a.d2 < b.d2 : a.id < b.id; }

struct Fz {
    double f;
    uint32_t id;
};
inline bool fz_less(const Fz& a, const Fz& b) { return a.f != b.f ? a.f < b.f : a.id < b.id; }

// left ends of the layer-h segments (split rule mid = L + (R-L)/2; left [L,mid], right [mid+1,R]);
// empty segments (possible only when a segment of one object is split) are dropped.
std::vector<int64_t> layer_starts(int64_t n, int h) {
    std::vector<std::pair<int64_t, int64_t>> cur{{0, n - 1}};
    for (int depth = 0; depth < h; ++depth) {
        std::vector<std::pair<int64_t, int64_t>> nxt;
        nxt.reserve(cur.size() * 2);
        for (auto [L, R] : cur) {
            int64_t mid = L + (R - L) / 2;
            nxt.emplace_back(L, mid);
            if (mid + 1 <= R) nxt.emplace_back(mid + 1, R);
        }
        cur.swap(nxt);
    }
    std::vector<int64_t> s;
    s.reserve(cur.size() + 1);
    for (auto& p : cur) s.push_back(p.first);
    s.push_back(n);
    return s;
}

struct Searcher {
    // greedy search of Alg. 1 over the temporary graph restricted to one segment
    std::vector<uint32_t> stamp;
    uint32_t epoch = 0;
    std::vector<Nb> pool;
    std::vector<uint8_t> flag;

    void init(int64_t n, int ef_c) {
        stamp.assign((size_t)n, 0);
        pool.reserve(ef_c + 1);
        flag.reserve(ef_c + 1);
    }

    void run(const float* V, int d, const uint32_t* pg, int m, const float* q, uint32_t ep,
             int ef_c, int patience, int top) {
        if (++epoch == 0) { std::fill(stamp.begin(), stamp.end(), 0); epoch = 1; }
        pool.clear();
        flag.clear();
        stamp[ep] = epoch;
        pool.push_back(Nb{sqdist(q, V + (int64_t)ep * d, d), ep});
        flag.push_back(0);
        int pat = patience;
        for (int it = 0; it < 4 * ef_c; ++it) {
            size_t i = 0;
            while (i < pool.size() && flag[i]) ++i;
            if (i >= pool.size()) break;
            flag[i] = 1;
            uint32_t u = pool[i].id;
            const uint32_t* nb = pg + (int64_t)u * m;
            bool improved = false;
            for (int j = 0; j < m; ++j) {
                uint32_t v = nb[j];
                if (v == BOT) continue;
                if (stamp[v] == epoch) continue;
                stamp[v] = epoch;
                Nb c{sqdist(q, V + (int64_t)v * d, d), v};
                if ((int)pool.size() >= ef_c && !nb_less(c, pool.back())) continue;
                size_t pos = std::lower_bound(pool.begin(), pool.end(), c, nb_less) - pool.begin();
                pool.insert(pool.begin() + pos, c);
                flag.insert(flag.begin() + pos, 0);
                if ((int)pool.size() > ef_c) { pool.pop_back(); flag.pop_back(); }
                if ((int)pos < top) improved = true;
            }
            if (improved) pat = patience;
            else if (--pat <= 0) break;
        }
    }
};

// RNG-style selection: visit candidates in the given (ascending) order, keep c iff it is closer to
// the source than to every neighbour kept so far; stop at m; back-fill with the first rejected.
void rng_select(const float* V, int d, const Nb* cand, int nc, int m, std::vector<Nb>& kept,
                std::vector<Nb>& pruned) {
    kept.clear();
    pruned.clear();
    for (int ci = 0; ci < nc; ++ci) {
        const Nb& c = cand[ci];
        bool ok = (int)kept.size() < m;
        if (ok)
            for (const Nb& p : kept)
                if (!(c.d2 < pair_sqdist(V + (int64_t)c.id * d, V + (int64_t)p.id * d, d))) {
                    ok = false;
                    break;
                }
        if (ok) kept.push_back(c); else pruned.push_back(c);
    }
    for (size_t j = 0; j < pruned.size() && (int)kept.size() < m; ++j) kept.push_back(pruned[j]);
}

struct FzNb {
    double f;
    Nb nb;
};
inline bool fznb_less(const FzNb& a, const FzNb& b) { return a.f != b.f ? a.f < b.f : a.nb.id < b.nb.id; }

// ENC row: candidates visited in ascending fusion distance (Eq. 3); c is kept iff it is closer
// (vector distance) to the source than to every ENC kept so far; back-fill in fusion order up to
// m; the row is stored in ascending fusion distance, empty entries at the tail.  With
// `fusion_nearest` the row is simply the m fusion-nearest candidates (the paper's rule).
void select_encs(const float* V, int d, const std::vector<FzNb>& byf, int m, bool fusion_nearest, uint32_t* erow) {
    std::vector<const FzNb*> kept, pruned;
    for (const FzNb& c : byf) {
        bool ok = (int)kept.size() < m;
        if (ok && !fusion_nearest)
            for (const FzNb* p : kept)
                if (!(c.nb.d2 < pair_sqdist(V + (int64_t)c.nb.id * d, V + (int64_t)p->nb.id * d, d))) {
                    ok = false;
                    break;
                }
        if (ok) kept.push_back(&c); else pruned.push_back(&c);
    }
    for (size_t j = 0; j < pruned.size() && (int)kept.size() < m; ++j) kept.push_back(pruned[j]);
    std::sort(kept.begin(), kept.end(), [](const FzNb* a, const FzNb* b) { return fznb_less(*a, *b); });
    for (int j = 0; j < m; ++j) erow[j] = j < (int)kept.size() ? kept[j]->nb.id : BOT;
}

bool write_all(FILE* f, const void* p, size_t bytes) {
    const char* c = (const char*)p;
    while (bytes) {
        size_t chunk = std::min<size_t>(bytes, (size_t)1 << 30);
        if (fwrite(c, 1, chunk, f) != chunk) return false;
        c += chunk;
        bytes -= chunk;
    }
    return true;
}

bool pad_to(FILE* f, uint64_t& pos, uint64_t target) {
    static const char zeros[128] = {0};
    while (pos < target) {
        size_t c = (size_t)std::min<uint64_t>(target - pos, sizeof(zeros));
        if (fwrite(zeros, 1, c, f) != c) return false;
        pos += c;
    }
    return true;
}

inline uint64_t align128(uint64_t x) { return (x + 127) & ~(uint64_t)127; }

}  // namespace

extern "C" double frog_fusion_distance(double delta_v, double delta_a, double beta, double gamma) {
    return delta_v * (1.0 - beta * (1.0 - std::pow(delta_a, gamma)));
}

extern "C" int32_t frog_retained_depth(int64_t n, int32_t n_inv) {
    int H = ceil_log2(n) + 1 - n_inv;
    return H < 1 ? 1 : H;
}

extern "C" int frog_index_build(const float* vectors, const int32_t* attrs, int64_t n, int32_t d,
                                const frog_build_params_t* params, const char* path) {
    if (!vectors || !attrs || !path || n < 1 || d < 1 || n >= ((int64_t)1 << 31) - 1) return 1;
    frog_build_params_t P{};
    if (params) P = *params;
    if (P.m == 0) P.m = d <= 300 ? 16 : 32;
    if (P.ef_c == 0) P.ef_c = d <= 300 ? 128 : 256;
    if (P.n_inv < 0) P.n_inv = d <= 300 ? 7 : 6;
    if (P.patience == 0) P.patience = 30;
    if (P.beta < 0) P.beta = 0.2f;
    if (P.gamma <= 0) P.gamma = 0.5f;
    if (P.m < 1 || P.m > 32 || P.ef_c < P.m || P.patience < 1) return 1;
    const int m = P.m;
    const int H = frog_retained_depth(n, P.n_inv);
    const int d_pad = (d + 3) / 4 * 4;
#ifdef _OPENMP
    if (P.threads > 0) omp_set_num_threads(P.threads);
    const int nthreads = omp_get_max_threads();
#else
    const int nthreads = 1;
#endif

    try {
        // ---- Sec. 4: rank domain -----------------------------------------------------------
        std::vector<int32_t> rank2id((size_t)n);
        std::iota(rank2id.begin(), rank2id.end(), 0);
        std::stable_sort(rank2id.begin(), rank2id.end(),
                         [&](int32_t a, int32_t b) { return attrs[a] < attrs[b]; });
        std::vector<int32_t> sorted_attr((size_t)n);
        std::unique_ptr<float[]> Vp(new float[(size_t)n * d_pad]);
        float* V = Vp.get();
#pragma omp parallel for schedule(static)
        for (int64_t r = 0; r < n; ++r) {
            sorted_attr[r] = attrs[rank2id[r]];
            const float* src = vectors + (int64_t)rank2id[r] * d;
            float* dst = V + r * d_pad;
            std::memcpy(dst, src, sizeof(float) * d);
            for (int j = d; j < d_pad; ++j) dst[j] = 0.f;
        }

        std::unique_ptr<uint32_t[]> encp(new uint32_t[(size_t)n * H * m]);
        uint32_t* enc = encp.get();
        std::unique_ptr<uint32_t[]> pgA(new uint32_t[(size_t)n * m]), pgB(new uint32_t[(size_t)n * m]);
        std::unique_ptr<float[]> pdA(new float[(size_t)n * m]), pdB(new float[(size_t)n * m]);
        // per-vertex nearest lists (unpruned, ascending by vector distance) of the current layer
        std::unique_ptr<uint32_t[]> annA(new uint32_t[(size_t)n * m]), annB(new uint32_t[(size_t)n * m]);
        uint32_t* ann_cur = annA.get();
        uint32_t* ann_nxt = annB.get();
        uint32_t* pg_cur = pgA.get();
        uint32_t* pg_nxt = pgB.get();
        float* pd_cur = pdA.get();
        float* pd_nxt = pdB.get();
        const double beta = P.beta, gamma = P.gamma;
        const double inv_span = n > 1 ? 1.0 / (double)(n - 1) : 0.0;
        auto fusion = [&](float d2, int64_t ru, int64_t rv) {
            const double da = (double)(ru > rv ? ru - rv : rv - ru) * inv_span;
            const double dv = std::sqrt((double)d2);
            const double za = gamma == 0.5 ? std::sqrt(da) : std::pow(da, gamma);   // both exact for 0.5
            return dv * (1.0 - beta * (1.0 - za));
        };

        // ---- layers H-1 .. 0 ----------------------------------------------------------------
        // Per layer: (1) every object collects its candidates in ascending (delta_v, rank) -- leaf
        // layer: the nearest CAND other objects of its leaf; inner layers: the m nearest it already
        // has in its own child segment plus the m found by a greedy search (Alg. 1) in the sibling's
        // temporary graph; (2) a forward graph row is RNG-selected from them; (3) each object adds
        // the sources of its incoming forward edges to its candidates (nearest CAND of the union)
        // and derives from this pool its nearest list, the parent's temporary graph row, and the
        // layer's ENCs.
        std::vector<Searcher> searchers(nthreads);
        if (H > 1)
            for (auto& s : searchers) s.init(n, P.ef_c);
        std::unique_ptr<Nb[]> c1p(new Nb[(size_t)n * CAND]);
        std::unique_ptr<uint32_t[]> pgF(new uint32_t[(size_t)n * m]);
        Nb* c1 = c1p.get();
        uint32_t* pg_fwd = pgF.get();
        const bool reverse_edges = !(P.reserved & FROG_BUILD_NO_REVERSE_EDGES);
        const bool fusion_nearest = (P.reserved & FROG_BUILD_ENC_FUSION_NEAREST) != 0;
        for (int h = H - 1; h >= 0; --h) {
            std::vector<int64_t> starts = layer_starts(n, h);
            // (1) + (2)
#pragma omp parallel
            {
#ifdef _OPENMP
                Searcher& S = searchers[omp_get_thread_num()];
#else
                Searcher& S = searchers[0];
#endif
                std::vector<Nb> cand, kept, pruned;
#pragma omp for schedule(dynamic, 64)
                for (int64_t u = 0; u < n; ++u) {
                    size_t s = std::upper_bound(starts.begin(), starts.end(), u) - starts.begin() - 1;
                    int64_t L = starts[s], R = starts[s + 1] - 1;
                    cand.clear();
                    if (h == H - 1) {
                        for (int64_t v = L; v <= R; ++v)
                            if (v != u) cand.push_back(Nb{sqdist(V + u * d_pad, V + v * d_pad, d_pad), (uint32_t)v});
                    } else {
                        int64_t mid = L + (R - L) / 2;
                        int64_t sL, sR;   // sibling child segment
                        if (u <= mid) { sL = mid + 1; sR = R; } else { sL = L; sR = mid; }
                        for (int j = 0; j < m; ++j)
                            if (ann_cur[u * m + j] != BOT) cand.push_back(Nb{pd_cur[u * m + j], ann_cur[u * m + j]});
                        if (sL <= sR) {
                            uint32_t ep = (uint32_t)(sL + (sR - sL) / 2);
                            S.run(V, d_pad, pg_cur, m, V + u * d_pad, ep, P.ef_c, P.patience, m);
                            size_t take = std::min<size_t>(m, S.pool.size());
                            for (size_t j = 0; j < take; ++j) cand.push_back(S.pool[j]);
                        }
                    }
                    std::sort(cand.begin(), cand.end(), nb_less);
                    if ((int)cand.size() > CAND) cand.resize(CAND);
                    for (int j = 0; j < CAND; ++j) c1[u * CAND + j] = j < (int)cand.size() ? cand[j] : Nb{0.f, BOT};
                    rng_select(V, d_pad, cand.data(), (int)cand.size(), m, kept, pruned);
                    for (int j = 0; j < m; ++j) pg_fwd[u * m + j] = j < (int)kept.size() ? kept[j].id : BOT;
                }
            }
            // reverse edges of the forward graph, grouped by target, sources ascending
            std::vector<uint32_t> rev_off((size_t)n + 1, 0), rev_src;
            if (reverse_edges) {
                for (int64_t e = 0; e < n * m; ++e)
                    if (pg_fwd[e] != BOT) ++rev_off[(size_t)pg_fwd[e] + 1];
                for (int64_t v = 0; v < n; ++v) rev_off[v + 1] += rev_off[v];
                rev_src.resize(rev_off[n]);
                std::vector<uint32_t> cur(rev_off.begin(), rev_off.end() - 1);
                for (int64_t u = 0; u < n; ++u)
                    for (int j = 0; j < m; ++j) {
                        uint32_t v = pg_fwd[u * m + j];
                        if (v != BOT) rev_src[cur[v]++] = (uint32_t)u;
                    }
            }
            // (3) final lists from candidates + reverse sources
#pragma omp parallel
            {
                std::vector<Nb> pool, kept, pruned;
                std::vector<FzNb> byf;
#pragma omp for schedule(dynamic, 64)
                for (int64_t u = 0; u < n; ++u) {
                    const Nb* cand = c1 + u * CAND;
                    pool.clear();
                    for (int j = 0; j < CAND && cand[j].id != BOT; ++j) pool.push_back(cand[j]);
                    const size_t base = pool.size();
                    for (uint32_t e = rev_off[u]; e < rev_off[u + 1]; ++e) {
                        uint32_t v = rev_src[e];
                        bool known = false;
                        for (size_t j = 0; j < base; ++j)
                            if (pool[j].id == v) { known = true; break; }
                        if (!known) pool.push_back(Nb{sqdist(V + u * d_pad, V + (int64_t)v * d_pad, d_pad), v});
                    }
                    std::sort(pool.begin(), pool.end(), nb_less);
                    if ((int)pool.size() > CAND) pool.resize(CAND);
                    const int np = (int)pool.size();
                    for (int j = 0; j < m; ++j) {
                        ann_nxt[u * m + j] = j < np ? pool[j].id : BOT;
                        pd_nxt[u * m + j] = j < np ? pool[j].d2 : 0.f;
                    }
                    rng_select(V, d_pad, pool.data(), np, m, kept, pruned);
                    for (int j = 0; j < m; ++j) pg_nxt[u * m + j] = j < (int)kept.size() ? kept[j].id : BOT;
                    // ENCs of this layer: the same selection with the pool in fusion-distance order
                    byf.clear();
                    for (int ci = 0; ci < np; ++ci) byf.push_back(FzNb{fusion(pool[ci].d2, u, pool[ci].id), pool[ci]});
                    std::sort(byf.begin(), byf.end(), fznb_less);
                    select_encs(V, d_pad, byf, m, fusion_nearest, enc + ((int64_t)u * H + h) * m);
                }
            }
            std::swap(pg_cur, pg_nxt);
            std::swap(ann_cur, ann_nxt);
            std::swap(pd_cur, pd_nxt);
        }

        // ---- write the file ------------------------------------------------------------------
        unsigned char hdr[256];
        std::memset(hdr, 0, sizeof(hdr));
        std::memcpy(hdr, "FROGIDX1", 8);
        uint32_t u32s[8] = {1u, (uint32_t)d, (uint32_t)d_pad, (uint32_t)H, (uint32_t)m,
                            (uint32_t)P.n_inv, (uint32_t)P.ef_c, (uint32_t)P.patience};
        std::memcpy(hdr + 8, u32s, sizeof(u32s));
        std::memcpy(hdr + 40, &P.beta, 4);
        std::memcpy(hdr + 44, &P.gamma, 4);
        uint64_t n64 = (uint64_t)n;
        std::memcpy(hdr + 48, &n64, 8);
        std::memcpy(hdr + 56, &P.seed, 8);
        uint32_t bot = BOT;
        std::memcpy(hdr + 64, &bot, 4);
        uint32_t flags = (uint32_t)P.reserved & (FROG_BUILD_NO_REVERSE_EDGES | FROG_BUILD_ENC_FUSION_NEAREST);
        std::memcpy(hdr + 68, &flags, 4);
        uint64_t off_attr = 256;
        uint64_t off_r2i = align128(off_attr + (uint64_t)n * 4);
        uint64_t off_vec = align128(off_r2i + (uint64_t)n * 4);
        uint64_t off_enc = align128(off_vec + (uint64_t)n * d_pad * 4);
        uint64_t total = off_enc + (uint64_t)n * H * m * 4;
        uint64_t offs[5] = {off_attr, off_r2i, off_vec, off_enc, total};
        std::memcpy(hdr + 72, offs, sizeof(offs));
        FILE* f = fopen(path, "wb");
        if (!f) return 2;
        uint64_t pos = 0;
        bool ok = write_all(f, hdr, 256);
        pos = 256;
        ok = ok && write_all(f, sorted_attr.data(), (size_t)n * 4);
        pos += (uint64_t)n * 4;
        ok = ok && pad_to(f, pos, off_r2i) && write_all(f, rank2id.data(), (size_t)n * 4);
        pos += (uint64_t)n * 4;
        ok = ok && pad_to(f, pos, off_vec) && write_all(f, V, (size_t)n * d_pad * 4);
        pos += (uint64_t)n * d_pad * 4;
        ok = ok && pad_to(f, pos, off_enc) && write_all(f, enc, (size_t)n * H * m * 4);
        if (fclose(f) != 0) ok = false;
        return ok ? 0 : 2;
    } catch (const std::bad_alloc&) {
        return 4;
    }
}
