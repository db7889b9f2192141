// FROG index builder (host, multi-threaded over objects).  Produces the index file read by the
// search library.  Structure per the paper: Sec. 4 (rank domain, implicit segment tree, dense
// n x H x m ENC array), Sec. 5.2 (fusion distance, Eq. 3), Sec. 6.1 (bottom-up construction:
// brute-force leaves, then per layer the own-child neighbours plus a greedy search, Alg. 1, in
// the sibling's temporary vector-distance graph), Sec. 6.2.2 (patience early termination).
// Choices where the paper is silent, and two additions:
//   * ranks by (attribute, object id); H = max(1, ceil(log2 n) + 1 - n_inv);
//   * delta_a = |rank_i - rank_j| / (n - 1); delta_f evaluated in double from sqrt of the fp32
//     squared distance; ENC rows stored in ascending (delta_f, rank), empty entries at the tail;
//   * sibling search (Alg. 1): pool width ef_c, entry point = middle rank of the sibling, the m
//     best of the pool are taken;
//   * own-child neighbours: every object carries its m nearest (unpruned) of the current segment
//     upward, next to the pruned graph row used for navigation;
//   * RNG prune (rule not spelled out in the paper): visit candidates in ascending order, keep c
//     iff it is closer to u than to every neighbour kept so far, stop at m, back-fill with the
//     first rejected ones;
//   * ADDITION 1, reverse edges: the sources of an object's incoming forward edges join its
//     candidates.  Without them hubs absorb the edges, about a third of the objects get no
//     incoming edge at the upper layers, the construction searches of the next layer cannot find
//     them, and search recall saturates near 0.75 on clustered data;
//   * ADDITION 2, ENC selection: the m ENCs are chosen by the same RNG rule applied in ascending
//     FUSION distance (the paper keeps the m fusion-nearest); plain top-m gives a k-NN-like
//     graph that navigates poorly on low-intrinsic-dimension mixtures;
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

inline float sqdist(const float* a, const float* b, int d) {
    // eight independent partial sums: vectorisable without re-association
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int i = 0;
    for (; i + 8 <= d; i += 8)
        for (int j = 0; j < 8; ++j) {
            float t = a[i + j] - b[i + j];
            acc[j] += t * t;
        }
    for (; i < d; ++i) {
        float t = a[i] - b[i];
        acc[i & 7] += t * t;
    }
    return ((acc[0] + acc[4]) + (acc[2] + acc[6])) + ((acc[1] + acc[5]) + (acc[3] + acc[7]));
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
        for (;;) {
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
                if (!(c.d2 < sqdist(V + (int64_t)c.id * d, V + (int64_t)p.id * d, d))) {
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
// m; the row is stored in ascending fusion distance, empty entries at the tail.
void select_encs(const float* V, int d, const std::vector<FzNb>& byf, int m, uint32_t* erow) {
    std::vector<const FzNb*> kept, pruned;
    for (const FzNb& c : byf) {
        bool ok = (int)kept.size() < m;
        if (ok)
            for (const FzNb* p : kept)
                if (!(c.nb.d2 < sqdist(V + (int64_t)c.nb.id * d, V + (int64_t)p->nb.id * d, d))) {
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
    if (P.m < 1 || P.m > 64 || P.ef_c < P.m || P.patience < 1) return 1;
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
            double da = (double)(ru > rv ? ru - rv : rv - ru) * inv_span;
            return frog_fusion_distance(std::sqrt((double)d2), da, beta, gamma);
        };

        // ---- leaves (layer H-1): brute force inside each leaf ------------------------------
        {
            std::vector<int64_t> starts = layer_starts(n, H - 1);
#pragma omp parallel
            {
                std::vector<Nb> byv, kept, pruned;
                std::vector<FzNb> byf;
#pragma omp for schedule(dynamic, 64)
                for (int64_t u = 0; u < n; ++u) {
                    size_t s = std::upper_bound(starts.begin(), starts.end(), u) - starts.begin() - 1;
                    int64_t L = starts[s], R = starts[s + 1] - 1;
                    byv.clear();
                    byf.clear();
                    for (int64_t v = L; v <= R; ++v) {
                        if (v == u) continue;
                        byv.push_back(Nb{sqdist(V + u * d_pad, V + v * d_pad, d_pad), (uint32_t)v});
                    }
                    std::sort(byv.begin(), byv.end(), nb_less);
                    for (const Nb& c : byv) byf.push_back(FzNb{fusion(c.d2, u, c.id), c});
                    std::sort(byf.begin(), byf.end(), fznb_less);
                    rng_select(V, d_pad, byv.data(), (int)byv.size(), m, kept, pruned);
                    for (int j = 0; j < m; ++j) {
                        pg_cur[u * m + j] = j < (int)kept.size() ? kept[j].id : BOT;
                        ann_cur[u * m + j] = j < (int)byv.size() ? byv[j].id : BOT;
                        pd_cur[u * m + j] = j < (int)byv.size() ? byv[j].d2 : 0.f;
                    }
                    select_encs(V, d_pad, byf, m, enc + ((int64_t)u * H + (H - 1)) * m);
                }
            }
        }

        // ---- inductive step, layers H-2 .. 0 -----------------------------------------------
        // Per layer: (1) every object collects 2m vector-distance candidates -- the m nearest it
        // already has in its own child segment plus the m found by a greedy search (Alg. 1) in the
        // sibling's temporary graph; (2) a forward graph row is RNG-pruned from them; (3) each
        // object adds the sources of its incoming forward edges to its candidates (without them a
        // third of the objects end up with no incoming edge and can never be found again, neither
        // by the next layer's construction searches nor at query time) and derives from this pool
        // its nearest list, the parent's temporary graph row, and the layer's ENCs.
        std::vector<Searcher> searchers(nthreads);
        const int C = 2 * m;   // candidates per object
        std::unique_ptr<Nb[]> c1p;
        std::unique_ptr<uint32_t[]> pgF;
        if (H > 1) {
            for (auto& s : searchers) s.init(n, P.ef_c);
            c1p.reset(new Nb[(size_t)n * C]);
            pgF.reset(new uint32_t[(size_t)n * m]);
        }
        Nb* c1 = c1p.get();
        uint32_t* pg_fwd = pgF.get();
        for (int h = H - 2; h >= 0; --h) {
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
                    int64_t mid = L + (R - L) / 2;
                    int64_t sL, sR;   // sibling child segment
                    if (u <= mid) { sL = mid + 1; sR = R; } else { sL = L; sR = mid; }
                    cand.clear();
                    for (int j = 0; j < m; ++j)
                        if (ann_cur[u * m + j] != BOT) cand.push_back(Nb{pd_cur[u * m + j], ann_cur[u * m + j]});
                    if (sL <= sR) {
                        uint32_t ep = (uint32_t)(sL + (sR - sL) / 2);
                        S.run(V, d_pad, pg_cur, m, V + u * d_pad, ep, P.ef_c, P.patience, m);
                        size_t take = std::min<size_t>(m, S.pool.size());
                        for (size_t j = 0; j < take; ++j) cand.push_back(S.pool[j]);
                    }
                    std::sort(cand.begin(), cand.end(), nb_less);
                    for (int j = 0; j < C; ++j) c1[u * C + j] = j < (int)cand.size() ? cand[j] : Nb{0.f, BOT};
                    rng_select(V, d_pad, cand.data(), (int)cand.size(), m, kept, pruned);
                    for (int j = 0; j < m; ++j) pg_fwd[u * m + j] = j < (int)kept.size() ? kept[j].id : BOT;
                }
            }
            // reverse edges of the forward graph, grouped by target, sources ascending
            std::vector<uint32_t> rev_off((size_t)n + 1, 0), rev_src;
            for (int64_t e = 0; e < n * m; ++e)
                if (pg_fwd[e] != BOT) ++rev_off[(size_t)pg_fwd[e] + 1];
            for (int64_t v = 0; v < n; ++v) rev_off[v + 1] += rev_off[v];
            rev_src.resize(rev_off[n]);
            {
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
                    const Nb* cand = c1 + u * C;
                    pool.clear();
                    for (int j = 0; j < C && cand[j].id != BOT; ++j) pool.push_back(cand[j]);
                    const size_t base = pool.size();
                    for (uint32_t e = rev_off[u]; e < rev_off[u + 1]; ++e) {
                        uint32_t v = rev_src[e];
                        bool known = false;
                        for (size_t j = 0; j < base; ++j)
                            if (pool[j].id == v) { known = true; break; }
                        if (!known) pool.push_back(Nb{sqdist(V + u * d_pad, V + (int64_t)v * d_pad, d_pad), v});
                    }
                    std::sort(pool.begin(), pool.end(), nb_less);
                    if ((int)pool.size() > 2 * C) pool.resize(2 * C);
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
                    select_encs(V, d_pad, byf, m, enc + ((int64_t)u * H + h) * m);
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
