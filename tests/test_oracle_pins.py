"""Pins of the CPU oracle against things other than itself: hand traces, closed forms,
invariants, brute force on small inputs and special cases with exact arithmetic.  No GPU."""
import os

import numpy as np
import pytest

import datagen
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------------------------
# Sec. 4: attribute -> rank interval holds exactly the valid objects
# ---------------------------------------------------------------------------------------------
def test_rank_interval_matches_attribute_scan():
    rng = np.random.default_rng(11)
    for n, top in ((1, 3), (7, 4), (200, 50), (1000, 100000)):
        attrs = np.sort(rng.integers(-top, top, size=n).astype(np.int32))
        cases = [(int(rng.integers(-top - 5, top + 5)), int(rng.integers(-top - 5, top + 5))) for _ in range(200)]
        cases += [(-2**31, 2**31 - 1), (int(attrs[0]), int(attrs[0])), (int(attrs[-1]), int(attrs[-1])),
                  (top + 10, top + 20), (-top - 20, -top - 10), (5, 4)]
        for lo, hi in cases:
            l, r = oracle.rank_interval(attrs, lo, hi)
            valid = np.nonzero((attrs >= lo) & (attrs <= hi))[0]
            if lo > hi or valid.size == 0:
                assert r - l + 1 <= 0
            else:
                assert (l, r) == (int(valid[0]), int(valid[-1]))
                assert r - l + 1 == valid.size      # contiguous: nothing invalid inside


def test_exact_slab_equals_definition_scan(tiny):
    """(G) through the index == (G) by scanning every object and testing its attribute."""
    wl, _, ix = tiny
    ids_a, d_a = oracle.exact_scan(wl.vectors, wl.attrs, wl.queries, wl.lo, wl.hi, 10, mode=0)
    ids_b, d_b, _ = oracle.exact_slab(ix, wl.queries, wl.lo, wl.hi, 10, mode=0)
    assert np.array_equal(ids_a, ids_b)
    assert np.array_equal(d_a, d_b)


def test_exact_scan_against_numpy_bruteforce():
    """Def. 2 written out with numpy in float64 on a small instance, incl. duplicate attributes."""
    rng = np.random.default_rng(5)
    n, d, nq, k = 300, 12, 40, 7
    V = rng.standard_normal((n, d)).astype(np.float32)
    a = rng.integers(0, 40, size=n).astype(np.int32)
    Q = rng.standard_normal((nq, d)).astype(np.float32)
    lo = rng.integers(-2, 40, size=nq).astype(np.int32)
    hi = (lo + rng.integers(-1, 12, size=nq)).astype(np.int32)
    ids, dists = oracle.exact_scan(V, a, Q, lo, hi, k, mode=0)
    for q in range(nq):
        valid = np.nonzero((a >= lo[q]) & (a <= hi[q]))[0]
        dd = ((V[valid].astype(np.float64) - Q[q].astype(np.float64)) ** 2).sum(1)
        order = np.lexsort((valid, dd))[:k]
        exp = valid[order]
        assert np.array_equal(ids[q][: exp.size], exp)
        assert np.all(ids[q][exp.size:] == -1) and np.all(np.isinf(dists[q][exp.size:]))
        assert np.allclose(dists[q][: exp.size], np.sqrt(dd[order]), rtol=1e-6)


# ---------------------------------------------------------------------------------------------
# Sec. 4: implicit segment tree
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N", [1, 2, 3, 16, 17, 100, 1000, 12345])
def test_segments_partition_and_nest(N):
    H = max(1, int(np.ceil(np.log2(N))) + 1) if N > 1 else 1
    prev = None
    for h in range(H):
        segs = sorted({oracle.segment_at(N, h, x) for x in range(N)})
        # partition of [0, N-1]
        assert segs[0][0] == 0 and segs[-1][1] == N - 1
        for (a, b), (c, _) in zip(segs, segs[1:]):
            assert c == b + 1
        sizes = [b - a + 1 for a, b in segs]
        assert max(sizes) - min(sizes) <= 1
        if prev is not None:
            # every segment is one half of a parent, left half gets the extra element
            for L, R in prev:
                mid = L + (R - L) // 2
                kids = [s for s in segs if L <= s[0] and s[1] <= R]
                assert kids == ([(L, mid), (mid + 1, R)] if R > L else [(L, R)])
        prev = segs


# ---------------------------------------------------------------------------------------------
# Alg. 3 hotspot localization
# ---------------------------------------------------------------------------------------------
def test_hotspot_hand_traces():
    with open(os.path.join(GOLDEN, "hotspot_traces.txt")) as f:
        rows = [list(map(int, ln.split())) for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 13
    for N, H, l, r, ls, le in rows:
        assert oracle.hotspot(l, r, H, N) == (ls, le), (N, H, l, r)


def _layer_segments(N, h):
    segs = [(0, N - 1)]
    for _ in range(h):
        nxt = []
        for L, R in segs:
            mid = L + (R - L) // 2
            nxt.append((L, mid))
            if mid + 1 <= R:
                nxt.append((mid + 1, R))
        segs = nxt
    return segs


def _hotspot_by_enumeration(l, r, H, N):
    """Rules 1-2 of Sec. 7.2 from explicit segment lists: L_start = deepest layer with one segment
    holding the whole range; then Eq. 6 with the boundaries that fall inside the range."""
    ls = 0
    for h in range(H):
        if any(L <= l and r <= R for L, R in _layer_segments(N, h)):
            ls = h
        else:
            break
    le = ls
    for h in range(ls + 1, H):
        inside = [R for L, R in _layer_segments(N, h) if l <= R < r]   # boundary = last rank of its left segment
        assert inside, "a layer below L_start always cuts the range"
        lhs = (min(inside) - l) + (r - max(inside))
        if lhs * (2 ** h) >= (r - l):
            le = h
        else:
            break
    return ls, le


def test_hotspot_matches_enumeration_and_invariants():
    rng = np.random.default_rng(3)
    for N, H in ((16, 4), (16, 5), (37, 4), (1000, 6), (1000, 10), (4097, 8)):
        for _ in range(300):
            l = int(rng.integers(0, N))
            r = int(rng.integers(l, N))
            ls, le = oracle.hotspot(l, r, H, N)
            assert 0 <= ls <= le <= H - 1
            assert (ls, le) == _hotspot_by_enumeration(l, r, H, N)
            L, R = oracle.segment_at(N, ls, l)
            assert L <= l and r <= R                      # one segment holds both ends at L_start
            if ls + 1 < H:
                L2, R2 = oracle.segment_at(N, ls + 1, l)
                assert not (L2 <= l and r <= R2)          # ... and none does one layer deeper


# ---------------------------------------------------------------------------------------------
# Alg. 4 EN identification == "first B passing entries in stored order"
# ---------------------------------------------------------------------------------------------
def test_en_identification_is_order_preserving_prefix():
    rng = np.random.default_rng(9)
    for _ in range(400):
        H = int(rng.integers(1, 9))
        m = int(rng.choice([4, 16, 32]))
        enc = rng.integers(0, 200, size=(H, m)).astype(np.uint32)
        enc[rng.random((H, m)) < 0.15] = 0xFFFFFFFF
        l = int(rng.integers(0, 200))
        r = int(rng.integers(l, 200))
        ls = int(rng.integers(0, H))
        le = int(rng.integers(ls, H))
        B = int(rng.integers(1, 33)) if rng.random() < 0.5 else int(rng.integers(33, 200))   # up to and beyond the kernels' 128
        flat = enc[ls:le + 1].ravel()
        expect = [int(v) for v in flat if v != 0xFFFFFFFF and l <= v <= r][:B]
        got = None
        for warp in (16, 32, 64):
            en, rows = oracle.en_identification(enc, l, r, ls, le, B, warp=warp)
            assert list(map(int, en)) == expect            # independent of the chunk width
            got = en
            assert 0 <= rows <= le - ls + 1
        # rows read with 32-entry chunks: enough rows to reach the B-th pass, in whole chunks
        en, rows = oracle.en_identification(enc, l, r, ls, le, B, warp=32)
        passing = np.nonzero([(v != 0xFFFFFFFF and l <= v <= r) for v in flat])[0]
        last_needed = passing[B - 1] if passing.size >= B else flat.size - 1
        chunk_end = min(flat.size, (last_needed // 32 + 1) * 32)
        assert rows == -(-chunk_end // m)
        assert got is not None


# ---------------------------------------------------------------------------------------------
# distance
# ---------------------------------------------------------------------------------------------
def test_distance_exact_on_integer_vectors():
    """Integer components in [0,255], d=128: every partial sum < 2^24, so fp32 is exact in any
    order and must equal int64 arithmetic bit for bit."""
    rng = np.random.default_rng(2)
    for d in (4, 32, 96, 128, 132):
        for _ in range(200):
            x = rng.integers(0, 256, size=d)
            q = rng.integers(0, 256, size=d)
            exact = int(((x - q) ** 2).sum())
            assert oracle.dist2(q.astype(np.float32), x.astype(np.float32)) == float(exact)


def test_distance_close_to_float64_and_structure():
    rng = np.random.default_rng(4)
    for d in (4, 8, 36, 96, 128, 768):
        x = rng.standard_normal(d).astype(np.float32)
        q = rng.standard_normal(d).astype(np.float32)
        ref = float(((x.astype(np.float64) - q.astype(np.float64)) ** 2).sum())
        got = oracle.dist2(q, x)
        assert abs(got - ref) <= 1e-5 * ref
        assert oracle.dist2(x, q) == got            # (x-q)^2 == (q-x)^2 term by term
        assert oracle.dist2(x, x) == 0.0
    # each coordinate enters once: perturbing coordinate i changes the result
    x = np.zeros(40, np.float32)
    q = np.zeros(40, np.float32)
    for i in range(40):
        y = x.copy()
        y[i] = 3.0
        assert oracle.dist2(q, y) == 9.0


def test_distance_summation_order_is_the_stated_one():
    """Replay of the stated order with numpy float32 scalars: 8 partial sums over 4-float groups,
    products exact in float64 and rounded once (fused), butterfly 4-2-1."""
    rng = np.random.default_rng(8)
    for d in (32, 96, 128):
        x = (rng.standard_normal(d) * 3).astype(np.float32)
        q = (rng.standard_normal(d) * 3).astype(np.float32)
        acc = [np.float32(0)] * 8
        for g in range(d // 4):
            t = g % 8
            for e in range(4):
                diff = np.float32(x[4 * g + e] - q[4 * g + e])
                # fused multiply-add: exact product and sum, one rounding.  The product of two
                # fp32 values is exact in fp64; the fp64 sum is exact here up to double rounding,
                # which the assertion below tolerates at 1 ulp.
                acc[t] = np.float32(np.float64(diff) * np.float64(diff) + np.float64(acc[t]))
        for off in (4, 2, 1):
            acc = [np.float32(acc[t] + acc[t ^ off]) for t in range(8)]
        got = np.float32(oracle.dist2(q, x))
        assert abs(float(got) - float(acc[0])) <= float(np.spacing(acc[0]))


# ---------------------------------------------------------------------------------------------
# entry points (Alg. 2 line 3)
# ---------------------------------------------------------------------------------------------
def test_entry_points_in_range_uniform_and_stateless():
    l, r = 1000, 1999
    pts = np.array([oracle.entry_point(7, l, r, j) for j in range(20000)])
    assert pts.min() >= l and pts.max() <= r
    hist = np.bincount((pts - l) // 100, minlength=10)
    assert np.all(np.abs(hist - 2000) < 250)             # 10 equal bins, ~5.5 sigma
    assert oracle.entry_point(7, l, r, 3) == pts[3]      # function of (seed, range, j) only
    assert any(oracle.entry_point(8, l, r, j) != pts[j] for j in range(16))
    assert oracle.entry_point(1, 5, 5, 0) == 5


# ---------------------------------------------------------------------------------------------
# whole search (Alg. 2): invariants and exact special cases
# ---------------------------------------------------------------------------------------------
@pytest.fixture(scope="module")
def tiny_runs(tiny):
    wl, _, ix = tiny
    gt_ids, gt_d, _ = oracle.exact_slab(ix, wl.queries, wl.lo, wl.hi, wl.k, mode=1)
    runs = {ef: oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, ef, trace_cap=8192) for ef in (16, 64, 128)}
    return wl, ix, gt_ids, gt_d, runs


def test_search_results_respect_the_range_and_order(tiny_runs):
    wl, ix, _, _, runs = tiny_runs
    id2attr = wl.attrs
    for ef, res in runs.items():
        for q in range(wl.nq):
            ids = res.ids[q]
            got = ids[ids >= 0]
            assert np.all((id2attr[got] >= wl.lo[q]) & (id2attr[got] <= wl.hi[q]))
            assert len(set(got.tolist())) == got.size                 # no duplicates
            dd = res.dists[q][: got.size]
            assert np.all(np.diff(dd) >= 0)
            assert np.all(ids[got.size:] == -1) and np.all(np.isinf(res.dists[q][got.size:]))
            # reported distance is the true one
            true = np.sqrt(((wl.vectors[got].astype(np.float64) - wl.queries[q].astype(np.float64)) ** 2).sum(1))
            assert np.allclose(dd, true, rtol=1e-5)


def test_small_ranges_are_exact_and_padded(tiny_runs):
    wl, ix, gt_ids, gt_d, runs = tiny_runs
    seen_exact = 0
    for ef, res in runs.items():
        for q in range(wl.nq):
            l, r = oracle.rank_interval(ix.sorted_attr, int(wl.lo[q]), int(wl.hi[q]))
            w = r - l + 1
            if w <= ef:
                seen_exact += 1
                assert res.status[q] & oracle.ST_EXACT
                assert np.array_equal(res.ids[q], gt_ids[q])
                assert np.array_equal(res.dists[q], gt_d[q])
                if w < wl.k:
                    assert res.status[q] & oracle.ST_SHORT
                    assert np.all(res.ids[q][w:] == -1)
    assert seen_exact > 0


def test_exact_below_extends_the_exact_rule(tiny_runs):
    """With exact_below = T every range of at most max(ef_s, T) objects equals the definition
    scan (ids and distances), the others are searched as before."""
    wl, ix, gt_ids, gt_d, runs = tiny_runs
    ef, T = 16, 700
    res = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, ef, exact_below=T)
    base = runs[ef]
    n_ext = 0
    for q in range(wl.nq):
        l, r = oracle.rank_interval(ix.sorted_attr, int(wl.lo[q]), int(wl.hi[q]))
        w = r - l + 1
        if 0 < w <= T:
            n_ext += w > ef
            assert res.status[q] & oracle.ST_EXACT
            assert np.array_equal(res.ids[q], gt_ids[q]) and np.array_equal(res.dists[q], gt_d[q])
            assert res.stats[q, 3] == w and res.stats[q, 0] == 0
        else:
            assert np.array_equal(res.ids[q], base.ids[q]) and np.array_equal(res.stats[q], base.stats[q])
    assert n_ext > 10


def test_range_with_at_most_k_points_returns_exactly_those(tiny):
    wl, _, ix = tiny
    srt = np.asarray(ix.sorted_attr)
    lo = np.array([srt[10], srt[500], srt[9990], srt[0]], dtype=np.int32)
    hi = np.array([srt[12], srt[509], srt[9999], srt[0]], dtype=np.int32)
    Q = wl.queries[:4]
    res = oracle.search(ix, Q, lo, hi, 10, 32)
    for q, (a, b) in enumerate(((10, 12), (500, 509), (9990, 9999), (0, 0))):
        exp = set(np.asarray(ix.rank2id)[a:b + 1].tolist())
        got = res.ids[q][res.ids[q] >= 0]
        assert set(got.tolist()) == exp
    # empty and inverted ranges
    res = oracle.search(ix, Q[:2], np.array([5, -100], np.int32), np.array([4, -50], np.int32), 10, 32)
    assert np.all(res.ids == -1) and np.all(res.status & oracle.ST_EMPTY)


def test_full_range_reduces_to_unfiltered_search(tiny):
    """With [lo, hi] covering everything the range predicate never fires: the search must equal
    the same search with the hotspot/predicate machinery given the whole domain, and its answers
    must be good against unfiltered brute force."""
    wl, _, ix = tiny
    nq = 60
    lo = np.full(nq, -2**31, np.int32)
    hi = np.full(nq, 2**31 - 1, np.int32)
    res = oracle.search(ix, wl.queries[:nq], lo, hi, 10, 128)
    lo2 = np.full(nq, int(ix.sorted_attr[0]), np.int32)
    hi2 = np.full(nq, int(ix.sorted_attr[-1]), np.int32)
    res2 = oracle.search(ix, wl.queries[:nq], lo2, hi2, 10, 128)
    assert np.array_equal(res.ids, res2.ids)
    # unfiltered brute force in numpy
    V = wl.vectors.astype(np.float64)
    hits = 0
    for q in range(nq):
        dd = ((V - wl.queries[q].astype(np.float64)) ** 2).sum(1)
        hits += np.intersect1d(np.argsort(dd, kind="stable")[:10], res.ids[q]).size
    assert hits / (10 * nq) >= 0.85
    # every layer row scanned at L_start = 0 passes the predicate: the budget fills in one chunk
    assert np.all(res.stats[:, 2] == 16 * res.stats[:, 0])


def test_search_counters_and_trace_are_consistent(tiny_runs):
    wl, ix, _, _, runs = tiny_runs
    res = runs[64]
    for q in range(wl.nq):
        n_exp, n_rows, n_en, n_dist = map(int, res.stats[q])
        l, r = oracle.rank_interval(ix.sorted_attr, int(wl.lo[q]), int(wl.hi[q]))
        w = r - l + 1
        assert n_dist <= w                               # every vertex evaluated at most once
        if res.status[q] & (oracle.ST_EXACT | oracle.ST_EMPTY):
            assert n_exp == 0
            continue
        tr = res.trace[q]
        ln = int(tr[0])
        pos, exps, ens, seen_u = 1, 0, 0, set()
        while pos < 1 + ln:
            u, cnt = int(tr[pos]), int(tr[pos + 1])
            en = tr[pos + 2: pos + 2 + cnt]
            assert l <= u <= r and u not in seen_u       # a vertex is expanded once
            seen_u.add(u)
            assert cnt <= 16 and np.all((en >= l) & (en <= r))
            # EN(u) is what Alg. 4 yields for this vertex
            ls, le = oracle.hotspot(l, r, ix.H, ix.n)
            exp_en, _ = oracle.en_identification(np.asarray(ix.enc[u]), l, r, ls, le, 16)
            assert np.array_equal(en, exp_en)
            pos += 2 + cnt
            exps += 1
            ens += cnt
        assert (exps, ens) == (n_exp, n_en)
        assert n_rows <= n_exp * ix.H and n_dist <= 16 + n_en


def test_eager_hash_check_ablation(tiny_runs):
    """Eager form of the hash check (visited test inside the predicate of Alg. 4).  (a) When the
    budget never binds (B >= H*m) it evaluates the same vertices as the lazy form, so ids,
    distances, expansions and distance counts coincide with the pinned lazy search.  (b) With
    the default budget, replaying the trace: no EN entry was evaluated before its expansion,
    repeats occur only inside one EN list, and the distance count is the number of distinct ids."""
    wl, ix, _, _, runs = tiny_runs
    big = ix.H * ix.m
    lazy = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 64, B=big)
    eager = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 64, B=big, eager_hash=True)
    assert np.array_equal(lazy.ids, eager.ids) and np.array_equal(lazy.dists, eager.dists)
    assert np.array_equal(lazy.stats[:, [0, 3]], eager.stats[:, [0, 3]])
    assert eager.stats[:, 2].sum() < lazy.stats[:, 2].sum()          # fewer admitted slots

    res = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 64, eager_hash=True, trace_cap=8192)
    searched = 0
    for q in range(wl.nq):
        if res.status[q] & (oracle.ST_EXACT | oracle.ST_EMPTY):
            continue
        searched += 1
        l, r = oracle.rank_interval(ix.sorted_attr, int(wl.lo[q]), int(wl.hi[q]))
        seen = {oracle.entry_point(0, l, r, j) for j in range(16)}
        tr = res.trace[q]
        pos, ln, n_en = 1, int(tr[0]), 0
        while pos < 1 + ln:
            cnt = int(tr[pos + 1])
            en = [int(x) for x in tr[pos + 2: pos + 2 + cnt]]
            assert cnt <= 16 and not (set(en) & seen)
            seen |= set(en)
            n_en += cnt
            pos += 2 + cnt
        assert n_en == int(res.stats[q, 2]) and len(seen) == int(res.stats[q, 3])
    assert searched > 50
    # the eager form spends its budget on unevaluated vertices only: at least as many distances
    # per expansion as the lazy form
    base = runs[64]
    m = (base.stats[:, 0] > 0)
    assert (res.stats[m, 3] / res.stats[m, 0]).mean() >= (base.stats[m, 3] / base.stats[m, 0]).mean()


@pytest.mark.parametrize("warp", [16, 32])
def test_eager_ablation_chunk_by_chunk_replay(tiny_runs, warp):
    """The eager form depends on the chunk width (a second copy of an id inside one chunk is admitted,
    takes a slot and fails the insertion).  Alg. 4 takes its chunks inside one layer row (width m = 16
    here); the CUDA kernel's ablation switch scans 32 entries, i.e. two rows, per chunk.  Both widths
    are replayed from the recorded sequence of expanded vertices with a plain sequential filter."""
    wl, ix, _, _, _ = tiny_runs
    B = 16
    res = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 48, B=B, eager_hash=True, warp=warp, trace_cap=8192)
    checked = 0
    for q in range(wl.nq):
        if res.status[q] & (oracle.ST_EXACT | oracle.ST_EMPTY):
            continue
        l, r = oracle.rank_interval(ix.sorted_attr, int(wl.lo[q]), int(wl.hi[q]))
        ls, le = oracle.hotspot(l, r, ix.H, ix.n)
        seen = {oracle.entry_point(0, l, r, j) for j in range(16)}
        tr = res.trace[q]
        pos, ln = 1, int(tr[0])
        while pos < 1 + ln:
            u, cnt = int(tr[pos]), int(tr[pos + 1])
            flat = [int(v) for v in np.asarray(ix.enc[u, ls:le + 1]).ravel()]
            expect = []
            for c0 in range(0, len(flat), warp):
                passing = [v for v in flat[c0:c0 + warp] if v != 0xFFFFFFFF and l <= v <= r and v not in seen]
                take = passing[:B - len(expect)]
                expect += take
                seen |= set(take)
                if len(expect) == B:
                    break
            assert [int(x) for x in tr[pos + 2: pos + 2 + cnt]] == expect
            pos += 2 + cnt
            checked += 1
    assert checked > 1000


def test_recall_improves_with_beam_and_is_high(tiny_runs):
    wl, ix, gt_ids, _, runs = tiny_runs
    rec = {ef: oracle.recall(res.ids, gt_ids) for ef, res in runs.items()}
    assert rec[16] <= rec[64] + 0.02 and rec[64] <= rec[128] + 0.02
    assert rec[128] >= 0.85


def test_search_is_deterministic_and_thread_independent(tiny):
    wl, _, ix = tiny
    a = oracle.search(ix, wl.queries, wl.lo, wl.hi, 10, 48, threads=1)
    b = oracle.search(ix, wl.queries, wl.lo, wl.hi, 10, 48, threads=4)
    assert np.array_equal(a.ids, b.ids) and np.array_equal(a.dists, b.dists) and np.array_equal(a.stats, b.stats)


def test_iteration_cap_sets_status(tiny):
    wl, _, ix = tiny
    lo = np.full(8, -2**31, np.int32)
    hi = np.full(8, 2**31 - 1, np.int32)
    res = oracle.search(ix, wl.queries[:8], lo, hi, 10, 64, max_iters=5)
    assert np.all(res.stats[:, 0] == 5) and np.all(res.status & oracle.ST_ITER_CAP)


# ---------------------------------------------------------------------------------------------
# Alg. 2 main loop (lines 5-18) against a run worked by hand on a 16-vertex index
# ---------------------------------------------------------------------------------------------
def _alg2_golden_index():
    from alg2_golden import load
    g = load()
    ix = oracle.OracleIndex(n=g["n"], d=g["d"], d_pad=g["d_pad"], H=g["H"], m=g["m"], n_inv=0, ef_c=0, patience=0,
                            beta=0.0, gamma=0.0, seed=0, sorted_attr=g["sorted_attr"], rank2id=g["rank2id"],
                            vectors=g["vectors"], enc=g["enc"])
    return g, ix


def test_alg2_hand_trace_preconditions():
    """The inputs the hand trace starts from: endpoints, hotspot layers, entry points."""
    g, ix = _alg2_golden_index()
    assert oracle.rank_interval(ix.sorted_attr, g["lo"], g["hi"]) == (g["l_q"], g["r_q"])
    assert list(oracle.hotspot(g["l_q"], g["r_q"], g["H"], g["n"])) == g["hotspot"]
    eps = [oracle.entry_point(g["seed"], g["l_q"], g["r_q"], j) for j in range(g["epn"])]
    assert eps == g["entry_points"]


@pytest.mark.parametrize("warp", [2, 3, 32])
def test_alg2_hand_trace(warp):
    """Sequence of expanded vertices, EN(u) of every expansion, the pool after every merge (read
    back by stopping the loop after t expansions with k = ef_s), the result and the counters."""
    g, ix = _alg2_golden_index()
    lo = np.array([g["lo"]], dtype=np.int32)
    hi = np.array([g["hi"]], dtype=np.int32)
    kw = dict(epn=g["epn"], B=g["B"], seed=g["seed"], warp=warp)
    res = oracle.search(ix, g["query"], lo, hi, g["k"], g["ef_s"], trace_cap=256, **kw)
    tr = res.trace[0]
    rec, p = [], 1
    while p < 1 + tr[0]:
        cnt = int(tr[p + 1])
        rec.append((int(tr[p]), [int(v) for v in tr[p + 2:p + 2 + cnt]]))
        p += 2 + cnt
    assert rec == [(e["u"], e["en"]) for e in g["exp"]]
    assert res.ids[0].tolist() == g["result_ids"]
    assert np.array_equal(res.dists[0], np.sqrt(np.array(g["result_dist2"], dtype=np.float32)))
    assert res.status[0] == 0
    assert res.stats[0, 0] == g["stats_expansions"] and res.stats[0, 2] == g["stats_en"]
    assert res.stats[0, 3] == g["stats_distances"]
    if warp in (3, 32):
        assert res.stats[0, 1] == g["stats_rows_chunk%d" % warp]
    # the pool after t merges: stop after t expansions and return the whole pool
    for t, e in enumerate(g["exp"], start=1):
        cut = oracle.search(ix, g["query"], lo, hi, g["ef_s"], g["ef_s"], max_iters=t, **kw)
        ranks = [r for r, _ in e["pool"]]
        assert cut.ids[0].tolist() == [int(g["rank2id"][r]) for r in ranks], t
        assert np.array_equal(cut.dists[0], np.sqrt(np.array([d2 for _, d2 in e["pool"]], dtype=np.float32))), t
        assert bool(cut.status[0] & oracle.ST_ITER_CAP) == (t < len(g["exp"]))
    # termination follows ef_s, not k: asking for fewer results does not shorten the run
    res2 = oracle.search(ix, g["query"], lo, hi, 2, g["ef_s"], **kw)
    assert res2.stats[0, 0] == g["stats_expansions"] and res2.ids[0].tolist() == g["result_ids"][:2]
