"""CUDA search path against the CPU oracle, element by element, through the C ABI."""
import ctypes
import os

import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def _gpu_search(frog, gix, wl_q, lo, hi, k, ef, trace_cap=0, **params):
    nq = wl_q.shape[0]
    q, tlo, thi = _dev(wl_q), _dev(lo), _dev(hi)
    status = torch.zeros(nq, dtype=torch.int32, device="cuda")
    stats = torch.zeros((nq, 4), dtype=torch.int32, device="cuda")
    trace = torch.zeros((nq, trace_cap), dtype=torch.int32, device="cuda") if trace_cap else None
    p = frog.Params(**params) if params else None
    ids, dists = gix.search(q, tlo, thi, k, ef, params=p, status=status, stats=stats, trace=trace)
    torch.cuda.synchronize()
    # the plain kernel (no counters, no trace) must give the same answers
    ids2, dists2 = gix.search(q, tlo, thi, k, ef, params=p)
    torch.cuda.synchronize()
    assert torch.equal(ids, ids2) and torch.equal(dists.view(torch.int32), dists2.view(torch.int32))   # bit for bit
    return (ids.cpu().numpy(), dists.cpu().numpy(), status.cpu().numpy().view(np.uint32),
            stats.cpu().numpy().view(np.uint32), None if trace is None else trace.cpu().numpy().view(np.uint32))


def _default_slots(ef):
    bits = 9
    while (1 << bits) < 16 * ef and bits < 13:
        bits += 1
    return 1 << bits


def _assert_parity(got, ref, check_dist_count=True, slots=None):
    ids, dists, status, stats, trace = got
    # returned ids: bit-exact; distances: identical arithmetic order, so also bit-exact, and in any
    # case within the 1e-4 relative tolerance the parity target states
    assert np.array_equal(ids, ref.ids)
    fin = np.isfinite(ref.dists)
    assert np.array_equal(np.isfinite(dists), fin)
    assert np.allclose(dists[fin], ref.dists[fin], rtol=1e-4, atol=0)
    assert np.array_equal(dists[fin], ref.dists[fin])
    forgot = (status & 16) != 0       # GPU-only bit: visited table overflowed (work, not results)
    assert np.array_equal(status & ~np.uint32(16), ref.status)
    # expansions, ENC rows read, ENs admitted: bit-exact (integer work)
    assert np.array_equal(stats[:, :3], ref.stats[:, :3])
    # distance evaluations: equal unless the GPU's bounded visited table forgot an entry, which
    # can only add evaluations
    assert np.all(stats[:, 3] >= ref.stats[:, 3])
    assert np.array_equal(stats[~forgot, 3], ref.stats[~forgot, 3])
    if slots is not None:
        # a sparsely filled table (1/8 load) has no probe run long enough to drop an entry
        assert not forgot[ref.stats[:, 3] <= slots // 8].any()
    elif check_dist_count:
        assert forgot.mean() <= 0.02
    if trace is not None and ref.trace is not None:
        assert np.array_equal(trace, ref.trace)         # every EN list of every expansion


@pytest.fixture(scope="module")
def tiny_gpu(libs, tiny):
    wl, path, ix = tiny
    gix = libs.Index.load(path, 0)
    yield wl, ix, gix
    gix.close()


@pytest.mark.parametrize("visited", ["bitmap", "hash"])
@pytest.mark.parametrize("ef", [16, 24, 32, 48, 64, 96, 128, 192, 256, 512])
def test_tiny_matches_oracle_at_every_beam_width(libs, tiny_gpu, ef, visited):
    wl, ix, gix = tiny_gpu
    ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, ef, trace_cap=40000 if ef <= 128 else 0)
    vis = libs.VISITED_BITMAP if visited == "bitmap" else libs.VISITED_HASH
    got = _gpu_search(libs, gix, wl.queries, wl.lo, wl.hi, wl.k, ef, trace_cap=40000 if ef <= 128 else 0,
                      visited=vis)
    _assert_parity(got, ref, slots=_default_slots(ef))
    if visited == "bitmap":
        # the bitmap is exact: nothing is ever evaluated twice
        assert not (got[2] & 16).any() and np.array_equal(got[3], ref.stats)


def test_tiny_plain_call_equals_ex_call(libs, tiny_gpu):
    wl, ix, gix = tiny_gpu
    q, lo, hi = _dev(wl.queries), _dev(wl.lo), _dev(wl.hi)
    ids, dists = gix.search(q, lo, hi, wl.k, 64)
    torch.cuda.synchronize()
    ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 64)
    assert np.array_equal(ids.cpu().numpy(), ref.ids)
    assert np.array_equal(dists.cpu().numpy(), ref.dists)


@pytest.mark.parametrize("params", [dict(epn=1), dict(epn=32), dict(budget=4), dict(budget=32), dict(budget=48),
                                    dict(budget=64), dict(budget=64, visited=2), dict(budget=40, no_hotspot=1),
                                    dict(no_hotspot=1), dict(seed=12345), dict(max_iters=7),
                                    dict(epn=7, budget=9, seed=3), dict(exact_below=700),
                                    dict(exact_below=3000, visited=2, budget=32), dict(eager_hash=1),
                                    dict(eager_hash=1, budget=64), dict(eager_hash=1, budget=5, epn=3),
                                    dict(eager_hash=1, no_hotspot=1, budget=33)])
def test_tiny_parameter_variants(libs, tiny_gpu, params):
    wl, ix, gix = tiny_gpu
    params = dict(params)
    okw = dict(epn=params.get("epn", 16), B=params.get("budget", 16), seed=params.get("seed", 0),
               no_hotspot=bool(params.get("no_hotspot", 0)), max_iters=params.get("max_iters", 0),
               exact_below=params.get("exact_below", 0), eager_hash=bool(params.get("eager_hash", 0)))
    cap = 0 if params.get("eager_hash") else 20000      # the eager ablation has no trace kernel
    ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 48, trace_cap=cap, **okw)
    got = _gpu_search(libs, gix, wl.queries, wl.lo, wl.hi, wl.k, 48, trace_cap=cap, **params)
    _assert_parity(got, ref, slots=_default_slots(48))


def test_k_equals_beam_and_k_one(libs, tiny_gpu):
    wl, ix, gix = tiny_gpu
    for k, ef in ((32, 32), (1, 16), (100, 128), (64, 64), (256, 512), (512, 512)):
        ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, k, ef)
        got = _gpu_search(libs, gix, wl.queries, wl.lo, wl.hi, k, ef)
        _assert_parity(got, ref, slots=_default_slots(ef))


def test_edge_ranges(libs, tiny_gpu):
    """Empty, inverted, single-object, fewer-than-k, exactly-beam-sized and full ranges."""
    wl, ix, gix = tiny_gpu
    srt = np.asarray(ix.sorted_attr)
    lo = np.array([5, -100, srt[0], srt[10], srt[100], srt[100], -2**31, srt[9999], srt[0]], np.int32)
    hi = np.array([4, -50, srt[0], srt[14], srt[131], srt[132], 2**31 - 1, 2**31 - 1, srt[9999]], np.int32)
    Q = wl.queries[: lo.size]
    ref = oracle.search(ix, Q, lo, hi, 10, 32, trace_cap=8000)
    got = _gpu_search(libs, gix, Q, lo, hi, 10, 32, trace_cap=8000)
    _assert_parity(got, ref, check_dist_count=False)
    assert ref.status[0] & oracle.ST_EMPTY and ref.status[1] & oracle.ST_EMPTY
    assert ref.status[4] & oracle.ST_EXACT and not (ref.status[5] & oracle.ST_EXACT)


def test_side_stream_and_back_to_back_calls(libs, tiny_gpu):
    """The call is asynchronous on the caller's stream: two searches queued back to back on a side
    stream (the second overwrites the scratch of the first) give the answers of separate calls."""
    wl, ix, gix = tiny_gpu
    q, lo, hi = _dev(wl.queries), _dev(wl.lo), _dev(wl.hi)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        a_ids, a_d = gix.search(q, lo, hi, wl.k, 32, stream=side, params=libs.Params(budget=64))
        b_ids, b_d = gix.search(q, lo, hi, wl.k, 96, stream=side)
    side.synchronize()
    ref_a = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 32, B=64)
    ref_b = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 96)
    assert np.array_equal(a_ids.cpu().numpy(), ref_a.ids) and np.array_equal(a_d.cpu().numpy(), ref_a.dists)
    assert np.array_equal(b_ids.cpu().numpy(), ref_b.ids) and np.array_equal(b_d.cpu().numpy(), ref_b.dists)


def test_concurrent_streams_share_one_index(libs, tiny_gpu):
    """Searches issued on different streams may overlap on the GPU: each stream works on its own
    scratch set (work counter, visited slabs, planning arrays), so the answers are those of
    separate calls.  More streams than scratch sets exist are served too (they queue)."""
    wl, ix, gix = tiny_gpu
    q, lo, hi = _dev(wl.queries), _dev(wl.lo), _dev(wl.hi)
    cfgs = [(32, 64), (96, 16), (48, 32), (64, 64), (24, 8), (128, 16), (100, 128)]   # (beam, budget) per stream
    refs = [oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, ef, B=B) for ef, B in cfgs]
    streams = [torch.cuda.Stream() for _ in cfgs]
    torch.cuda.synchronize()
    outs = [[] for _ in cfgs]
    for rep in range(4):
        for j, (ef, B) in enumerate(cfgs):
            outs[j].append(gix.search(q, lo, hi, wl.k, ef, stream=streams[j], params=libs.Params(budget=B)))
    torch.cuda.synchronize()
    for j, ref in enumerate(refs):
        for ids, dists in outs[j]:
            assert np.array_equal(ids.cpu().numpy(), ref.ids) and np.array_equal(dists.cpu().numpy(), ref.dists)


def test_non_finite_queries_terminate(libs, tiny_gpu):
    """Non-finite query components: the results are unspecified, but the call returns, every
    reported id lies in the query's range and no wait ran into its limit."""
    wl, ix, gix = tiny_gpu
    Q = wl.queries[:64].copy()
    Q[0::4, 3] = np.nan
    Q[1::4, :] = np.inf
    Q[2::4, 5] = -np.inf
    Q[3::4, :] = 3.0e38
    got = _gpu_search(libs, gix, Q, wl.lo[:64], wl.hi[:64], wl.k, 48, budget=64)
    ids, dists, status, stats, _ = got
    assert not (status & 32).any()
    assert np.all(stats[:, 0] <= 16 * 48)                                  # the expansion cap held
    valid = ids >= 0
    a = wl.attrs[np.where(valid, ids, 0)]
    assert np.all(~valid | ((a >= wl.lo[:64, None]) & (a <= wl.hi[:64, None])))


def test_small_visited_table_changes_work_not_results(libs, tiny_gpu):
    """A visited table far too small forgets entries: more distance evaluations, same answers."""
    wl, ix, gix = tiny_gpu
    ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 64, trace_cap=20000)
    got = _gpu_search(libs, gix, wl.queries, wl.lo, wl.hi, wl.k, 64, trace_cap=20000, hash_bits=6,
                      visited=libs.VISITED_HASH)
    _assert_parity(got, ref, check_dist_count=False)
    assert got[3][:, 3].sum() > ref.stats[:, 3].sum()
    assert (got[2] & 16).any()


def test_search_kernel_time_is_reported_on_request(libs, tiny_gpu):
    """debug_flags bit 4 makes the call record events around the search kernel alone; the time read
    back is positive and no longer than the whole call (two planning kernels included) as timed by
    events on the same stream; without the flag there is nothing to read."""
    wl, ix, gix = tiny_gpu
    q, lo, hi = _dev(wl.queries), _dev(wl.lo), _dev(wl.hi)
    side = torch.cuda.Stream()
    with pytest.raises(libs.FrogError):
        gix.kernel_ms(stream=side)                         # no timed launch on this stream yet
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    gix.search(q, lo, hi, wl.k, 64, params=libs.Params(debug_flags=16), stream=side)    # warm
    side.synchronize()
    e0.record(side)
    ids, _ = gix.search(q, lo, hi, wl.k, 64, params=libs.Params(debug_flags=16), stream=side)
    e1.record(side)
    ms = gix.kernel_ms(stream=side)
    side.synchronize()
    assert 0.0 < ms <= e0.elapsed_time(e1) * 1.05
    ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 64)
    assert np.array_equal(ids.cpu().numpy(), ref.ids)
    gix.search(q, lo, hi, wl.k, 64, stream=side)            # an untimed launch on the same stream
    with pytest.raises(libs.FrogError):
        gix.kernel_ms(stream=side)
    # the launch-wide status word: nothing to report after a normal launch; unknown streams are refused
    assert gix.last_status(stream=side) == 0
    with pytest.raises(libs.FrogError):
        gix.last_status(stream=torch.cuda.Stream())


def test_empty_batch_and_argument_errors(libs, tiny_gpu):
    wl, ix, gix = tiny_gpu
    q, lo, hi = _dev(wl.queries), _dev(wl.lo), _dev(wl.hi)
    ids, _ = gix.search(q[:0], lo[:0], hi[:0], 10, 32)
    assert ids.shape == (0, 10)
    for k, ef in ((0, 32), (33, 32), (10, 0), (10, 513)):
        with pytest.raises(libs.FrogError) as e:
            gix.search(q, lo, hi, k, ef)
        assert e.value.code == 1
    with pytest.raises(libs.FrogError):
        gix.search(q, lo, hi, 10, 32, params=libs.Params(epn=33))
    with pytest.raises(libs.FrogError):
        gix.search(q, lo, hi, 10, 32, params=libs.Params(budget=129))
    with pytest.raises(libs.FrogError):
        gix.search(q, lo, hi, 10, 32, params=libs.Params(exact_below=-1))
    with pytest.raises(libs.FrogError):                  # the ablation exists for the bitmap form only
        gix.search(q, lo, hi, 10, 32, params=libs.Params(eager_hash=1, visited=libs.VISITED_HASH))
    # a failed call leaves the index usable
    ids, _ = gix.search(q, lo, hi, 10, 32)
    torch.cuda.synchronize()
    assert ids.shape == (wl.nq, 10)


def test_exact_search_matches_definition(libs, tiny_gpu):
    wl, ix, gix = tiny_gpu
    q, lo, hi = _dev(wl.queries), _dev(wl.lo), _dev(wl.hi)
    for k in (1, 10, 100):
        ids, dists = gix.exact_search(q, lo, hi, k)
        torch.cuda.synchronize()
        ref_ids, ref_d, _ = oracle.exact_slab(ix, wl.queries, wl.lo, wl.hi, k, mode=1)
        assert np.array_equal(ids.cpu().numpy(), ref_ids)
        assert np.array_equal(dists.cpu().numpy(), ref_d)
        # against the float64 definition: same ids except at near-ties, distances within 1e-4
        def_ids, def_d = oracle.exact_scan(wl.vectors, wl.attrs, wl.queries, wl.lo, wl.hi, k, mode=0)
        fin = np.isfinite(def_d)
        assert np.allclose(dists.cpu().numpy()[fin], def_d[fin], rtol=1e-4)
        assert (ids.cpu().numpy() == def_ids).mean() > 0.999


def test_host_buffer_call_matches(libs, tiny_gpu):
    wl, ix, gix = tiny_gpu
    ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 64)
    ids, dists = gix.search_host(torch.from_numpy(wl.queries).pin_memory(),
                                 torch.from_numpy(wl.lo).pin_memory(),
                                 torch.from_numpy(wl.hi).pin_memory(), wl.k, 64)
    assert np.array_equal(ids.numpy(), ref.ids) and np.array_equal(dists.numpy(), ref.dists)
    # pageable inputs and outputs take the staged path; a second, larger call regrows the staging area
    p_ids = torch.empty((wl.nq, wl.k), dtype=torch.int32)
    p_d = torch.empty((wl.nq, wl.k), dtype=torch.float32)
    gix.search_host(wl.queries, wl.lo, wl.hi, wl.k, 64, out_ids=p_ids, out_dists=p_d)
    assert np.array_equal(p_ids.numpy(), ref.ids) and np.array_equal(p_d.numpy(), ref.dists)
    reps = 3
    Q = np.tile(wl.queries, (reps, 1))
    ids, dists = gix.search_host(Q, np.tile(wl.lo, reps), np.tile(wl.hi, reps), wl.k, 64)
    assert np.array_equal(ids.numpy(), np.tile(ref.ids, (reps, 1)))


def test_recall_within_tolerance_of_oracle(libs, tiny_gpu):
    wl, ix, gix = tiny_gpu
    gt, _, _ = oracle.exact_slab(ix, wl.queries, wl.lo, wl.hi, wl.k, mode=0)
    for ef in (16, 64):
        ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, ef)
        got = _gpu_search(libs, gix, wl.queries, wl.lo, wl.hi, wl.k, ef)
        assert abs(oracle.recall(got[0], gt) - oracle.recall(ref.ids, gt)) <= 0.005


# ---- the other workload shapes at sizes the oracle finishes in seconds ------------------------
@pytest.mark.parametrize("name,n,nq", [("sift", 60_000, 300), ("deep1m", 50_000, 300),
                                        ("deep10m", 70_001, 300), ("text", 20_000, 150)])
def test_scaled_workloads_match_oracle(libs, cache_dir, name, n, nq):
    from conftest import build_scaled
    wl, path, ix = build_scaled(libs, cache_dir, name, n, nq)
    gix = libs.Index.load(path, 0)
    try:
        for ef, k, B, vis in ((32, 10, 16, libs.VISITED_BITMAP), (100, 100, 16, libs.VISITED_HASH),
                              (64, 10, 32, libs.VISITED_BITMAP), (48, 10, 24, libs.VISITED_HASH),
                              (48, 10, 64, libs.VISITED_BITMAP), (32, 10, 96, libs.VISITED_BITMAP),
                              (40, 10, 128, libs.VISITED_HASH), (24, 10, 128, libs.VISITED_BITMAP),
                              (300, 10, 96, libs.VISITED_BITMAP)):
            ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, k, ef, B=B, trace_cap=60000)
            got = _gpu_search(libs, gix, wl.queries, wl.lo, wl.hi, k, ef, trace_cap=60000, budget=B, visited=vis)
            _assert_parity(got, ref, slots=_default_slots(ef))
        q, lo, hi = _dev(wl.queries), _dev(wl.lo), _dev(wl.hi)
        ids, dists = gix.exact_search(q, lo, hi, 10)
        torch.cuda.synchronize()
        ref_ids, ref_d, _ = oracle.exact_slab(ix, wl.queries, wl.lo, wl.hi, 10, mode=1)
        assert np.array_equal(ids.cpu().numpy(), ref_ids) and np.array_equal(dists.cpu().numpy(), ref_d)
    finally:
        gix.close()


@pytest.mark.parametrize("name,n,nq", [("sift", 60_000, 300), ("deep1m", 50_000, 300)])
def test_row_specialised_kernel_at_every_pool_size(libs, cache_dir, name, n, nq):
    """Rows of 512 and 384 bytes are searched by a kernel specialised for them (every pool size from
    32 to 512 keys — 32, 64, 128, 192, 256, 512 — is its own instantiation).  The plain call (which takes it) against the oracle and,
    inside _gpu_search, against the counting variant of the general kernel, bit for bit; then the
    general kernel forced by debug_flags bit 2 against the same reference."""
    from conftest import build_scaled
    wl, path, ix = build_scaled(libs, cache_dir, name, n, nq)
    gix = libs.Index.load(path, 0)
    try:
        for ef, k, kw in ((24, 10, dict(budget=64)), (64, 64, dict(budget=64, epn=32)), (128, 10, dict(budget=64)),
                          (176, 10, dict(budget=64)), (32, 10, dict(budget=96)), (160, 10, dict(budget=128)),
                          (200, 100, dict(budget=48)), (256, 10, dict(budget=64, max_iters=40)),
                          (512, 10, dict(budget=64)), (96, 10, dict(budget=64, exact_below=2000)),
                          (40, 10, dict(budget=64, no_hotspot=1, seed=9))):
            ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, k, ef, epn=kw.get("epn", 16), B=kw["budget"],
                                max_iters=kw.get("max_iters", 0), exact_below=kw.get("exact_below", 0),
                                no_hotspot=bool(kw.get("no_hotspot", 0)), seed=kw.get("seed", 0))
            got = _gpu_search(libs, gix, wl.queries, wl.lo, wl.hi, k, ef, **kw)
            _assert_parity(got, ref)
            q, lo, hi = _dev(wl.queries), _dev(wl.lo), _dev(wl.hi)
            ids, dists = gix.search(q, lo, hi, k, ef, params=libs.Params(debug_flags=4, **kw))
            torch.cuda.synchronize()
            assert np.array_equal(ids.cpu().numpy(), ref.ids) and np.array_equal(dists.cpu().numpy(), ref.dists)
    finally:
        gix.close()


@pytest.mark.parametrize("name,n,nq", [("sift", 60_000, 300), ("deep1m", 50_000, 300), ("text", 20_000, 150)])
def test_a_row_copy_that_never_completes_is_reported(libs, cache_dir, name, n, nq):
    """The error path of the search kernels, exercised without a fault: with debug_flags bit 5 the kernel
    requests no row copy and its bounded waits give up after 64 polls, so every gather ends the way a
    copy time-out would, with nothing in flight.  Every row is then padding, every query that had
    anything to evaluate carries FROG_ST_COPY_TIMEOUT, the launch-wide status word reports it to a
    caller that passed no status array, and the next call on the same index answers normally.
    Without `stats` the kernel for 384- and 512-byte rows runs (the general one for other rows, which
    ignores the flag there: its plain form is checked through the counting variant), with `stats` the
    counting variant of the general kernel."""
    from conftest import build_scaled
    wl, path, ix = build_scaled(libs, cache_dir, name, n, nq)
    gix = libs.Index.load(path, 0)
    try:
        q, lo, hi = _dev(wl.queries), _dev(wl.lo), _dev(wl.hi)
        ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, 10, 32, B=64)
        nonempty = (ref.status & 1) == 0
        assert nonempty.sum() > nq // 2
        prm = libs.Params(budget=64, debug_flags=32)
        for with_stats in ([False, True] if name != "text" else [True]):
            status = torch.zeros(nq, dtype=torch.int32, device="cuda")
            stats = torch.zeros((nq, 4), dtype=torch.int32, device="cuda") if with_stats else None
            ids, dists = gix.search(q, lo, hi, 10, 32, params=prm, status=status, stats=stats)
            torch.cuda.synchronize()
            st = status.cpu().numpy().view(np.uint32)
            assert (ids.cpu().numpy() == -1).all() and np.isinf(dists.cpu().numpy()).all(), with_stats
            assert ((st[nonempty] & 32) != 0).all(), with_stats
            assert gix.last_status() & 32, with_stats
            # the same launch for a caller without a status array: the launch-wide word still tells
            gix.search(q, lo, hi, 10, 32, params=prm, stats=stats)
            torch.cuda.synchronize()
            assert gix.last_status() & 32, with_stats
            # ... and the index answers normally afterwards
            got = _gpu_search(libs, gix, wl.queries, wl.lo, wl.hi, 10, 32, budget=64)
            _assert_parity(got, ref)
            assert gix.last_status() == 0
    finally:
        gix.close()


@pytest.mark.parametrize("name,n,nq", [("sift", 60_000, 300), ("deep1m", 50_000, 300), ("deep10m", 70_001, 300)])
def test_visited_hash_table_form(libs, cache_dir, name, n, nq):
    """The visited set as a hash table of ranks in global scratch (what large indexes get at beam widths
    up to 64), forced here on small indexes: with the full-size table no query outgrows it; with 256 and
    64 slots almost every query moves to its bitmap slab part of the way.  Results equal the oracle's
    and the bitmap form's bit for bit, launch after launch (tables and slabs are left clean)."""
    from conftest import build_scaled
    wl, path, ix = build_scaled(libs, cache_dir, name, n, nq)
    gix = libs.Index.load(path, 0)
    try:
        q, lo, hi = _dev(wl.queries), _dev(wl.lo), _dev(wl.hi)
        for ef, k, B in ((32, 10, 64), (64, 10, 64), (24, 5, 16), (48, 48, 33), (24, 10, 96), (100, 10, 128)):
            ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, k, ef, B=B)
            for bits in (0, 8, 6, 0):
                prm = libs.Params(budget=B, debug_flags=8 | (bits << 8))
                ids, dists = gix.search(q, lo, hi, k, ef, params=prm)
                torch.cuda.synchronize()
                assert np.array_equal(ids.cpu().numpy(), ref.ids), (ef, bits)
                assert np.array_equal(dists.cpu().numpy(), ref.dists), (ef, bits)
            ids, dists = gix.search(q, lo, hi, k, ef, params=libs.Params(budget=B, visited=libs.VISITED_BITMAP))
            torch.cuda.synchronize()
            assert np.array_equal(ids.cpu().numpy(), ref.ids) and np.array_equal(dists.cpu().numpy(), ref.dists)
    finally:
        gix.close()


def test_odd_dimension(libs, cache_dir):
    rng = np.random.default_rng(2)
    V = rng.standard_normal((3000, 10)).astype(np.float32)
    a = rng.integers(0, 500, 3000).astype(np.int32)
    path = os.path.join(cache_dir, "odd_gpu.idx")
    libs.build_index(V, a, path, n_inv=5)
    ix = oracle.load_index(path)
    gix = libs.Index.load(path, 0)
    Q = rng.standard_normal((64, 10)).astype(np.float32)
    lo = rng.integers(0, 400, 64).astype(np.int32)
    hi = (lo + rng.integers(0, 100, 64)).astype(np.int32)
    ref = oracle.search(ix, Q, lo, hi, 5, 32)
    got = _gpu_search(libs, gix, Q, lo, hi, 5, 32)
    _assert_parity(got, ref)
    gix.close()


@pytest.mark.parametrize("n,d,m,n_inv", [(1, 8, 16, 7), (2, 16, 16, 7), (33, 24, 16, 3), (200, 40, 8, 4),
                                          (1000, 64, 32, 5), (777, 12, 4, 2)])
def test_small_and_odd_indexes(libs, cache_dir, n, d, m, n_inv):
    """Degenerate index shapes: a single object, fewer objects than a warp, one retained layer,
    row sizes that do and do not qualify for the 4-row tensor gather (slots of 32, 64, 96, 160, 256
    and 48 bytes), several ENC widths."""
    rng = np.random.default_rng(100 + n)
    V = rng.standard_normal((n, d)).astype(np.float32)
    a = rng.integers(0, max(2, n // 2), n).astype(np.int32)
    path = os.path.join(cache_dir, f"small_{n}_{d}_{m}.idx")
    libs.build_index(V, a, path, m=m, n_inv=n_inv, ef_c=64)
    ix = oracle.load_index(path)
    gix = libs.Index.load(path, 0)
    try:
        nq = 96
        Q = rng.standard_normal((nq, d)).astype(np.float32)
        lo = rng.integers(-2, max(2, n // 2), nq).astype(np.int32)
        hi = (lo + rng.integers(0, max(2, n // 2) + 2, nq)).astype(np.int32)
        for k, ef, B in ((1, 8, 16), (5, 16, 64), (10, 48, 33)):
            ref = oracle.search(ix, Q, lo, hi, k, ef, B=B)
            got = _gpu_search(libs, gix, Q, lo, hi, k, ef, budget=B)
            _assert_parity(got, ref)
    finally:
        gix.close()


def test_index_info_and_from_host(libs, tiny):
    wl, path, ix = tiny
    gix = libs.Index.load(path, 0)
    info = gix.info
    assert (info.n, info.d, info.d_pad, info.H, info.m) == (ix.n, ix.d, ix.d_pad, ix.H, ix.m)
    assert info.device_bytes >= ix.n * (8 + 4 * ix.d_pad + 4 * ix.H * ix.m)
    h = ctypes.c_void_p()
    shape = libs.IndexInfo(n=ix.n, d=ix.d, d_pad=ix.d_pad, H=ix.H, m=ix.m)
    arrs = [np.ascontiguousarray(a) for a in (ix.sorted_attr, ix.rank2id, ix.vectors, ix.enc)]
    rc = libs._lib.frog_index_from_host(*[a.ctypes.data_as(ctypes.c_void_p) for a in arrs],
                                        ctypes.byref(shape), 0, ctypes.byref(h))
    assert rc == 0
    g2 = libs.Index(h)
    ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, wl.k, 32)
    got = _gpu_search(libs, g2, wl.queries, wl.lo, wl.hi, wl.k, 32)
    _assert_parity(got, ref)
    g2.close()
    gix.close()


# ---- half-precision storage -----------------------------------------------------------------------
@pytest.mark.parametrize("name,n,nq", [("tiny", 10_000, 200), ("deep1m", 50_000, 300), ("text", 20_000, 100),
                                        ("sift", 60_000, 300)])
def test_f16_storage_equals_oracle_on_rounded_vectors(libs, cache_dir, name, n, nq):
    """fp16 storage, fp32 arithmetic: bit-exact against the oracle run on the fp16-rounded vectors;
    recall against the fp32 ground truth stays close to the fp32 search."""
    from conftest import build_scaled
    wl, path, ix = build_scaled(libs, cache_dir, name, n, nq)
    ix16 = oracle.rounded_to_f16(ix)
    gix = libs.Index.load(path, 0)
    try:
        gix.enable_f16()
        gix.enable_f16()                                    # idempotent
        for ef, B in ((48, 16), (64, 32)):
            ref = oracle.search(ix16, wl.queries, wl.lo, wl.hi, 10, ef, B=B, trace_cap=60000)
            got = _gpu_search(libs, gix, wl.queries, wl.lo, wl.hi, 10, ef, trace_cap=60000, budget=B,
                              storage=libs.STORAGE_F16)
            _assert_parity(got, ref, slots=_default_slots(ef))
            assert np.array_equal(got[3], ref.stats)
        gt, _, _ = oracle.exact_slab(ix, wl.queries, wl.lo, wl.hi, 10, mode=0)
        ref32 = oracle.search(ix, wl.queries, wl.lo, wl.hi, 10, 64, B=32)
        assert abs(oracle.recall(got[0], gt) - oracle.recall(ref32.ids, gt)) <= 0.01
        if name == "sift":
            # integer components 0..255 are exact in fp16: the two storages give the same answer
            assert np.array_equal(got[0], ref32.ids) and np.array_equal(got[1], ref32.dists)
        # the request is refused where it cannot be served
        with pytest.raises(libs.FrogError):
            _gpu_search(libs, gix, wl.queries, wl.lo, wl.hi, 10, 32, storage=libs.STORAGE_F16,
                        visited=libs.VISITED_HASH)
    finally:
        gix.close()
    g2 = libs.Index.load(path, 0)
    with pytest.raises(libs.FrogError):                      # not enabled on this handle
        _gpu_search(libs, g2, wl.queries, wl.lo, wl.hi, 10, 32, storage=libs.STORAGE_F16)
    g2.close()
