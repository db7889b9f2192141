"""CUDA index builder against the host builder, element by element (the two follow the same steps
in the same arithmetic order and must write the same file), plus structural validity of the output,
determinism, the construction switches, the report of a copy that never completes, and search parity
(CUDA vs oracle) on the index it writes."""
import os

import numpy as np
import pytest

import datagen
import oracle

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

BOT = 0xFFFFFFFF


@pytest.fixture(scope="module")
def built(libs, cache_dir):
    wl = datagen.make_workload("sift", n=40_000, nq=400)
    pg = os.path.join(cache_dir, "gpu_builder.idx")
    pc = os.path.join(cache_dir, "cpu_builder.idx")
    libs.build_index_gpu(wl.vectors, wl.attrs, pg, seed=wl.seed)
    libs.build_index(wl.vectors, wl.attrs, pc, seed=wl.seed)
    return wl, pg, pc


def test_header_and_rank_domain_match_the_host_builder(built):
    wl, pg, pc = built
    g, c = oracle.load_index(pg), oracle.load_index(pc)
    assert (g.n, g.d, g.d_pad, g.H, g.m, g.n_inv, g.ef_c, g.patience) == \
           (c.n, c.d, c.d_pad, c.H, c.m, c.n_inv, c.ef_c, c.patience)
    assert np.array_equal(g.sorted_attr, c.sorted_attr) and np.array_equal(g.rank2id, c.rank2id)
    assert np.array_equal(g.vectors, c.vectors)


def test_files_are_identical_to_the_host_builder(built):
    wl, pg, pc = built
    g, c = oracle.load_index(pg), oracle.load_index(pc)
    assert np.array_equal(np.asarray(g.enc), np.asarray(c.enc))            # every ENC row of every layer
    with open(pg, "rb") as a, open(pc, "rb") as b:
        assert a.read() == b.read()


@pytest.mark.parametrize("name,n,kw", [("deep1m", 50_000, {}), ("text", 20_000, {}), ("deep10m", 30_001, {}),
                                        ("tiny", 10_000, {}), ("tiny", 3_000, dict(m=8, ef_c=40, n_inv=4)),
                                        ("sift", 20_000, dict(flags=3)), ("deep1m", 20_000, dict(flags=1)),
                                        ("text", 8_000, dict(flags=2)), ("tiny", 4_000, dict(beta=0.0)),
                                        ("tiny", 300, dict(n_inv=12)), ("tiny", 70, dict(n_inv=2)),
                                        ("tiny", 2, {}), ("tiny", 1, {})])
def test_enc_arrays_equal_the_host_builder_on_other_shapes(libs, cache_dir, name, n, kw):
    """Row sizes of 384, 512 and 3,072 bytes (the last takes the candidate-to-candidate distances in
    six column chunks), m = 32 / ef_c = 256, duplicate attributes, leaves above and below 65 objects,
    a single retained layer, the construction switches (3 = the paper's Sec. 6.1 as written) and
    beta = 0 (ENC order = vector-distance order)."""
    wl = datagen.make_workload(name, n=n, nq=4)
    pg = os.path.join(cache_dir, f"eq_gpu_{name}_{n}.idx")
    pc = os.path.join(cache_dir, f"eq_cpu_{name}_{n}.idx")
    libs.build_index_gpu(wl.vectors, wl.attrs, pg, seed=wl.seed, **kw)
    libs.build_index(wl.vectors, wl.attrs, pc, seed=wl.seed, **kw)
    g, c = oracle.load_index(pg), oracle.load_index(pc)
    assert (g.H, g.m) == (c.H, c.m)
    eg, ec = np.asarray(g.enc), np.asarray(c.enc)
    diff = np.argwhere(eg != ec)
    assert diff.size == 0, f"{len(diff)} ENC entries differ, first at (rank, layer, slot) = {diff[0]}"
    with open(pg, "rb") as a, open(pc, "rb") as b:
        assert a.read() == b.read()
    os.remove(pg)
    os.remove(pc)


def test_construction_switches_change_the_index_as_described(libs, cache_dir):
    """FROG_BUILD_ENC_FUSION_NEAREST: every ENC row holds the m fusion-nearest of the object's
    candidates, i.e. no row of the default build is fusion-nearer at any position; and the switches
    are recorded in the file header."""
    import struct
    wl = datagen.make_workload("tiny", n=5_000, nq=4)
    paths = {}
    for flags in (0, 1, 2, 3):
        paths[flags] = os.path.join(cache_dir, f"sw_{flags}.idx")
        libs.build_index_gpu(wl.vectors, wl.attrs, paths[flags], seed=wl.seed, flags=flags)
        with open(paths[flags], "rb") as f:
            assert struct.unpack_from("<I", f.read(256), 68)[0] == flags
    base, lit = oracle.load_index(paths[0]), oracle.load_index(paths[2])
    assert not np.array_equal(np.asarray(base.enc), np.asarray(lit.enc))
    V = np.asarray(base.vectors, dtype=np.float64)

    def fusion(u, row):
        row = row[row != BOT].astype(np.int64)
        dv = np.sqrt(((V[row] - V[u]) ** 2).sum(1))
        return dv * (1 - 0.2 * (1 - (np.abs(row - u) / (base.n - 1)) ** 0.5))
    h = base.H - 1          # leaf rows: the same candidates under both rules (no reverse-edge effect on the set)
    for u in range(0, base.n, 211):
        a, b = fusion(u, np.asarray(lit.enc[u, h])), fusion(u, np.asarray(base.enc[u, h]))
        k = min(a.size, b.size)
        assert np.all(a[:k] <= b[:k] * (1 + 1e-9))


def test_a_copy_that_never_completes_is_reported(libs, cache_dir):
    """The builder's kernels wait for their bulk copies with a polling limit and record a give-up;
    the call then returns the CUDA error code and writes no file.  The test hook (bits 16..31 of the
    switches) issues no copy and lets every wait run out after 3 polls: nothing is in flight, nothing
    faults, and the device stays usable."""
    wl = datagen.make_workload("tiny", n=2_000, nq=4)
    p = os.path.join(cache_dir, "never.idx")
    with pytest.raises(libs.FrogError) as e:
        libs.build_index_gpu(wl.vectors, wl.attrs, p, seed=wl.seed, flags=3 << 16)
    assert e.value.code == 5 and not os.path.exists(p)
    libs.build_index_gpu(wl.vectors, wl.attrs, p, seed=wl.seed)            # the next build is fine
    assert oracle.load_index(p).n == 2_000


def test_enc_rows_are_valid(built):
    wl, pg, _ = built
    ix = oracle.load_index(pg)
    enc = np.asarray(ix.enc)
    us = np.arange(0, ix.n, 13)
    for h in range(ix.H):
        seg = np.array([oracle.segment_at(ix.n, h, int(u)) for u in us])
        rows = enc[us, h, :]
        valid = rows != BOT
        assert np.all(((rows >= seg[:, :1]) & (rows <= seg[:, 1:])) | ~valid)      # inside the segment
        assert not np.any(rows == us[:, None])                                    # never itself
        for r in rows[:400]:
            v = r[r != BOT]
            assert len(set(v.tolist())) == v.size and np.all(r[v.size:] == BOT)   # no repeats, empties last
    # rows are stored in ascending fusion distance
    V = np.asarray(ix.vectors, dtype=np.float64)
    for u in range(0, ix.n, 997):
        for h in (0, ix.H // 2, ix.H - 1):
            row = enc[u, h]
            row = row[row != BOT]
            dv = np.sqrt(((V[row] - V[u]) ** 2).sum(1))
            da = np.abs(row.astype(np.int64) - u) / (ix.n - 1)
            df = dv * (1 - 0.2 * (1 - da ** 0.5))
            assert np.all(np.diff(df) >= -1e-6 * df[:-1].clip(1e-12))


def test_build_is_deterministic(libs, built, cache_dir):
    wl, pg, _ = built
    p2 = os.path.join(cache_dir, "gpu_builder_again.idx")
    libs.build_index_gpu(wl.vectors, wl.attrs, p2, seed=wl.seed)
    with open(pg, "rb") as a, open(p2, "rb") as b:
        assert a.read() == b.read()


def test_search_quality_matches_the_host_builder(libs, built):
    wl, pg, pc = built
    q = torch.from_numpy(wl.queries).cuda()
    lo = torch.from_numpy(wl.lo).cuda()
    hi = torch.from_numpy(wl.hi).cuda()
    rec = {}
    for name, path in (("gpu", pg), ("cpu", pc)):
        ix = libs.Index.load(path, 0)
        gt, _ = ix.exact_search(q, lo, hi, 10)
        ids, _ = ix.search(q, lo, hi, 10, 64, params=libs.Params(budget=32))
        torch.cuda.synchronize()
        rec[name] = oracle.recall(ids.cpu().numpy(), gt.cpu().numpy())
        ix.close()
    assert rec["gpu"] >= 0.93 and abs(rec["gpu"] - rec["cpu"]) <= 0.02


def test_search_parity_on_the_gpu_built_index(libs, built):
    wl, pg, _ = built
    ix = oracle.load_index(pg)
    gix = libs.Index.load(pg, 0)
    q = torch.from_numpy(wl.queries).cuda()
    lo = torch.from_numpy(wl.lo).cuda()
    hi = torch.from_numpy(wl.hi).cuda()
    ref = oracle.search(ix, wl.queries, wl.lo, wl.hi, 10, 48, B=32)
    ids, d = gix.search(q, lo, hi, 10, 48, params=libs.Params(budget=32))
    torch.cuda.synchronize()
    assert np.array_equal(ids.cpu().numpy(), ref.ids) and np.array_equal(d.cpu().numpy(), ref.dists)
    gix.close()


def test_other_shapes_and_limits(libs, cache_dir):
    # d not a multiple of 4, m = 32 / ef_c = 256 defaults of high dimension, tiny n, one layer
    rng = np.random.default_rng(3)
    for n, d, kw in ((5000, 10, {}), (3000, 320, {}), (300, 16, dict(n_inv=12)), (1, 8, {})):
        V = rng.standard_normal((n, d)).astype(np.float32)
        a = rng.integers(0, 1000, n).astype(np.int32)
        p = os.path.join(cache_dir, f"gb_{n}_{d}.idx")
        libs.build_index_gpu(V, a, p, **kw)
        ix = oracle.load_index(p)
        assert ix.n == n and ix.d == d
        if n > 100:
            Q = rng.standard_normal((50, d)).astype(np.float32)
            lo = np.full(50, 0, np.int32)
            hi = np.full(50, 999, np.int32)
            res = oracle.search(ix, Q, lo, hi, 5, 64, B=32)
            gt, _, _ = oracle.exact_slab(ix, Q, lo, hi, 5)
            assert oracle.recall(res.ids, gt) > 0.8
    V = np.zeros((100, 8), np.float32)
    a = np.arange(100, dtype=np.int32)
    with pytest.raises(libs.FrogError) as e:
        libs.build_index_gpu(V, a, os.path.join(cache_dir, "x.idx"), m=48, ef_c=64)
    assert e.value.code == 6
