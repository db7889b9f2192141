"""CUDA index builder: structural validity of its output, determinism, search quality on a par with
the host builder, and search parity (CUDA vs oracle) on the index it writes."""
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
