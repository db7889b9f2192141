"""Host index builder: closed forms of the fusion distance (Eq. 3), structural invariants of the
n x H x m ENC array (Sec. 4), determinism, and the file format.  No GPU."""
import os
import struct

import numpy as np
import pytest

import datagen
import oracle


def test_fusion_distance_limits_and_monotonicity(libs):
    f = libs.fusion_distance
    # Eq. 3: delta_a = 0 -> (1 - beta) delta_v; delta_a = 1 -> delta_v; beta = 0 -> delta_v
    assert f(2.0, 0.0, 0.2, 0.5) == pytest.approx(1.6)
    assert f(2.0, 1.0, 0.2, 0.5) == pytest.approx(2.0)
    assert f(2.0, 0.37, 0.0, 0.5) == pytest.approx(2.0)
    za = np.linspace(0, 1, 50)
    vals = [f(1.0, z, 0.2, 0.5) for z in za]
    assert np.all(np.diff(vals) > 0)                        # increases with attribute distance
    # worked value: 3 * (1 - 0.2 * (1 - 0.25^0.5)) = 3 * 0.9
    assert f(3.0, 0.25, 0.2, 0.5) == pytest.approx(2.7)
    # pairwise rule of Sec. 5.2: x before y iff X_x / X_y < W(Z_y) / W(Z_x)
    rng = np.random.default_rng(0)
    for _ in range(200):
        xx, xy = rng.uniform(0.1, 3, 2)
        zx, zy = rng.uniform(0, 1, 2)
        w = lambda z: 1 - 0.2 + 0.2 * z ** 0.5
        assert (f(xx, zx, 0.2, 0.5) < f(xy, zy, 0.2, 0.5)) == (xx / xy < w(zy) / w(zx))


def test_fusion_distance_first_order_shift_of_attribute_distance(libs):
    """Sec. 5.2: keeping the q-fraction of candidates with the smallest fusion distance lowers the
    mean attribute distance of the kept ones by alpha * beta * C_gamma to first order in beta, with
    C_gamma = gamma / (2 (gamma + 1)(gamma + 2)) for Z ~ U(0,1), when X and Z are independent and
    F_X(x) ~ x^alpha near 0.  Monte Carlo with X = U^(1/alpha) (F_X(x) = x^alpha exactly)."""
    f = libs.fusion_distance
    rng = np.random.default_rng(11)
    N, q, alpha, gamma = 400_000, 0.02, 2.0, 0.5
    X = rng.uniform(0, 1, N) ** (1.0 / alpha)
    Z = rng.uniform(0, 1, N)
    c_gamma = gamma / (2 * (gamma + 1) * (gamma + 2))
    keep = int(q * N)
    base = Z[np.argsort(X)[:keep]].mean()                   # beta = 0: selection ignores Z
    assert abs(base - 0.5) < 0.01
    shifts = {}
    for beta in (0.05, 0.1):
        Y = np.fromiter((f(float(x), float(z), beta, gamma) for x, z in zip(X, Z)), dtype=np.float64, count=N)
        shifts[beta] = base - Z[np.argsort(Y)[:keep]].mean()
        predicted = alpha * beta * c_gamma
        assert 0.7 * predicted < shifts[beta] < 1.4 * predicted, (beta, shifts[beta], predicted)
    assert shifts[0.1] > 1.6 * shifts[0.05]                 # first order in beta


def test_retained_depth(libs):
    # H = ceil(log2 n) + 1 - n_inv
    assert libs.retained_depth(10_000, 7) == 8
    assert libs.retained_depth(1_000_000, 7) == 14
    assert libs.retained_depth(10_000_000, 7) == 18
    assert libs.retained_depth(1_000_000, 6) == 15
    assert libs.retained_depth(100, 20) == 1


def test_file_format_and_rank_domain(tiny):
    wl, path, ix = tiny
    with open(path, "rb") as f:
        hdr = f.read(256)
    assert hdr[:8] == b"FROGIDX1"
    assert struct.unpack_from("<I", hdr, 8)[0] == 1
    assert (ix.n, ix.d, ix.d_pad, ix.H, ix.m) == (10_000, 32, 32, 8, 16)
    assert os.path.getsize(path) == struct.unpack_from("<Q", hdr, 104)[0]
    # Sec. 4: ranks by ascending attribute; rank2id is a permutation; vectors in rank order
    assert np.all(np.diff(ix.sorted_attr) >= 0)
    r2i = np.asarray(ix.rank2id)
    assert np.array_equal(np.sort(r2i), np.arange(ix.n))
    assert np.array_equal(wl.attrs[r2i], ix.sorted_attr)
    assert np.array_equal(wl.vectors[r2i], ix.vectors[:, : ix.d])


def test_enc_rows_stay_inside_their_segment(tiny):
    _, _, ix = tiny
    enc = np.asarray(ix.enc)
    BOT = 0xFFFFFFFF
    for h in range(ix.H):
        seg = np.array([oracle.segment_at(ix.n, h, u) for u in range(0, ix.n, 7)])
        rows = enc[::7, h, :]
        valid = rows != BOT
        assert np.all((rows >= seg[:, :1]) | ~valid) and np.all((rows <= seg[:, 1:]) | ~valid)
        assert not np.any(rows == np.arange(0, ix.n, 7)[:, None])        # never itself
        for r in rows[:200]:
            v = r[r != BOT]
            assert len(set(v.tolist())) == v.size                        # no repeats in a row
            assert np.all(r[v.size:] == BOT)                             # empties only at the tail
    assert (enc != BOT).mean() > 0.99


def test_leaf_rows_are_ordered_by_fusion_distance(tiny, libs):
    _, _, ix = tiny
    V = np.asarray(ix.vectors, dtype=np.float64)
    h = ix.H - 1
    for u in range(0, ix.n, 503):
        row = np.asarray(ix.enc[u, h])
        row = row[row != 0xFFFFFFFF]
        dv = np.sqrt(((V[row] - V[u]) ** 2).sum(1))
        da = np.abs(row.astype(np.int64) - u) / (ix.n - 1)
        df = [libs.fusion_distance(a, b, 0.2, 0.5) for a, b in zip(dv, da)]
        assert np.all(np.diff(df) >= -1e-9)
        # the fusion-nearest object of the leaf is always kept (first pick of the selection rule)
        L, R = oracle.segment_at(ix.n, h, u)
        others = np.array([v for v in range(L, R + 1) if v != u])
        dv_all = np.sqrt(((V[others] - V[u]) ** 2).sum(1))
        df_all = dv_all * (1 - 0.2 * (1 - (np.abs(others - u) / (ix.n - 1)) ** 0.5))
        assert row[0] == others[np.argmin(df_all)]


def test_boundary_effect_closed_form(libs, cache_dir):
    """Eq. 1 and its average (l+1)/3: with beta -> 0 and attributes independent of the vectors,
    the rank distance from an object to its leaf ENCs averages (l+1)/3 over positions and about
    l/2 for an object on the leaf boundary."""
    rng = np.random.default_rng(1)
    n, d = 4096, 8
    V = rng.standard_normal((n, d)).astype(np.float32)
    a = rng.permutation(n).astype(np.int32)
    path = os.path.join(cache_dir, "eq1.idx")
    libs.build_index(V, a, path, m=4, ef_c=32, n_inv=6, beta=1e-9)
    ix = oracle.load_index(path)
    h = ix.H - 1
    L, R = oracle.segment_at(ix.n, h, 0)
    ell = R - L + 1
    assert ell == 64
    rows = np.asarray(ix.enc[:, h, :]).astype(np.int64)
    dist = np.abs(rows - np.arange(n)[:, None])
    assert dist.mean() == pytest.approx((ell + 1) / 3, rel=0.04)
    edge = dist[np.arange(n) % ell == 0]
    assert edge.mean() == pytest.approx(ell / 2, rel=0.08)


def test_build_is_thread_count_independent(libs, cache_dir):
    wl = datagen.make_workload("tiny", n=3000, nq=4)
    p1 = os.path.join(cache_dir, "t1.idx")
    p4 = os.path.join(cache_dir, "t4.idx")
    libs.build_index(wl.vectors, wl.attrs, p1, threads=1)
    libs.build_index(wl.vectors, wl.attrs, p4, threads=4)
    with open(p1, "rb") as f1, open(p4, "rb") as f4:
        assert f1.read() == f4.read()


def test_builder_rejects_bad_arguments(libs, cache_dir):
    V = np.zeros((10, 4), np.float32)
    a = np.arange(10, dtype=np.int32)
    with pytest.raises(libs.FrogError):
        libs.build_index(V, a, os.path.join(cache_dir, "no_such_dir", "x.idx"))
    with pytest.raises(libs.FrogError):
        libs.build_index(V, a, os.path.join(cache_dir, "x.idx"), m=4, ef_c=2)


def test_odd_dimension_is_zero_padded(libs, cache_dir):
    rng = np.random.default_rng(2)
    V = rng.standard_normal((500, 10)).astype(np.float32)
    a = rng.integers(0, 50, 500).astype(np.int32)
    path = os.path.join(cache_dir, "odd.idx")
    libs.build_index(V, a, path, n_inv=5)
    ix = oracle.load_index(path)
    assert (ix.d, ix.d_pad) == (10, 12)
    assert np.all(ix.vectors[:, 10:] == 0)
    Q = rng.standard_normal((20, 10)).astype(np.float32)
    lo = np.full(20, 0, np.int32)
    hi = np.full(20, 49, np.int32)
    res = oracle.search(ix, Q, lo, hi, 5, 32)
    gt, _, _ = oracle.exact_slab(ix, Q, lo, hi, 5)
    assert oracle.recall(res.ids, gt) > 0.8
