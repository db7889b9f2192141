"""frog_search_static: the search entry point for callers that may not allocate device memory
(stream capture, fixed memory budgets, a foreign caching allocator owning the free memory).

Its scratch is a fixed device array inside the library instead of buffers owned by the index.  The
check: it returns what the CPU oracle computes for the same index (and therefore what the regular
entry point returns) -- twice in a row, since the array keeps the previous call's contents and a stale
counter or stale visited bits would show up on the second call -- and the device's free-memory reading
is the same before and after a call once the first call has done its one-time set-up.  Collected last
so that a failure here cannot hide other results."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _run(libs, n, nq, beam, budget):
    import os
    import tempfile

    import datagen
    import oracle

    wl = datagen.make_workload("sift", n=n, nq=nq)
    with tempfile.TemporaryDirectory() as tmp:
        path = os.path.join(tmp, "static.idx")
        libs.build_index(wl.vectors, wl.attrs, path, seed=wl.seed)
        ix = libs.Index.load(path, 0)
        ref = oracle.search(oracle.load_index(path), wl.queries, wl.lo, wl.hi, wl.k, beam, B=budget)
    q = torch.from_numpy(wl.queries).cuda()
    lo = torch.from_numpy(wl.lo).cuda()
    hi = torch.from_numpy(wl.hi).cuda()
    prm = libs.Params(budget=budget)
    # the regular entry point agrees with the oracle too (it allocates its scratch on first use)
    reg_ids, reg_d = ix.search(q, lo, hi, wl.k, beam, params=prm)
    torch.cuda.synchronize()
    assert np.array_equal(reg_ids.cpu().numpy(), ref.ids)
    out_ids = torch.empty((nq, wl.k), dtype=torch.int32, device="cuda")
    out_d = torch.empty((nq, wl.k), dtype=torch.float32, device="cuda")
    fin = np.isfinite(ref.dists)
    for call in range(3):
        out_ids.fill_(-7)
        out_d.fill_(-7.0)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        ix.search_static(q, lo, hi, wl.k, beam, out_ids=out_ids, out_dists=out_d, params=prm)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        if call > 0:
            # nothing was allocated (or freed) on the device by the call; the first call on a device may
            # load the library's module and is not held to this
            assert free_after == free_before, f"free device memory changed across call {call}"
        assert np.array_equal(out_ids.cpu().numpy(), ref.ids), f"ids differ from the oracle on call {call}"
        got = out_d.cpu().numpy()
        assert np.array_equal(np.isfinite(got), fin)
        assert np.allclose(got[fin], ref.dists[fin], rtol=1e-4, atol=0), f"distances differ on call {call}"
    return ix


def test_static_scratch_entry_point_matches_regular_search(libs):
    ix = _run(libs, n=30_000, nq=500, beam=48, budget=16)
    # a second index of another size reuses the same array right after
    ix2 = _run(libs, n=12_345, nq=300, beam=32, budget=32)
    ix.close()
    ix2.close()


def test_static_scratch_rejects_what_does_not_fit(libs):
    import ctypes

    # argument errors are reported before anything touches the device array
    rc = libs._lib.frog_search_static(None, None, None, None, 1, 1, 1, None, None, None, None)
    assert rc == 1
    # an index beyond the stated maximum is refused with its own error code; a header-only fake of
    # that size is enough because the size check comes first
    n_big = 2_097_152 + 1
    shape = libs.IndexInfo(n=n_big, d=4, d_pad=4, H=1, m=1)
    a = np.zeros(n_big, dtype=np.int32)
    v = np.zeros((n_big, 4), dtype=np.float32)
    e = np.full((n_big, 1), 0xFFFFFFFF, dtype=np.uint32)
    h = ctypes.c_void_p()
    rc = libs._lib.frog_index_from_host(a.ctypes.data_as(ctypes.c_void_p), a.ctypes.data_as(ctypes.c_void_p),
                                        v.ctypes.data_as(ctypes.c_void_p), e.ctypes.data_as(ctypes.c_void_p),
                                        ctypes.byref(shape), 0, ctypes.byref(h))
    assert rc == 0
    big = libs.Index(h)
    q = torch.zeros((4, 4), dtype=torch.float32, device="cuda")
    lo = torch.zeros(4, dtype=torch.int32, device="cuda")
    hi = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(libs.FrogError) as err:
        big.search_static(q, lo, hi, 1, 16)
    assert err.value.code == 7 and "too large" in str(err.value)
    big.close()
