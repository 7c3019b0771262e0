"""The library's host-side batch former (Sec. 4.3) against the oracle, bit for bit, on random and edge inputs.
Pure host code: runs without a GPU."""
import ctypes

import numpy as np
import pytest

import paper_2607_12121_b200 as fd
from oracle import scheduler as sch


@pytest.mark.parametrize("seed", range(6))
def test_pack_matches_oracle(seed):
    g = np.random.default_rng(seed)
    for _ in range(40):
        G = int(g.integers(1, 9))
        n = int(g.integers(0, 65))
        # integer-valued and fractional costs; many ties when the values are small integers
        load = g.integers(0, 5, size=G).astype(np.float64) if seed % 2 else g.uniform(0, 4, size=G)
        cost = g.integers(0, 6, size=n).astype(np.float64) if seed % 2 else g.uniform(0, 3, size=n)
        home = g.integers(-1, G, size=n).astype(np.int32)
        want_a, want_l = sch.pack(load, cost, home)
        got_l = load.copy()
        got_a = fd.fd_sched_pack(got_l, cost, home)
        assert np.array_equal(got_a, want_a)
        assert np.array_equal(got_l, want_l)


def test_pack_workload_shape():
    """The serving shape of the paper's evaluation: 8 devices, requests with 8-32 patch monotasks whose costs are
    their token counts; patches of a request prefer the device that holds the request's first patch."""
    g = np.random.default_rng(11)
    load = np.zeros(8)
    ref = load.copy()
    for req in range(40):
        R = int(g.choice([8, 16, 32]))
        cost = g.integers(16, 513, size=R).astype(np.float64)
        first = fd.fd_sched_pack(load, cost[:1], np.array([-1], np.int32))
        rest = fd.fd_sched_pack(load, cost[1:], np.full(R - 1, first[0], np.int32))
        a0, ref = sch.pack(ref, cost[:1], [-1])
        a1, ref = sch.pack(ref, cost[1:], [int(a0[0])] * (R - 1))
        assert np.array_equal(first, a0) and np.array_equal(rest, a1)
    assert np.array_equal(load, ref)
    assert load.max() - load.min() <= 512                         # never further apart than one monotask


@pytest.mark.parametrize("seed", range(4))
def test_form_batch_matches_oracle(seed):
    g = np.random.default_rng(100 + seed)
    for _ in range(60):
        n = int(g.integers(0, 40))
        prio = g.integers(0, 4, size=n).astype(np.int32)
        arr = g.integers(0, 10, size=n).astype(np.int64)          # repeated arrival numbers: the index decides
        tok = (g.integers(0, 9, size=n) * 128).astype(np.int32)
        res = (g.random(n) < 0.4).astype(np.uint8)
        max_res = int(res.sum()) + int(g.integers(0, 4)) - int(g.integers(0, 2))
        max_res = max(max_res, 0)
        budget = int(g.integers(0, 40)) * 128
        want_c, want_r = sch.form_batch(prio, arr, tok, res, budget, max_res)
        got_r = res.copy()
        got_c = fd.fd_sched_form_batch(prio, arr, tok, got_r, budget, max_res)
        assert np.array_equal(got_c, want_c)
        assert np.array_equal(got_r, want_r)


def test_invalid_arguments_are_refused_and_nothing_is_written():
    load = np.array([1.0, 2.0])
    with pytest.raises(fd.FlashDiffError):
        fd.fd_sched_pack(load, [1.0], [2])                         # home out of range
    with pytest.raises(fd.FlashDiffError):
        fd.fd_sched_pack(load, [-1.0], [0])
    with pytest.raises(fd.FlashDiffError):
        fd.fd_sched_pack(load, [np.nan], [0])
    with pytest.raises(fd.FlashDiffError):
        fd.fd_sched_pack(np.array([np.inf]), [1.0], [0])
    assert load.tolist() == [1.0, 2.0]
    assert fd.lib.fd_sched_pack(0, None, 0, None, None, None) == fd.FD_ERR_INVALID_ARG
    res = np.zeros(2, np.uint8)
    with pytest.raises(fd.FlashDiffError):
        fd.fd_sched_form_batch([0, 0], [0, 1], [5, -1], res, 10, 2)
    with pytest.raises(fd.FlashDiffError):
        fd.fd_sched_form_batch([0, 0], [0, 1], [5, 1], res, -1, 2)
    assert res.tolist() == [0, 0]
    assert fd.lib.fd_sched_form_batch(0, None, None, None, None, ctypes.c_int64(0), 0, None) == fd.FD_OK


def test_batch_former_drives_a_step_mask():
    """The chosen requests keep their gate mask, the others get an all-zero mask for this step (they wait at the
    step boundary); the active-token total of the formed step never exceeds the budget."""
    g = np.random.default_rng(5)
    B, R = 8, 16
    sizes = g.integers(16, 129, size=(B, R))
    gate = (g.random((B, R)) < 0.5).astype(np.uint8)
    tok = (sizes * gate).sum(1).astype(np.int32)
    res = np.ones(B, np.uint8)
    chosen = fd.fd_sched_form_batch(g.integers(0, 3, size=B), np.arange(B), tok, res, int(tok.sum() // 2), B)
    step_mask = gate * chosen[:, None]
    assert (sizes * step_mask).sum() <= tok.sum() // 2
    assert chosen.any() and not chosen.all()


def test_rsearch_matches_oracle_step_by_step():
    g = np.random.default_rng(21)
    for _ in range(300):
        lo = int(g.integers(1, 20))
        hi = lo + int(g.integers(0, 200))
        start = int(g.integers(lo, hi + 1))
        kind = int(g.integers(0, 3))
        peak = int(g.integers(lo, hi + 1))
        noise = g.random(hi - lo + 1) * (0.0 if kind == 0 else 3.0)           # kind 0: unimodal; else: noisy profiles
        flat = kind == 2                                                      # plateaus: ties count as "not better"
        f = lambda r: (-(abs(r - peak) // 4) if flat else -abs(r - peak)) + noise[r - lo]
        ref = sch.RSearch(lo, hi, start)
        st = fd.fd_rsearch_init(lo, hi, start)
        r = start
        for it in range(400):
            want = ref.update(f(r))
            got = fd.fd_rsearch_update(st, f(r))
            assert got == want, (lo, hi, start, it)
            assert (st.accepted, st.step, st.dir, bool(st.converged)) == (ref.accepted, ref.step, ref.dir, ref.converged)
            r = got
            if ref.converged:
                break
        assert ref.converged
        if kind == 0:
            assert st.accepted == peak


def test_rsearch_invalid_arguments():
    with pytest.raises(fd.FlashDiffError):
        fd.fd_rsearch_init(0, 8, 4)
    with pytest.raises(fd.FlashDiffError):
        fd.fd_rsearch_init(4, 3, 4)
    with pytest.raises(fd.FlashDiffError):
        fd.fd_rsearch_init(2, 8, 9)
    st = fd.fd_rsearch_init(2, 8, 4)
    with pytest.raises(fd.FlashDiffError):
        fd.fd_rsearch_update(st, float("nan"))
    assert st.accepted == 4 and not st.have_ref
