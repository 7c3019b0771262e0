"""Pins for the partition oracle: brute force, Otsu identities, closed forms, cover."""
from fractions import Fraction

import numpy as np
import pytest

import gen
import oracle
from oracle import partitioner as P


def _brute_cut(q_sorted, R_node, m_min, m_max):
    """All cuts, between-class variance omega_f omega_c (mu_f - mu_c)^2 in exact rationals and
    the allocation by scanning every r."""
    n = len(q_sorted)
    best = None
    for p in range(1, n):
        if q_sorted[p - 1] == q_sorted[p]:
            continue
        c, f = q_sorted[:p], q_sorted[p:]
        n_c, n_f = len(c), len(f)
        r_f = min(range(1, R_node), key=lambda r: (abs(Fraction(r) - Fraction(R_node * n_f, n)), r))
        r_c = R_node - r_f
        if not (m_min * r_f <= n_f <= m_max * r_f and m_min * r_c <= n_c <= m_max * r_c):
            continue
        var_b = Fraction(n_f, n) * Fraction(n_c, n) * (Fraction(sum(f), n_f) - Fraction(sum(c), n_c)) ** 2
        if best is None or var_b > best[0]:
            best = (var_b, p, r_f)
    return None if best is None else (best[1], best[2])


def test_allocate_matches_full_scan_and_closed_forms():
    for R in range(2, 12):
        for n_f in range(1, 30):
            for n_c in range(1, 30):
                n = n_f + n_c
                ref = min(range(1, R), key=lambda r: (abs(Fraction(r) - Fraction(R * n_f, n)), r))
                assert P.allocate(n_f, n_c, R) == ref
    assert P.allocate(5, 90, 2) == 1 and P.allocate(90, 5, 2) == 1
    for R in (2, 4, 8, 64):
        assert P.allocate(17, 17, R) == R // 2


def test_best_cut_against_brute_force():
    rng = np.random.default_rng(0)
    for trial in range(200):
        n = int(rng.integers(2, 33))
        q = sorted(int(v) for v in rng.integers(0, 40 if trial % 2 else 65536, size=n))
        R_node = int(rng.integers(2, min(n, 6) + 1))
        m_min = int(rng.integers(1, 3))
        m_max = int(rng.integers(4, 40))
        assert P.best_cut(q, R_node, m_min, m_max) == _brute_cut(q, R_node, m_min, m_max)


def test_variance_decomposition_at_the_chosen_threshold():
    rng = np.random.default_rng(1)
    q = sorted(int(v) for v in rng.integers(0, 65536, size=40))
    p, _ = P.best_cut(q, 2, 1, 40)
    c, f = np.array(q[:p], float), np.array(q[p:], float)
    n = len(q)
    w_c, w_f = len(c) / n, len(f) / n
    var_b = w_c * w_f * (f.mean() - c.mean()) ** 2
    var_w = w_c * c.var() + w_f * f.var()
    assert np.isclose(np.var(np.array(q, float)), var_b + var_w, rtol=1e-12)
    # and it is the maximiser over every threshold
    for pp in range(1, n):
        cc, ff = np.array(q[:pp], float), np.array(q[pp:], float)
        vb = len(cc) * len(ff) / n ** 2 * (ff.mean() - cc.mean()) ** 2
        assert vb <= var_b * (1 + 1e-12)


def test_textbook_otsu_on_8bit_histogram():
    """Histogram Otsu (class probabilities and means from a 256-bin histogram), restated in
    numpy, picks the same threshold on data that already sits on 256 levels."""
    rng = np.random.default_rng(2)
    for _ in range(20):
        vals = np.concatenate([rng.normal(60, 15, 70), rng.normal(170, 25, 50)]).clip(0, 255).round()
        vals[0], vals[1] = 0, 255
        S = (vals / 255.0).astype(np.float32)
        q = P.quantise(S)
        assert np.array_equal(q, (vals * 257).astype(np.int64))      # exact 16-bit images of 8-bit levels
        qs = sorted(int(v) for v in q)
        p, _ = P.best_cut(qs, 2, 1, len(qs))
        theta = qs[p] // 257
        hist = np.bincount(vals.astype(int), minlength=256).astype(float)
        prob = hist / hist.sum()
        lv = np.arange(256)
        best_t, best_v = None, -1.0
        for t in range(1, 256):           # focus = level >= t
            w1, w0 = prob[t:].sum(), prob[:t].sum()
            if w0 == 0 or w1 == 0:
                continue
            m1, m0 = (prob[t:] * lv[t:]).sum() / w1, (prob[:t] * lv[:t]).sum() / w0
            v = w0 * w1 * (m1 - m0) ** 2
            if v > best_v * (1 + 1e-12):
                best_t, best_v = t, v
        # histogram thresholds between two occupied levels are equivalent; compare the split
        assert (vals >= best_t).sum() == (vals >= theta).sum()


def test_two_level_map_splits_at_the_level_change():
    S = np.zeros(24, np.float32)
    hot = [1, 2, 3, 10, 11, 17, 18, 19, 20, 23]
    S[hot] = 1.0
    lab = P.partition_request(S, 2)
    assert set(np.nonzero(lab == lab[1])[0]) == set(hot)
    assert lab[0] == 0 and lab[1] == 1     # numbered by smallest token index


@pytest.mark.parametrize("name", ["image_small", "mmdit_small", "video_small"])
def test_cover_count_bounds(name):
    wl = gen.workload(name)
    amap = gen.saliency_map(wl, 7)
    labels, sizes = oracle.partition(amap, None, wl.R, wl.m_min, wl.m_max)
    assert labels.shape == (wl.B, wl.n_grid)
    assert labels.min() == 0 and labels.max() == wl.R - 1
    for b in range(wl.B):
        cnt = np.bincount(labels[b], minlength=wl.R)
        assert np.array_equal(cnt, sizes[b])
        assert cnt.sum() == wl.n_grid and (cnt > 0).all()          # every token once, R regions
        first = [np.nonzero(labels[b] == r)[0][0] for r in range(wl.R)]
        assert first == sorted(first)


def test_size_bounds_hold_without_fallback_on_image_map():
    wl = gen.workload("image").replace(B=1)
    amap = gen.saliency_map(wl, 3)
    labels, sizes = oracle.partition(amap, None, wl.R, wl.m_min, wl.m_max)
    assert sizes.min() >= wl.m_min and sizes.max() <= wl.m_max
    assert (sizes > 0).all() and sizes.sum() == wl.n_grid


def test_constant_map_falls_back_to_equal_chunks():
    lab = P.partition_request(np.full(10, 0.3, np.float32), 3)
    assert lab.tolist() == [0, 0, 0, 0, 1, 1, 1, 2, 2, 2]
    lab = P.partition_request(np.arange(7, dtype=np.float32), 7)
    assert sorted(lab.tolist()) == list(range(7))


def test_saliency_mean_and_column_permutation():
    rng = np.random.default_rng(3)
    amap = (rng.integers(0, 256, size=(1, 48, 6)) / 256.0).astype(np.float32)   # exact in fp32
    cols = np.array([4, 1, 5], np.int32)
    s = P.saliency(amap[0], cols)
    np.testing.assert_array_equal(s, amap[0][:, [1, 4, 5]].astype(np.float64).mean(1).astype(np.float32))
    a, _ = oracle.partition(amap, cols, 6)
    b, _ = oracle.partition(amap, cols[::-1].copy(), 6)
    assert np.array_equal(a, b)
    c, _ = oracle.partition(amap[:, :, [1, 4, 5]].copy(), None, 6)
    assert np.array_equal(a, c)


def test_affine_change_of_the_map_keeps_the_partition():
    rng = np.random.default_rng(4)
    S = (rng.integers(0, 1024, size=64) / 1024.0).astype(np.float32)
    a = P.partition_request(S, 5)
    b = P.partition_request((S * np.float32(4.0) + np.float32(8.0)).astype(np.float32), 5)
    assert np.array_equal(a, b)


def test_hand_worked_three_region_cases_pin_which_side_gets_r_f():
    """Sec. 4.1 allocation rule worked by hand: the FOCUS side (saliency >= threshold) hosts
    r_f = argmin_r |r - R n_f / (n_f + n_c)| regions, the context side the rest.

    Case 1: saliency 0,0,0,0,1,1 and R = 3.  The only threshold separates {4,5} (focus, n_f = 2) from {0..3}
    (context, n_c = 4); R n_f / n = 1, so r_f = 1 and r_c = 2: the focus stays whole, the context (all values equal,
    no further threshold) is chopped in index order into {0,1} and {2,3}.  Giving r_f to the wrong side would keep
    the context whole and split the focus instead.
    Case 2: five tokens at 0, then 0.9, 1.0, 0.9, 1.0 and R = 3.  Otsu separates the zeros (n_c = 5) from the rest
    (n_f = 4); R n_f / n = 4/3, so r_f = 1 (distance 1/3 against 2/3 for r = 2) and r_c = 2: focus {5,6,7,8} is one
    region, the zeros are chopped into {0,1,2} and {3,4}.  The wrong side would give {0..4}, {5,7}, {6,8}.
    Case 3: the mirror image of case 1 with the large side in focus: saliency 1,1,1,1,0,0 gives n_f = 4, n_c = 2,
    R n_f / n = 2, r_f = 2: the focus is chopped into {0,1}, {2,3} and the context {4,5} stays whole."""
    def run(values, R):
        S = np.asarray(values, np.float32)
        lab, sizes = oracle.partition(S.reshape(1, -1, 1), None, R)
        return lab[0].tolist(), sizes[0].tolist()

    assert run([0, 0, 0, 0, 1, 1], 3) == ([0, 0, 1, 1, 2, 2], [2, 2, 2])
    assert run([0, 0, 0, 0, 0, 0.9, 1.0, 0.9, 1.0], 3) == ([0, 0, 0, 1, 1, 2, 2, 2, 2], [3, 2, 4])
    assert run([1, 1, 1, 1, 0, 0], 3) == ([0, 0, 1, 1, 2, 2], [2, 2, 2])
    # the same rule one level down: 12 tokens, two loud ones, R = 4 -> r_f = argmin |r - 4*2/12| = 1
    lab, sizes = run([0] * 10 + [1, 1], 4)
    assert lab == [0, 0, 0, 0, 1, 1, 1, 2, 2, 2, 3, 3] and sizes == [4, 3, 3, 2]
