"""Pins of the batch-former oracle (Sec. 4.3: patch monotasks, least-maximum-load packing) against things
it does not compute itself: closed forms, brute force over all assignments / subsets, the classical
list-scheduling bounds, and hand-worked examples of the tie-breaking."""
import itertools

import numpy as np
import pytest

from oracle import scheduler as sch


def _opt_makespan(load, cost):
    G = len(load)
    best = np.inf
    for a in itertools.product(range(G), repeat=len(cost)):
        L = list(load)
        for j, g in enumerate(a):
            L[g] += cost[j]
        best = min(best, max(L))
    return best


def test_pack_hand_examples():
    # loads 5,1,3 and a monotask of cost 2: going to device 0 makes the straggler 7, anywhere else it stays 5
    a, L = sch.pack([5, 1, 3], [2], [0])
    assert a.tolist() == [1] and L.tolist() == [5, 3, 3]                # home 0 is not a minimiser -> least loaded
    a, L = sch.pack([5, 1, 3], [1], [2])
    assert a.tolist() == [2] and L.tolist() == [5, 1, 4]                # home 2 ties with 1 -> locality wins
    a, L = sch.pack([5, 1, 3], [1], [-1])
    assert a.tolist() == [1]                                            # warm-up task: least loaded device
    a, L = sch.pack([2, 2, 2], [1, 1, 1, 1], [-1, -1, -1, -1])
    assert a.tolist() == [0, 1, 2, 0]                                   # equal loads -> smallest index
    a, L = sch.pack([4, 1], [3, 3], [0, 1])
    assert a.tolist() == [1, 1] and L.tolist() == [4, 7]                # 2nd: both give 7, home 1 wins over index 0
    a, L = sch.pack([0.0], [1.5, 2.5], [-1, 0])
    assert a.tolist() == [0, 0] and L.tolist() == [4.0]


def test_pack_objective_closed_form_and_bounds():
    g = np.random.default_rng(0)
    for trial in range(60):
        G = int(g.integers(1, 4))
        n = int(g.integers(1, 8))
        load = g.integers(0, 6, size=G).astype(float)
        cost = g.integers(1, 9, size=n).astype(float)
        home = g.integers(-1, G, size=n)
        a, L = sch.pack(load, cost, home)
        # every single decision attains min_g max(...) = max(max L, min L + w)
        cur = load.copy()
        for j in range(n):
            want = max(cur.max(), cur.min() + cost[j])
            cur[a[j]] += cost[j]
            assert cur.max() == want
        assert np.array_equal(cur, L)
        # Graham's list-scheduling bound against the brute-force optimum (empty start only)
        a0, L0 = sch.pack(np.zeros(G), cost, home)
        opt = _opt_makespan([0.0] * G, list(cost))
        assert L0.max() <= (2.0 - 1.0 / G) * opt + 1e-12
        # longest-first order: the 4/3 - 1/(3G) bound
        srt = np.sort(cost)[::-1]
        a1, L1 = sch.pack(np.zeros(G), srt, [-1] * n)
        assert L1.max() <= (4.0 / 3.0 - 1.0 / (3.0 * G)) * opt + 1e-12
        assert abs(L0.sum() - cost.sum()) < 1e-9


def test_pack_equal_costs_balance_and_locality_only_breaks_ties():
    a, L = sch.pack(np.zeros(4), np.ones(10), [-1] * 10)
    assert sorted(L.tolist()) == [2, 2, 3, 3]
    # a home that is strictly worse than another device is never used
    g = np.random.default_rng(1)
    for _ in range(50):
        load = g.integers(0, 10, size=3).astype(float)
        w = float(g.integers(1, 5))
        h = int(g.integers(0, 3))
        a, _ = sch.pack(load, [w], [h])
        worst_h = max(load.max(), load[h] + w)
        worst_a = max(load.max(), load[a[0]] + w)
        assert worst_a <= worst_h
        if worst_h == max(load.max(), load.min() + w):
            assert a[0] == h


def _lex_max_feasible(order, tokens, resident, budget, free_slots):
    """Brute force: among all feasible subsets the one whose indicator, read in priority order, is greatest."""
    n = len(order)
    best = None
    for bits in itertools.product((1, 0), repeat=n):        # descending lexicographic order of the indicator
        S = [order[k] for k in range(n) if bits[k]]
        if sum(tokens[i] for i in S) > budget:
            continue
        if sum(1 for i in S if not resident[i]) > free_slots:
            continue
        if any(tokens[i] == 0 and not resident[i] for i in S):
            continue
        best = S
        break
    return set(best)


def test_form_batch_hand_example():
    #          prio arrival tokens resident
    reqs = [(1, 0, 600, 1),     # resident, low priority
            (5, 3, 700, 0),     # urgent newcomer
            (5, 1, 500, 1),     # urgent, earlier arrival -> first
            (3, 2, 100, 0)]     # fits into the leftover but no slot is free after request 1 took it
    p, a, t, r = (list(c) for c in zip(*reqs))
    chosen, res = sch.form_batch(p, a, t, r, token_budget=1300, max_resident=3)
    assert chosen.tolist() == [0, 1, 1, 0] and res.tolist() == [1, 1, 1, 0]
    chosen, res = sch.form_batch(p, a, t, r, token_budget=1300, max_resident=4)
    assert chosen.tolist() == [0, 1, 1, 1] and res.tolist() == [1, 1, 1, 1]      # 500 + 700 + 100
    chosen, res = sch.form_batch(p, a, t, r, token_budget=1100, max_resident=4)
    assert chosen.tolist() == [0, 0, 1, 1] and res.tolist() == [1, 0, 1, 1]      # 700 does not fit after 500; 100 does
    # no free slot: the newcomers wait and the low-priority resident request uses the leftover
    chosen, res = sch.form_batch(p, a, t, r, token_budget=1100, max_resident=2)
    assert chosen.tolist() == [1, 0, 1, 0] and res.tolist() == [1, 0, 1, 0]
    # a request with nothing active runs (a pure cached-drift update) only if its state is resident
    chosen, res = sch.form_batch([2, 2], [0, 1], [0, 0], [1, 0], token_budget=0, max_resident=2)
    assert chosen.tolist() == [1, 0] and res.tolist() == [1, 0]


def test_form_batch_is_the_lexicographic_maximum_over_feasible_sets():
    g = np.random.default_rng(3)
    for _ in range(200):
        n = int(g.integers(1, 8))
        prio = g.integers(0, 3, size=n)
        arr = g.permutation(n)
        tok = g.integers(0, 6, size=n) * 100
        res = g.integers(0, 2, size=n)
        max_res = int(res.sum() + g.integers(0, 3))
        budget = int(g.integers(0, 12)) * 100
        chosen, res_after = sch.form_batch(prio, arr, tok, res, budget, max_res)
        order = sorted(range(n), key=lambda i: (-prio[i], arr[i], i))
        want = _lex_max_feasible(order, tok, res, budget, max_res - int(res.sum()))
        assert set(np.nonzero(chosen)[0].tolist()) == want
        assert int(tok[chosen.astype(bool)].sum()) <= budget
        assert int(res_after.sum()) <= max(max_res, int(res.sum()))
        assert np.array_equal(res_after, res | (chosen & (1 - res)).astype(res.dtype))


def _run_search(f, lo, hi, start, limit=200):
    s = sch.RSearch(lo, hi, start)
    r, evals = start, 0
    while not s.converged and evals < limit:
        r = s.update(f(r))
        evals += 1
    return s.accepted, evals


def test_rsearch_finds_the_peak_of_every_small_unimodal_profile():
    """Brute force: every strictly unimodal profile on ranges up to 9 values (all peak positions, random slopes),
    every starting point: the search ends on the arg max within a bounded number of observations."""
    g = np.random.default_rng(7)
    for n in range(1, 10):
        for peak in range(n):
            for trial in range(6):
                up = np.sort(g.random(peak))
                down = np.sort(g.random(n - peak - 1))[::-1]
                prof = np.concatenate([up, [2.0], down]) + np.arange(n) * 0          # strictly unimodal, peak value 2
                for start in range(n):
                    got, evals = _run_search(lambda r: prof[r - 4], 4, 4 + n - 1, 4 + start)
                    assert got == 4 + peak, (prof, start)
                    assert evals <= 4 * int(np.ceil(np.log2(n + 1))) + 6


def test_rsearch_is_logarithmic_on_large_ranges_and_hand_example():
    for lo, hi in ((1, 64), (2, 257), (8, 1024)):
        for peak in (lo, hi, (lo + hi) // 2, lo + 5, hi - 3):
            f = lambda r: -abs(r - peak)
            for start in (lo, hi, (lo + 3 * hi) // 4):
                got, evals = _run_search(f, lo, hi, start, limit=500)
                assert got == peak
                assert evals <= 4 * int(np.ceil(np.log2(hi - lo + 1))) + 6
    # hand-worked: range 1..16, start 4, peak at 11, f = -|r - 11|; initial step 8
    s = sch.RSearch(1, 16, 4)
    seq = [4]
    while not s.converged:
        seq.append(s.update(-abs(seq[-1] - 11)))
    # 4 (ref -7) -> 12 (-1, accepted) -> 16 (clamped 20; -5 worse: flip, step 4) -> 8 (-3 worse: flip, step 2)
    # -> 14 (-3 worse: flip, step 1) -> 11 (0, accepted) -> 10 (worse: flip, 1st failure at step 1) -> 12 (worse: 2nd) -> stop
    assert seq == [4, 12, 16, 8, 14, 11, 10, 12, 11]
    assert s.accepted == 11
    # a single admissible value needs no search
    s = sch.RSearch(5, 5, 5)
    assert s.converged and s.update(1.0) == 5
