"""Pins for the gate and compaction oracle: identities and closed forms the paper fixes."""
import numpy as np

import gen
import oracle

WL = gen.workload("audio_small")


def _draw(seed=1, fractions=None, wl=WL):
    labels = gen.uniform_labels(wl)
    fr = gen.request_fractions(wl, seed) if fractions is None else fractions
    lat = gen.latent_pair(wl, seed, labels, fractions=fr)
    return labels, lat


def test_weights_sum_to_one_and_threshold_rule():
    labels, lat = _draw()
    st = oracle.initial_state(WL.B, WL.R)
    score, weight, mask = oracle.activity_gate(lat["z_cur"], lat["z_prev"], labels, lat["eps"], st, WL.R)
    np.testing.assert_allclose(weight.astype(np.float64).sum(1), 1.0, rtol=1e-6)
    # skipped iff w < eps (no forcing on a fresh state)
    assert np.array_equal(mask, (weight.astype(np.float64) >= lat["eps"][:, None]).astype(np.uint8))
    # the generator's gap makes the active count equal the requested one, with margin
    assert np.array_equal(mask.sum(1), lat["n_loud"])
    rel = np.abs(weight / lat["eps"][:, None] - 1.0)
    assert rel.min() >= 1e-3


def test_rms_of_constant_change_and_equal_weights():
    wl = WL.replace(R=16)                 # 1/16 is exact in fp32: the boundary w == eps is hit exactly
    labels = gen.uniform_labels(wl)
    z = np.random.default_rng(0).standard_normal((wl.B, wl.N, wl.D)).astype(np.float32)
    c = np.float32(0.25)
    st = oracle.initial_state(wl.B, wl.R)
    eps = np.full(wl.B, 1.0 / wl.R, np.float32)        # w_i = 1/R >= eps -> all active
    score, weight, mask = oracle.activity_gate(z + c, z, labels, eps, st, wl.R, eta=0.0)
    assert np.all(score == c)
    assert np.all(weight == np.float32(1.0 / wl.R))
    assert mask.all()
    st = oracle.initial_state(wl.B, wl.R)
    eps = np.full(wl.B, 1.01 / wl.R, np.float32)       # just above 1/R -> all skipped
    _, _, mask = oracle.activity_gate(z + c, z, labels, eps, st, wl.R, eta=0.0)
    assert not mask.any()


def test_rms_against_direct_numpy_and_sign_of_difference():
    labels, lat = _draw(seed=4)
    st = oracle.initial_state(WL.B, WL.R)
    score, _, _ = oracle.activity_gate(lat["z_cur"], lat["z_prev"], labels, lat["eps"], st, WL.R)
    d = (lat["z_cur"].astype(np.float64) - lat["z_prev"].astype(np.float64)) ** 2
    seg = WL.N // WL.R
    ref = np.sqrt(d.reshape(WL.B, WL.R, seg * WL.D).mean(-1))
    np.testing.assert_allclose(score, ref, rtol=1e-6)
    # the measured change tracks the generator's noise scale
    np.testing.assert_allclose(score, lat["sigma"], rtol=0.2)


def test_eps_zero_activates_everything_and_eps_is_monotone():
    labels, lat = _draw(seed=6)
    prev = None
    for e in [0.0, 1e-4, 1e-3, 1e-2, 5e-2, 0.3, 1.1]:
        st = oracle.initial_state(WL.B, WL.R)
        _, _, mask = oracle.activity_gate(lat["z_cur"], lat["z_prev"], labels,
                                          np.full(WL.B, e, np.float32), st, WL.R)
        if e == 0.0:
            assert mask.all()
        if prev is not None:
            assert np.all(mask <= prev)            # raising eps never switches a region on
        prev = mask
    assert not prev.any()


def test_scale_invariance_of_the_mask():
    labels, lat = _draw(seed=8)
    st = oracle.initial_state(WL.B, WL.R)
    _, w1, m1 = oracle.activity_gate(lat["z_cur"], lat["z_prev"], labels, lat["eps"], st, WL.R)
    zc = lat["z_cur"].astype(np.float64)
    zp2 = (zc + 4.0 * (lat["z_prev"].astype(np.float64) - zc)).astype(np.float32)
    st = oracle.initial_state(WL.B, WL.R)
    _, w2, m2 = oracle.activity_gate(lat["z_cur"], zp2, labels, lat["eps"], st, WL.R)
    assert np.array_equal(m1, m2)
    np.testing.assert_allclose(w1, w2, rtol=1e-4)


def test_frozen_delta_and_forced_reactivation():
    """A skipped patch keeps its cached change; it is skipped at most K steps in a row and
    then forced on; K = 0 never skips."""
    K = 3
    labels, lat = _draw(seed=10, fractions=[0.25] * WL.B)
    st = oracle.initial_state(WL.B, WL.R)
    rng = np.random.default_rng(5)
    runs = np.zeros((WL.B, WL.R), np.int64)
    z_prev = lat["z_prev"]
    z_cur = lat["z_cur"]
    forced_seen = False
    for step in range(12):
        before = st["delta"].copy()
        was_active = st["prev_active"].copy().astype(bool)
        skip_before = st["skip_count"].copy()
        score, weight, mask = oracle.activity_gate(z_cur, z_prev, labels, lat["eps"], st, WL.R, K=K)
        if step > 0:
            assert np.array_equal(score[~was_active].view(np.uint32), before[~was_active].view(np.uint32))
        gate_only = weight.astype(np.float64) >= lat["eps"][:, None]
        forced = mask.astype(bool) & ~gate_only
        assert np.all(skip_before[forced] >= K)
        forced_seen |= bool(forced.any())
        runs = np.where(mask.astype(bool), 0, runs + 1)
        assert runs.max() <= K
        assert np.array_equal(st["skip_count"], runs)
        assert np.array_equal(st["prev_active"], mask)
        # next step: same quiet/loud structure, new noise
        z_prev = z_cur
        z_cur = (z_cur + (z_cur - lat["z_prev"]) * 0 +
                 (lat["z_cur"] - lat["z_prev"]) * np.float32(rng.uniform(0.9, 1.1))).astype(np.float32)
    assert forced_seen
    st = oracle.initial_state(WL.B, WL.R)
    _, _, mask = oracle.activity_gate(lat["z_cur"], lat["z_prev"], labels, lat["eps"], st, WL.R, K=0)
    assert mask.all()


def test_always_active_label_is_outside_the_gate():
    wl = gen.workload("mmdit_small")
    lab = np.concatenate([np.arange(wl.n_grid) % wl.R, np.full(wl.n_text, wl.R)]).astype(np.int32)
    labels = np.ascontiguousarray(np.broadcast_to(lab, (wl.B, wl.N)))
    lat = gen.latent_pair(wl, 3, labels, fractions=[0.5, 0.25])
    st = oracle.initial_state(wl.B, wl.R)
    score, weight, mask = oracle.activity_gate(lat["z_cur"], lat["z_prev"], labels, lat["eps"], st, wl.R)
    np.testing.assert_allclose(weight.astype(np.float64).sum(1), 1.0, rtol=1e-6)
    idx, cu = oracle.compact(mask, labels, wl.R)
    tok = np.zeros(wl.B * wl.N, bool)
    tok[idx] = True
    assert tok.reshape(wl.B, wl.N)[:, wl.n_grid:].all()


def test_compaction_against_vectorised_restatement():
    wl = gen.workload("image_small")
    rng = np.random.default_rng(2)
    labels = rng.integers(0, wl.R, size=(wl.B, wl.N)).astype(np.int32)
    mask = gen.region_mask(wl, 4, [0.5, 0.75])
    idx, cu = oracle.compact(mask, labels, wl.R)
    flags = np.take_along_axis(mask, labels.astype(np.int64), axis=1).astype(bool)
    assert np.array_equal(idx, np.nonzero(flags.reshape(-1))[0].astype(np.int32))
    assert np.all(np.diff(idx) > 0)
    sizes = np.stack([np.bincount(labels[b], minlength=wl.R) for b in range(wl.B)])
    assert np.array_equal(np.diff(cu), (sizes * mask).sum(1))
    assert cu[0] == 0 and cu[-1] == idx.size


def test_tiny_workload_threshold_gives_about_half_active():
    wl = gen.workload("tiny")
    labels = gen.uniform_labels(wl)
    fracs = []
    for seed in range(12):
        lat = gen.latent_pair(wl, seed, labels, eps_fixed=1e-2)
        st = oracle.initial_state(wl.B, wl.R)
        _, weight, mask = oracle.activity_gate(lat["z_cur"], lat["z_prev"], labels, lat["eps"], st, wl.R)
        assert np.abs(weight / 1e-2 - 1).min() >= 1e-3
        assert np.array_equal(mask.sum(1), lat["n_loud"])
        fracs.append(mask.mean())
    assert 0.35 < np.mean(fracs) < 0.75
