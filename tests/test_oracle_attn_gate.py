"""Pins of the oracle's attention-mass signal and its gate (paper Sec. 4.2: R_i, Delta_i = |R_i - Rbar_i|)."""
import numpy as np

import gen
import oracle


def _labels(B, N, sizes):
    lab = np.concatenate([np.full(n, i, np.int32) for i, n in enumerate(sizes)])
    assert lab.size == N
    return np.ascontiguousarray(np.broadcast_to(lab, (B, N)))


def test_uniform_attention_gives_one_over_n_for_every_region():
    """Zero queries: every row of SA is 1/N, so R_i = (1/|A_i|^2) |A_i| |A_i| / N = 1/N whatever the region."""
    B, N, H, heads = 2, 24, 16, 2
    sizes = [3, 9, 12]
    labels = _labels(B, N, sizes)
    k = np.random.default_rng(0).standard_normal((B, N, H)).astype(np.float32)
    idx = np.arange(B * N)
    mass = oracle.attention_mass(np.zeros((B * N, H), np.float32), k, labels, idx, heads, 3)
    r = mass / np.square(np.array(sizes, np.float64))[None]
    np.testing.assert_allclose(r, 1.0 / N, rtol=1e-12)


def test_attention_confined_to_the_own_region_gives_one_over_region_size():
    """Keys of a region share one direction and the region's queries point along it with a huge gain: all of a row's
    mass falls on its own region, so R_i = (1/|A_i|^2) |A_i| * 1 = 1/|A_i|."""
    B, N, H, heads = 1, 20, 8, 1
    sizes = [4, 6, 10]
    labels = _labels(B, N, sizes)
    dirs = np.eye(3, H, dtype=np.float32)
    k = dirs[labels[0]][None].copy()
    q = 200.0 * dirs[labels[0]]
    mass = oracle.attention_mass(q.astype(np.float32), k, labels, np.arange(N), heads, 3)
    np.testing.assert_allclose(mass[0] / np.square(np.array(sizes, np.float64)), 1.0 / np.array(sizes), rtol=1e-9)


def test_mass_matches_a_dense_softmax_matrix_and_skips_inactive_queries_and_unlabelled_tokens():
    g = np.random.default_rng(3)
    B, N, H, heads, R = 2, 18, 12, 3, 3
    labels = g.integers(0, R + 1, size=(B, N)).astype(np.int32)          # label R = always-active tokens, in no region
    q_all = g.standard_normal((B * N, H)).astype(np.float32)
    k = g.standard_normal((B, N, H)).astype(np.float32)
    idx = np.sort(g.choice(B * N, size=20, replace=False))
    mass = oracle.attention_mass(q_all[idx], k, labels, idx, heads, R)
    d = H // heads
    ref = np.zeros((B, R))
    for b in range(B):
        sa = np.zeros((N, N))
        for hd in range(heads):
            s = q_all.reshape(B, N, H)[b, :, hd * d:(hd + 1) * d].astype(np.float64) @ k[b, :, hd * d:(hd + 1) * d].astype(np.float64).T
            e = np.exp((s - s.max(-1, keepdims=True)) / np.sqrt(d))
            sa += e / e.sum(-1, keepdims=True) / heads
        for i in range(R):
            rows = [j for j in range(N) if labels[b, j] == i and (b * N + j) in set(idx.tolist())]
            cols = np.nonzero(labels[b] == i)[0]
            ref[b, i] = sa[np.ix_(rows, cols)].sum() if rows else 0.0
    np.testing.assert_allclose(mass, ref, rtol=1e-9, atol=1e-12)


def test_gate_tracks_the_change_of_importance_and_freezes_skipped_regions():
    B, R = 1, 4
    sizes = np.array([[2, 4, 4, 5]], np.int32)
    st = oracle.initial_state(B, R)
    st["rbar"] = np.zeros((B, R), np.float32)
    eps = np.array([0.15], np.float32)
    m1 = np.array([[0.4, 1.6, 3.2, 2.5]])                               # R = 0.1, 0.1, 0.2, 0.1
    imp, w, mask = oracle.attention_gate(m1, sizes, eps, st, R, K=5, eta=0.0)
    np.testing.assert_allclose(imp, [[0.1, 0.1, 0.2, 0.1]], rtol=1e-6)
    np.testing.assert_allclose(st["delta"], [[0.1, 0.1, 0.2, 0.1]], rtol=1e-6)      # Rbar started at zero
    np.testing.assert_allclose(w, [[0.2, 0.2, 0.4, 0.2]], rtol=1e-6)
    assert mask.tolist() == [[1, 1, 1, 1]]
    m2 = np.array([[0.4, 2.4, 3.2, 5.0]])                               # R = 0.1, 0.15, 0.2, 0.2: changes 0, 0.05, 0, 0.1
    imp, w, mask = oracle.attention_gate(m2, sizes, eps, st, R, K=5, eta=0.0)
    np.testing.assert_allclose(st["delta"], [[0.0, 0.05, 0.0, 0.1]], atol=1e-7)
    np.testing.assert_allclose(w, [[0.0, 1 / 3, 0.0, 2 / 3]], atol=1e-6)
    assert mask.tolist() == [[0, 1, 0, 1]]
    m3 = np.array([[99.0, 2.4, 99.0, 7.5]])                             # regions 0 and 2 were skipped: their mass is ignored
    imp, w, mask = oracle.attention_gate(m3, sizes, eps, st, R, K=5, eta=0.0)
    np.testing.assert_allclose(st["delta"], [[0.0, 0.0, 0.0, 0.1]], atol=1e-7)
    np.testing.assert_allclose(st["rbar"], [[0.1, 0.15, 0.2, 0.3]], rtol=1e-6)
    assert st["skip_count"].tolist() == [[2, 1, 2, 0]]


def test_forced_reactivation_applies_to_the_attention_gate_too():
    B, R = 1, 2
    sizes = np.array([[3, 3]], np.int32)
    st = oracle.initial_state(B, R)
    st["rbar"] = np.zeros((B, R), np.float32)
    st["delta"][:] = [[1e-6, 1.0]]
    st["prev_active"][:] = [[0, 1]]
    eps = np.array([0.1], np.float32)
    seen = []
    for step in range(4):
        _, _, mask = oracle.attention_gate(np.array([[0.9, 9.0 * (step + 2)]]), sizes, eps, st, R, K=2, eta=0.0)
        seen.append(int(mask[0, 0]))
    assert seen == [0, 0, 1, 0] or seen[:3] == [0, 0, 1]                 # skipped twice, then forced on


def test_block0_projection_reproduces_the_key_and_value_rows_the_block_oracle_wrote():
    """The helper that supplies the queries is the same projection as the one for K and V; the C block oracle
    (written separately) stores exactly those K / V rows in its cache, so they pin the helper's LayerNorm,
    modulation chunk order and weight slicing."""
    wl = gen.workload("audio_small")
    labels = gen.uniform_labels(wl)
    w = gen.block_weights(wl, 3, n_blocks=1)
    inp = gen.step_inputs(wl, 3, labels)
    kv = np.zeros((1, wl.B, 2, wl.N, wl.H), np.float32)
    y = np.zeros((wl.B, wl.N, wl.H), np.float32)
    mask = gen.region_mask(wl, 3, [0.5] * wl.B)
    idx, cu = oracle.regional_step(inp["x_cur"], inp["cond"], labels, mask, w, kv, y, wl.heads, wl.R)
    for part in (1, 2):
        rows = oracle.block0_projection(inp["x_cur"], inp["cond"], w, idx, part)
        got = kv[0][:, part - 1].reshape(wl.B * wl.N, wl.H)[idx]
        np.testing.assert_allclose(rows, got, rtol=0, atol=2e-5)
    q = oracle.block0_queries(inp["x_cur"], inp["cond"], w, idx)
    assert q.shape == (idx.size, wl.H) and not np.allclose(q, rows)
