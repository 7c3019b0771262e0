"""Pins of the sampler-closure oracle (Appendix A.1, Eq. sf-update) against what the mathematics fixes."""
import numpy as np

import gen
import oracle


def _setup(seed=0, B=2, N=12, D=8, H=32):
    g = np.random.default_rng(seed)
    z = g.standard_normal((B, N, D)).astype(np.float32)
    y = g.standard_normal((B, N, H)).astype(np.float32)
    w_out = (g.standard_normal((D, H)) / np.sqrt(H)).astype(np.float32)
    b_out = (0.1 * g.standard_normal(D)).astype(np.float32)
    return g, z, y, w_out, b_out


def test_zero_step_size_leaves_latent_unchanged():
    g, z, y, w_out, b_out = _setup()
    drift = g.standard_normal(z.shape).astype(np.float32)
    zn = oracle.sampler_update(z, y, np.arange(z.shape[0] * z.shape[1]), w_out, b_out, np.zeros(2, np.float32), drift)
    assert np.array_equal(zn, z)


def test_all_active_is_a_plain_euler_step_of_the_final_layer():
    """With every token active the update is x + h * W_out LN(y) + b_out, written here with library routines."""
    g, z, y, w_out, b_out = _setup(1)
    B, N, D = z.shape
    h = np.array([0.3, -0.7], np.float32)
    drift = np.full(z.shape, np.nan, np.float32)                      # nothing cached is read
    zn = oracle.sampler_update(z, y, np.arange(B * N), w_out, b_out, h, drift, ln_eps=1e-6)
    y64 = y.astype(np.float64)
    u = (y64 - y64.mean(-1, keepdims=True)) / np.sqrt(y64.var(-1, keepdims=True) + 1e-6)
    ref = z.astype(np.float64) + h[:, None, None].astype(np.float64) * (
        np.einsum("bnh,dh->bnd", u, w_out.astype(np.float64)) + b_out.astype(np.float64)).astype(np.float32)
    np.testing.assert_allclose(zn, ref, rtol=0, atol=2e-6)
    assert not np.isnan(drift).any()                                  # every token's drift was refreshed


def test_skipped_tokens_move_along_their_cached_drift_and_keep_it():
    """A token skipped k steps in a row has moved k * h * c with c the drift of its last active step, and the rows of
    y belonging to skipped tokens are never read (NaN there must not matter)."""
    g, z, y, w_out, b_out = _setup(2)
    B, N, D = z.shape
    h = np.array([0.25, 0.5], np.float32)
    drift = np.zeros(z.shape, np.float32)
    z1 = oracle.sampler_update(z, y, np.arange(B * N), w_out, b_out, h, drift)
    cached = drift.copy()
    active = np.array([0, 1, 2, 5, N + 3, N + 4], np.int64)             # the rest is skipped from now on
    skipped = np.setdiff1d(np.arange(B * N), active)
    zk = z1
    for k in range(3):
        y2 = g.standard_normal(y.shape).astype(np.float32)
        y2.reshape(B * N, -1)[skipped] = np.nan
        zk = oracle.sampler_update(zk, y2, active, w_out, b_out, h, drift)
    assert np.array_equal(drift.reshape(B * N, D)[skipped], cached.reshape(B * N, D)[skipped])
    hb = np.repeat(h, N)[skipped, None].astype(np.float64)
    expect = z1.reshape(B * N, D)[skipped].astype(np.float64) + 3 * hb * cached.reshape(B * N, D)[skipped]
    np.testing.assert_allclose(zk.reshape(B * N, D)[skipped], expect, rtol=0, atol=3e-6)
    assert not np.isnan(zk).any()
    assert not np.array_equal(drift.reshape(B * N, D)[active], cached.reshape(B * N, D)[active])


def test_final_layer_is_invariant_to_shift_and_scale_of_its_input_row():
    g, z, y, w_out, b_out = _setup(3)
    d0 = oracle.token_drift(y[0, 0], w_out, b_out, 1e-12)
    d1 = oracle.token_drift(3.5 * y[0, 0] + 11.0, w_out, b_out, 1e-12)
    np.testing.assert_allclose(d1, d0, rtol=1e-6, atol=1e-7)
    # a constant row has no direction: only the bias is left
    np.testing.assert_allclose(oracle.token_drift(np.full(32, 4.0, np.float32), w_out, b_out, 1e-6), b_out, atol=1e-7)


def test_embedding_is_the_linear_map_plus_bias_plus_position():
    wl = gen.workload("audio_small")
    sw = gen.sampler_weights(wl, 5)
    g = np.random.default_rng(4)
    z = g.standard_normal((wl.B, wl.N, wl.D)).astype(np.float32)
    x = oracle.sampler_embed(z, sw["w_in"], sw["b_in"], sw["pos"])
    ref = np.einsum("bnd,hd->bnh", z.astype(np.float64), sw["w_in"].astype(np.float64)) + sw["b_in"] + sw["pos"][None]
    np.testing.assert_allclose(x, ref, rtol=0, atol=1e-5)
    # linearity: a zero latent gives bias + position exactly
    x0 = oracle.sampler_embed(np.zeros_like(z), sw["w_in"], sw["b_in"], sw["pos"])
    np.testing.assert_array_equal(x0[0], (sw["b_in"].astype(np.float64) + sw["pos"].astype(np.float64)).astype(np.float32))
