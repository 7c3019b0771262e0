"""GPU parity of the paper's own gate signal (Sec. 4.2): the first block's own-region attention mass written by
fd_regional_step_mass, and the gate fd_region_activity_attn built on it, against the oracle."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2607_12121_b200 as fd
from harness import StepBuffers, dev, host, labels_for, make_ctx, tdtype

pytestmark = pytest.mark.gpu


def _sizes(labels, R):
    return np.stack([np.bincount(l[l < R], minlength=R) for l in labels]).astype(np.int32)


def _step_mass(ctx, wl, x, cond, labels, mask, buf, mass):
    fd.fd_regional_step_mass(ctx, x, cond, labels, mask, wl.R, buf.kv, buf.y, buf.active_idx, buf.cu_active, mass)
    fd.fd_poll_status(ctx)
    cu = host(buf.cu_active)
    return host(buf.active_idx)[: cu[-1]]


@pytest.mark.parametrize("name,engine", [("tiny", fd.FD_ENGINE_SIMT), ("audio_small", fd.FD_ENGINE_SIMT),
                                         ("mmdit_small", fd.FD_ENGINE_SIMT), ("audio_tc", fd.FD_ENGINE_TC),
                                         ("image_tc", fd.FD_ENGINE_TC), ("wide_tc", fd.FD_ENGINE_TC),
                                         ("mmdit_tc", fd.FD_ENGINE_TC), ("audio_tc_few_ctas", fd.FD_ENGINE_TC),
                                         ("audio_tc_cut", fd.FD_ENGINE_TC), ("image_tc_cut", fd.FD_ENGINE_TC),
                                         ("wide_tc_cut", fd.FD_ENGINE_TC)])
def test_region_mass_matches_oracle(monkeypatch, name, engine):
    if name.endswith("_cut"):             # the attention items are cut along the keys and put together by a second kernel
        monkeypatch.setenv("FD_ATT_SPLIT", "2")
        wl = gen.workload(name[:-len("_cut")])
    elif name.endswith("_few_ctas"):        # several items per CTA, odd key-tile count: the tile parity an item starts on alternates
        monkeypatch.setenv("FD_TC_MAX_CTAS", "2")
        wl = gen.workload(name[:-len("_few_ctas")]).replace(grid=(330,), R=10)
    else:
        wl = gen.workload(name)
    labels = labels_for(wl, 4)
    w = gen.block_weights(wl, 4)
    w["w_qkv"][:, :wl.H] *= np.float32(4.0)                      # sharper attention: the mass differs from region to region
    inp = gen.step_inputs(wl, 4, labels)
    ctx = make_ctx(wl, w, engine=engine)
    buf = StepBuffers(wl, wl.L)
    dt = tdtype(wl)
    B, N, H, L = wl.B, wl.N, wl.H, wl.L
    kv_ref, y_ref = np.zeros((L, B, 2, N, H), np.float32), np.zeros((B, N, H), np.float32)
    mass = torch.full((B, wl.R), -1.0, dtype=torch.float64, device="cuda")
    masks = [np.ones((B, wl.R), np.uint8), gen.region_mask(wl, 5, [0.5] * B)]
    for x_np, mask in zip((inp["x_prev"], inp["x_cur"]), masks):
        idx = _step_mass(ctx, wl, dev(x_np, dt), dev(inp["cond"], dt), dev(labels), dev(mask), buf, mass)
        o_idx, _ = oracle.regional_step(x_np, inp["cond"], labels, mask, w, kv_ref, y_ref, wl.heads, wl.R)
        assert np.array_equal(idx, o_idx)
        q = oracle.block0_queries(x_np, inp["cond"], w, o_idx)
        ref = oracle.attention_mass(q, kv_ref[0][:, 0], labels, o_idx, wl.heads, wl.R)
        got = host(mass)
        ran = mask.astype(bool)
        assert np.all(got[~ran] == 0.0)                          # regions that did not run report nothing
        tol = 2e-2 if wl.dtype == "bf16" else 1e-4               # bf16 Q / K rounding moves softmax probabilities by ~1 %
        np.testing.assert_allclose(got[ran], ref[ran], rtol=tol, atol=1e-6)
    assert ref[ran].std() / ref[ran].mean() > 0.005              # the signal is not trivially uniform


def test_attention_gate_matches_oracle_over_steps():
    """Masses drawn directly (no block stack): the gate's arithmetic, state and forced reactivation, step by step."""
    B, R, K = 3, 40, 3
    g = np.random.default_rng(8)
    sizes = g.integers(4, 40, size=(B, R)).astype(np.int32)
    wl = gen.workload("audio_small").replace(B=B, R=R)
    ctx = make_ctx(wl, gen.block_weights(wl, 1, n_blocks=1), n_blocks=1, engine=fd.FD_ENGINE_SIMT, max_skip_k=K)
    st = oracle.initial_state(B, R)
    st["rbar"] = np.zeros((B, R), np.float32)
    d = {k: dev(v.copy()) for k, v in st.items()}
    out = [torch.empty((B, R), dtype=torch.float32, device="cuda"), torch.empty((B, R), dtype=torch.float32, device="cuda"),
           torch.empty((B, R), dtype=torch.uint8, device="cuda")]
    eps = np.array([0.01, 0.02, 0.03], np.float32)
    base = g.uniform(0.5, 2.0, size=(B, R)) * sizes
    forced = False
    for step in range(8):
        mass = base * (1.0 + 0.2 * g.standard_normal((B, R)) * (g.random((B, R)) < 0.4))
        o_imp, o_w, o_mask = oracle.attention_gate(mass, sizes, eps, st, R, K=K, eta=1e-12)
        assert np.abs(o_w / eps[:, None] - 1).min() >= 1e-3      # the seeded draws keep every decision off the threshold
        fd.fd_region_activity_attn(ctx, dev(mass), dev(sizes), dev(eps), d["rbar"], d["delta"], d["skip_count"],
                                   d["prev_active"], out[0], out[1], out[2])
        fd.fd_poll_status(ctx)
        assert np.array_equal(host(out[2]), o_mask), step
        np.testing.assert_allclose(host(out[0]), o_imp, rtol=1e-6)
        np.testing.assert_allclose(host(out[1]), o_w, rtol=1e-5, atol=1e-12)
        assert np.array_equal(host(d["skip_count"]), st["skip_count"])
        assert np.array_equal(host(d["prev_active"]), st["prev_active"])
        np.testing.assert_allclose(host(d["delta"]), st["delta"], rtol=1e-6, atol=1e-12)
        forced |= bool((o_mask.astype(bool) & (o_w < eps[:, None])).any())
    assert forced and 0 < o_mask.sum() < B * R


def test_closed_loop_with_the_attention_gate():
    """step (+ mass) -> attention gate -> next step's mask, GPU against oracle, fp32 engine: the masks the two sides
    derive agree step by step (weights away from the threshold), starting from the all-active warm-up."""
    wl = gen.workload("tiny")
    B, N, H, L, R = wl.B, wl.N, wl.H, wl.L, wl.R
    labels = labels_for(wl, 6)
    sizes = _sizes(labels, R)
    w = gen.block_weights(wl, 6)
    w["w_qkv"][:, :H] *= np.float32(4.0)
    inp = gen.step_inputs(wl, 6, labels)
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_SIMT)
    buf = StepBuffers(wl, L)
    kv_ref, y_ref = np.zeros((L, B, 2, N, H), np.float32), np.zeros((B, N, H), np.float32)
    st = oracle.initial_state(B, R)
    st["rbar"] = np.zeros((B, R), np.float32)
    d = {k: dev(v.copy()) for k, v in st.items()}
    out = [torch.empty((B, R), dtype=torch.float32, device="cuda"), torch.empty((B, R), dtype=torch.float32, device="cuda"),
           torch.empty((B, R), dtype=torch.uint8, device="cuda")]
    mass = torch.zeros((B, R), dtype=torch.float64, device="cuda")
    eps = np.full(B, 0.03, np.float32)
    mask = np.ones((B, R), np.uint8)
    g = np.random.default_rng(1)
    x_np = inp["x_prev"]
    gated = 0
    for step in range(5):
        idx = _step_mass(ctx, wl, dev(x_np), dev(inp["cond"]), dev(labels), dev(mask), buf, mass)
        o_idx, _ = oracle.regional_step(x_np, inp["cond"], labels, mask, w, kv_ref, y_ref, wl.heads, R)
        assert np.array_equal(idx, o_idx)
        q = oracle.block0_queries(x_np, inp["cond"], w, o_idx)
        o_mass = oracle.attention_mass(q, kv_ref[0][:, 0], labels, o_idx, wl.heads, R)
        o_imp, o_w, o_mask = oracle.attention_gate(o_mass, sizes, eps, st, R)
        fd.fd_region_activity_attn(ctx, mass, dev(sizes), dev(eps), d["rbar"], d["delta"], d["skip_count"],
                                   d["prev_active"], out[0], out[1], out[2])
        fd.fd_poll_status(ctx)
        assert np.abs(o_w / eps[:, None] - 1).min() >= 2e-2      # the oracle's (seeded, deterministic) trajectory stays off the threshold
        assert np.array_equal(host(out[2]), o_mask), step
        np.testing.assert_allclose(host(out[1]), o_w, rtol=5e-3, atol=1e-9)
        mask = o_mask
        gated += int(mask.sum() < B * R)
        x_np = (x_np + np.float32(0.05) * g.standard_normal(x_np.shape).astype(np.float32)).astype(np.float32)
    assert gated >= 1
