"""GPU parity of the sampler closure (patch embedding, final layer, latent update with cached drift:
Appendix A.1, Eq. sf-update) against the oracle, and a closed multi-step loop around the regional step."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2607_12121_b200 as fd
from harness import StepBuffers, dev, gpu_step, host, labels_for, make_ctx, max_abs, rel_l2, tdtype

pytestmark = pytest.mark.gpu


def _sampler(wl, seed):
    sw_np = gen.sampler_weights(wl, seed)
    sw_dev = {k: dev(v, tdtype(wl)) for k, v in sw_np.items()}
    return sw_np, sw_dev, fd.make_sampler_weights(sw_dev, wl.D)


@pytest.mark.parametrize("name,engine", [("tiny", fd.FD_ENGINE_SIMT), ("audio_small", fd.FD_ENGINE_SIMT),
                                         ("image_tc", fd.FD_ENGINE_TC), ("mmdit_tc", fd.FD_ENGINE_TC),
                                         ("audio", fd.FD_ENGINE_AUTO), ("video", fd.FD_ENGINE_AUTO)])     # full shapes
def test_embed_latent(name, engine):
    wl = gen.workload(name)
    ctx = make_ctx(wl, gen.block_weights(wl, 1, n_blocks=1), n_blocks=1, engine=engine)
    sw_np, sw_dev, sw = _sampler(wl, 3)
    z = np.random.default_rng(5).standard_normal((wl.B, wl.N, wl.D)).astype(np.float32)
    x = torch.empty((wl.B, wl.N, wl.H), dtype=tdtype(wl), device="cuda")
    fd.fd_embed_latent(ctx, sw, dev(z), x)
    fd.fd_poll_status(ctx)
    ref = oracle.sampler_embed(z, sw_np["w_in"], sw_np["b_in"], sw_np["pos"])
    if wl.dtype == "bf16":      # one bf16 rounding of an O(1) value
        assert max_abs(host(x), ref) <= 3e-2 and rel_l2(host(x), ref) <= 4e-3
    else:
        assert max_abs(host(x), ref) <= 1e-4 and rel_l2(host(x), ref) <= 1e-5


@pytest.mark.parametrize("name,engine,frac", [("tiny", fd.FD_ENGINE_SIMT, 0.5), ("audio_small", fd.FD_ENGINE_SIMT, 0.3),
                                              ("image_tc", fd.FD_ENGINE_TC, 0.7), ("mmdit_tc", fd.FD_ENGINE_TC, 1.0),
                                              ("audio_small", fd.FD_ENGINE_SIMT, 0.0),
                                              ("audio", fd.FD_ENGINE_AUTO, 0.64), ("video", fd.FD_ENGINE_AUTO, 0.45)])
def test_update_latent(name, engine, frac):
    """Active tokens get a fresh drift from their row of y; every other token keeps its cached drift bit for bit
    and moves along it; rows of y that belong to skipped tokens are not read (NaN there is harmless)."""
    wl = gen.workload(name)
    B, N, D, H = wl.B, wl.N, wl.D, wl.H
    ctx = make_ctx(wl, gen.block_weights(wl, 1, n_blocks=1), n_blocks=1, engine=engine)
    sw_np, sw_dev, sw = _sampler(wl, 4)
    g = np.random.default_rng(11)
    z = g.standard_normal((B, N, D)).astype(np.float32)
    y = g.standard_normal((B, N, H)).astype(np.float32) * np.float32(1.5) + np.float32(0.3)
    y = gen.round_bf16(y) if wl.dtype == "bf16" else y
    drift0 = g.standard_normal((B, N, D)).astype(np.float32)
    h = g.uniform(-0.5, 0.5, size=B).astype(np.float32)
    act = np.sort(g.choice(B * N, size=int(round(frac * B * N)), replace=False)).astype(np.int32)
    cu = np.concatenate([[0], np.cumsum(np.bincount(act // N, minlength=B))]).astype(np.int32)
    y_dev = y.copy()
    skipped = np.setdiff1d(np.arange(B * N), act)
    y_dev.reshape(B * N, H)[skipped] = np.nan
    idx_buf = np.full(B * N, -1, np.int32)
    idx_buf[:act.size] = act
    d_drift, d_zn = dev(drift0.copy()), torch.empty((B, N, D), dtype=torch.float32, device="cuda")
    fd.fd_update_latent(ctx, sw, dev(z), dev(y_dev, tdtype(wl)), dev(idx_buf), dev(cu), dev(h), d_drift, d_zn)
    fd.fd_poll_status(ctx)
    o_drift = drift0.copy()
    o_zn = oracle.sampler_update(z, y, act, sw_np["w_out"], sw_np["b_out"], h, o_drift, ln_eps=1e-6)
    got_drift, got_zn = host(d_drift).reshape(B * N, D), host(d_zn).reshape(B * N, D)
    assert np.array_equal(got_drift[skipped], drift0.reshape(B * N, D)[skipped])
    assert not np.isnan(got_zn).any()
    tol = 2e-3 if wl.dtype == "bf16" else 2e-5                  # fp32 accumulation over H terms of bf16 / fp32 products
    if act.size:
        assert max_abs(got_drift[act], o_drift.reshape(B * N, D)[act]) <= tol * 5
        assert rel_l2(got_drift[act], o_drift.reshape(B * N, D)[act]) <= tol
    assert max_abs(got_zn[skipped], o_zn.reshape(B * N, D)[skipped]) <= 1e-6
    assert max_abs(got_zn, o_zn.reshape(B * N, D)) <= tol * 5


@pytest.mark.parametrize("name,engine,steps", [("tiny", fd.FD_ENGINE_SIMT, 6), ("audio_tc", fd.FD_ENGINE_TC, 5)])
def test_closed_loop_matches_oracle(name, engine, steps):
    """embed -> regional step -> latent update, several steps on the device against the same loop in the oracle
    (fixed mask schedule: one all-active warm-up step, then half of the regions per step)."""
    wl = gen.workload(name)
    B, N, D, H, L = wl.B, wl.N, wl.D, wl.H, wl.L
    labels = labels_for(wl, 2)
    w = gen.block_weights(wl, 2)
    cond = gen.step_inputs(wl, 2, labels)["cond"]
    sw_np, sw_dev, sw = _sampler(wl, 6)
    ctx = make_ctx(wl, w, engine=engine)
    buf = StepBuffers(wl, L)
    dt = tdtype(wl)
    masks = [np.ones((B, wl.R), np.uint8)] + [gen.region_mask(wl, 20 + s, [0.5] * B) for s in range(steps - 1)]
    h = np.full(B, 0.1, np.float32)
    z0 = np.random.default_rng(9).standard_normal((B, N, D)).astype(np.float32)
    d_z, d_drift = dev(z0.copy()), torch.zeros((B, N, D), dtype=torch.float32, device="cuda")
    d_x = torch.empty((B, N, H), dtype=dt, device="cuda")
    o_z, o_drift = z0.copy(), np.zeros((B, N, D), np.float32)
    kv_ref, y_ref = np.zeros((L, B, 2, N, H), np.float32), np.zeros((B, N, H), np.float32)
    bf16 = wl.dtype == "bf16"
    for s, mask in enumerate(masks):
        fd.fd_embed_latent(ctx, sw, d_z, d_x)
        idx, cu = gpu_step(ctx, wl, d_x, dev(cond, dt), dev(labels), dev(mask), buf)
        fd.fd_update_latent(ctx, sw, d_z, buf.y, buf.active_idx, buf.cu_active, dev(h), d_drift, d_z)
        fd.fd_poll_status(ctx)
        o_x = oracle.sampler_embed(o_z, sw_np["w_in"], sw_np["b_in"], sw_np["pos"])
        o_x = gen.round_bf16(o_x) if bf16 else o_x              # the step's input is stored in the storage type
        o_idx, o_cu = oracle.regional_step(o_x, cond, labels, mask, w, kv_ref, y_ref, wl.heads, wl.R)
        assert np.array_equal(idx, o_idx) and np.array_equal(cu, o_cu)
        o_z = oracle.sampler_update(o_z, y_ref, o_idx, sw_np["w_out"], sw_np["b_out"], h, o_drift, ln_eps=1e-6)
        # the two trajectories drift apart slowly (bf16 block stack against the fp32 oracle); per step the latent
        # moves by h * |drift| ~ 0.1, of which the parity error is a few per cent at most
        tol = (3e-2 if bf16 else 2e-4) * (s + 1)
        assert max_abs(host(d_z), o_z) <= tol, s
        assert rel_l2(host(d_z), o_z) <= tol / 3, s
    assert idx.size < B * N                                     # the last steps really were gated


@pytest.mark.parametrize("name,engine", [("audio_small", fd.FD_ENGINE_SIMT), ("audio_tc", fd.FD_ENGINE_TC)])
def test_batch_former_defers_whole_requests(name, engine):
    """Sec. 4.3 on one device: under a token budget the batch former lets the high-priority requests run and the
    others wait at the step boundary (zero mask, zero step size).  A waiting request's latent, K/V cache and cached
    output stay bit for bit what they were; the running ones match the oracle's loop."""
    wl = gen.workload(name)
    B, N, D, H, L = wl.B, wl.N, wl.D, wl.H, wl.L
    labels = labels_for(wl, 4)
    w = gen.block_weights(wl, 4)
    cond = gen.step_inputs(wl, 4, labels)["cond"]
    sw_np, sw_dev, sw = _sampler(wl, 8)
    ctx = make_ctx(wl, w, engine=engine)
    buf = StepBuffers(wl, L)
    dt = tdtype(wl)
    bf16 = wl.dtype == "bf16"
    sizes = np.stack([np.bincount(labels[b][labels[b] < wl.R], minlength=wl.R) for b in range(B)])
    prio = np.arange(B) % 3
    z0 = np.random.default_rng(13).standard_normal((B, N, D)).astype(np.float32)
    d_z, d_drift = dev(z0.copy()), torch.zeros((B, N, D), dtype=torch.float32, device="cuda")
    d_x = torch.empty((B, N, H), dtype=dt, device="cuda")
    o_z, o_drift = z0.copy(), np.zeros((B, N, D), np.float32)
    kv_ref, y_ref = np.zeros((L, B, 2, N, H), np.float32), np.zeros((B, N, H), np.float32)
    resident = np.ones(B, np.uint8)
    waited = 0
    for s in range(3):
        gate = np.ones((B, wl.R), np.uint8) if s == 0 else gen.region_mask(wl, 40 + s, [0.6] * B)
        tok = (sizes * gate).sum(1).astype(np.int32)
        budget = int(tok.sum()) if s == 0 else int(tok.sum() * 0.6)
        chosen = fd.fd_sched_form_batch(prio, np.arange(B), tok, resident, budget, B)
        mask = gate * chosen[:, None]
        h = np.where(chosen, 0.1, 0.0).astype(np.float32)
        z_before, kv_before, y_before = host(d_z).copy(), host(buf.kv).copy(), host(buf.y).copy()
        fd.fd_embed_latent(ctx, sw, d_z, d_x)
        idx, cu = gpu_step(ctx, wl, d_x, dev(cond, dt), dev(labels), dev(mask), buf)
        fd.fd_update_latent(ctx, sw, d_z, buf.y, buf.active_idx, buf.cu_active, dev(h), d_drift, d_z)
        fd.fd_poll_status(ctx)
        o_x = oracle.sampler_embed(o_z, sw_np["w_in"], sw_np["b_in"], sw_np["pos"])
        o_x = gen.round_bf16(o_x) if bf16 else o_x
        o_idx, _ = oracle.regional_step(o_x, cond, labels, mask, w, kv_ref, y_ref, wl.heads, wl.R)
        assert np.array_equal(idx, o_idx)
        o_z = oracle.sampler_update(o_z, y_ref, o_idx, sw_np["w_out"], sw_np["b_out"], h, o_drift, ln_eps=1e-6)
        z_after, kv_after, y_after = host(d_z), host(buf.kv), host(buf.y)
        for b in np.nonzero(chosen == 0)[0]:
            waited += 1
            assert np.array_equal(z_after[b], z_before[b])
            assert np.array_equal(kv_after[:, b], kv_before[:, b]) and np.array_equal(y_after[b], y_before[b])
        tol = (3e-2 if bf16 else 2e-4) * (s + 1)
        assert max_abs(z_after, o_z) <= tol, s
        assert int((sizes * mask).sum()) <= budget
    assert waited > 0
