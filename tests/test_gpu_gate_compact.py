"""GPU parity: gate (scores 1e-5 relative, mask bit-exact) and compaction (bit-exact)."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2607_12121_b200 as fd
from harness import dev, host, make_ctx, labels_for

pytestmark = pytest.mark.gpu


def _ctx(wl):
    w = gen.block_weights(wl, 1, n_blocks=1)
    return make_ctx(wl, w, n_blocks=1, engine=fd.FD_ENGINE_SIMT)


class GateState:
    def __init__(self, B, R):
        self.delta = torch.zeros((B, R), dtype=torch.float32, device="cuda")
        self.skip = torch.zeros((B, R), dtype=torch.int32, device="cuda")
        self.prev = torch.ones((B, R), dtype=torch.uint8, device="cuda")
        self.score = torch.empty((B, R), dtype=torch.float32, device="cuda")
        self.weight = torch.empty((B, R), dtype=torch.float32, device="cuda")
        self.mask = torch.empty((B, R), dtype=torch.uint8, device="cuda")


def _gate(ctx, wl, z_cur, z_prev, labels, eps, st):
    fd.fd_region_activity(ctx, z_cur, z_prev, labels, wl.R, eps, st.delta, st.skip, st.prev, st.score, st.weight,
                          st.mask)
    fd.fd_poll_status(ctx)
    return host(st.score), host(st.weight), host(st.mask)


@pytest.mark.parametrize("name,seed", [("tiny", 0), ("audio_small", 1), ("image_small", 2), ("mmdit_small", 3),
                                       ("video_small", 4), ("audio", 5), ("mmdit", 6), ("video", 7),
                                       ("image", 8)])                                        # ... and full shapes
def test_gate_single_step(name, seed):
    wl = gen.workload(name)
    labels = labels_for(wl, seed)
    if name == "tiny":
        lat = gen.latent_pair(wl, seed, labels, eps_fixed=1e-2)
    else:
        lat = gen.latent_pair(wl, seed, labels, fractions=gen.request_fractions(wl, seed))
    ost = oracle.initial_state(wl.B, wl.R)
    o_score, o_weight, o_mask = oracle.activity_gate(lat["z_cur"], lat["z_prev"], labels, lat["eps"], ost, wl.R)
    assert np.abs(o_weight / np.maximum(lat["eps"][:, None], 1e-30) - 1).min() >= 1e-3
    ctx = _ctx(wl)
    st = GateState(wl.B, wl.R)
    score, weight, mask = _gate(ctx, wl, dev(lat["z_cur"]), dev(lat["z_prev"]), dev(labels), dev(lat["eps"]), st)
    assert np.array_equal(mask, o_mask)
    np.testing.assert_allclose(score, o_score, rtol=1e-5, atol=0)
    np.testing.assert_allclose(weight, o_weight, rtol=1e-5, atol=0)
    assert np.array_equal(host(st.prev), ost["prev_active"])
    assert np.array_equal(host(st.skip), ost["skip_count"])


def test_gate_multi_step_state_and_forced_reactivation():
    wl = gen.workload("audio_small")
    labels = gen.uniform_labels(wl)
    lat = gen.latent_pair(wl, 7, labels, fractions=[0.25, 0.5, 0.75])
    ctx = make_ctx(wl, gen.block_weights(wl, 1, n_blocks=1), n_blocks=1, engine=fd.FD_ENGINE_SIMT, max_skip_k=3)
    st = GateState(wl.B, wl.R)
    ost = oracle.initial_state(wl.B, wl.R)
    rng = np.random.default_rng(0)
    z_prev, z_cur = lat["z_prev"], lat["z_cur"]
    step_delta = lat["z_cur"] - lat["z_prev"]
    forced = False
    for step in range(9):
        o_score, o_weight, o_mask = oracle.activity_gate(z_cur, z_prev, labels, lat["eps"], ost, wl.R, K=3)
        score, weight, mask = _gate(ctx, wl, dev(z_cur), dev(z_prev), dev(labels), dev(lat["eps"]), st)
        assert np.array_equal(mask, o_mask), step
        np.testing.assert_allclose(score, o_score, rtol=1e-5)
        np.testing.assert_allclose(weight, o_weight, rtol=1e-5)
        assert np.array_equal(host(st.skip), ost["skip_count"])
        forced |= bool((o_mask.astype(bool) & (o_weight < lat["eps"][:, None])).any())
        z_prev = z_cur
        z_cur = (z_cur + step_delta * np.float32(rng.uniform(0.95, 1.05))).astype(np.float32)
    assert forced


def test_gate_odd_channel_count_uses_scalar_path():
    wl = gen.workload("audio_small").replace(D=6)
    labels = gen.uniform_labels(wl)
    lat = gen.latent_pair(wl, 9, labels, fractions=[0.5, 0.5, 0.5])
    ost = oracle.initial_state(wl.B, wl.R)
    o_score, o_weight, o_mask = oracle.activity_gate(lat["z_cur"], lat["z_prev"], labels, lat["eps"], ost, wl.R)
    ctx = _ctx(wl)
    st = GateState(wl.B, wl.R)
    score, weight, mask = _gate(ctx, wl, dev(lat["z_cur"]), dev(lat["z_prev"]), dev(labels), dev(lat["eps"]), st)
    assert np.array_equal(mask, o_mask)
    np.testing.assert_allclose(score, o_score, rtol=1e-5)


def test_gate_streaming_kernel_edges():
    """Shapes that cross every boundary of the streaming reduction: a token count that is no multiple of the ring
    stage, a channel count whose vector count is no power of two, requests that share a CTA, runs of frozen
    regions longer than a stage (copied by nobody), always-active tokens (label R) and a frozen/fresh mix."""
    B, N, D, R, K, eta = 3, 1000, 48, 7, 5, 1e-12
    rng = np.random.default_rng(123)
    labels = np.empty((B, N), np.int32)
    for b in range(B):
        t, runs = 0, []
        while t < N:
            n = int(rng.integers(1, 260))
            runs.append((min(n, N - t), int(rng.integers(0, R + 1))))
            t += n
        labels[b] = np.concatenate([np.full(n, l, np.int32) for n, l in runs])[:N]
    labels[0, 100:420] = 2                                  # a long run of a region that is frozen below
    z_prev = rng.standard_normal((B, N, D)).astype(np.float32)
    scale = np.float32(10.0) ** rng.uniform(-3, -1, size=(B, N, 1)).astype(np.float32)
    z_cur = (z_prev + scale * rng.standard_normal((B, N, D)).astype(np.float32)).astype(np.float32)
    ost = oracle.initial_state(B, R)
    ost["prev_active"][:, 2] = 0
    ost["prev_active"][1, 5] = 0
    ost["delta"][:, 2] = np.float32(0.02)
    ost["delta"][1, 5] = np.float32(0.004)
    ost["skip_count"][:, 2] = 1
    ost["skip_count"][1, 5] = 2
    eps = np.array([0.11, 0.14, 0.17], np.float32)
    st = GateState(B, R)
    st.delta.copy_(dev(ost["delta"])); st.skip.copy_(dev(ost["skip_count"])); st.prev.copy_(dev(ost["prev_active"]))
    o_score, o_weight, o_mask = oracle.activity_gate(z_cur, z_prev, labels, eps, ost, R, K=K, eta=eta)
    assert np.abs(o_weight / eps[:, None] - 1).min() >= 1e-3       # no decision sits on the threshold
    assert 0 < o_mask.sum() < B * R
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    fd.fd_region_activity_noalloc(dev(z_cur), dev(z_prev), dev(labels), R, dev(eps), eta, K, st.delta, st.skip,
                                  st.prev, st.score, st.weight, st.mask, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(host(st.mask), o_mask)
    np.testing.assert_allclose(host(st.score), o_score, rtol=1e-5, atol=0)
    np.testing.assert_allclose(host(st.weight), o_weight, rtol=1e-5, atol=0)
    assert np.array_equal(host(st.prev), ost["prev_active"])
    assert np.array_equal(host(st.skip), ost["skip_count"])


def _eps_in_a_gap(weight):
    """A threshold per request that sits in the widest relative gap between neighbouring weights of the
    middle half of the sorted weights, so that no decision lands within 1e-3 of it."""
    eps = np.empty(weight.shape[0], np.float32)
    for b, w in enumerate(weight):
        s = np.sort(w.astype(np.float64))
        lo, hi = len(s) // 4, max(len(s) // 4 + 1, 3 * len(s) // 4)
        k = lo + int(np.argmax(s[lo + 1:hi + 1] / np.maximum(s[lo:hi], 1e-300)))
        eps[b] = np.float32(np.sqrt(s[k] * s[k + 1]))
    return eps


@pytest.mark.parametrize("B,N,D,R,via", [(2, 300, 2052, 9, "ctx"),            # rows wider than a ring stage
                                         (2, 300, 2052, 9, "noalloc"),
                                         (1, 24000, 8, 12000, "noalloc"),     # accumulators beyond the default shared-memory size
                                         (1, 16400, 4, 16384, "noalloc"),     # the entry point's largest region count
                                         (1, 20000, 4, 18000, "ctx")])        # accumulators beyond any shared-memory size
def test_gate_reductions_beyond_the_streaming_form(B, N, D, R, via):
    """Shapes the bulk-copy reduction does not take: the plain vector-load kernel with its per-CTA accumulators in
    (opt-in sized) shared memory, and the one-warp-per-token kernel that adds straight into global memory."""
    K, eta = 5, 1e-12
    rng = np.random.default_rng(1000 + R + D)
    labels = rng.integers(0, R + 1, size=(B, N)).astype(np.int32)
    labels[:, : min(N, R)] = np.arange(min(N, R), dtype=np.int32)            # every region has at least one token
    z_prev = rng.standard_normal((B, N, D)).astype(np.float32)
    scale = (np.float32(10.0) ** rng.uniform(-3, -1, size=(B, R + 1)).astype(np.float32))
    sc_tok = np.take_along_axis(scale, labels.astype(np.int64), axis=1)[..., None]
    z_cur = (z_prev + sc_tok * rng.standard_normal((B, N, D)).astype(np.float32)).astype(np.float32)
    frozen = rng.random((B, R)) < 0.1

    def start_state():
        st = oracle.initial_state(B, R)
        st["prev_active"][frozen] = 0
        st["delta"][frozen] = np.float32(0.01)
        st["skip_count"][frozen] = 2
        return st

    probe = start_state()
    _, w0, _ = oracle.activity_gate(z_cur, z_prev, labels, np.zeros(B, np.float32), probe, R, K=K, eta=eta)
    eps = _eps_in_a_gap(w0)
    ost = start_state()
    o_score, o_weight, o_mask = oracle.activity_gate(z_cur, z_prev, labels, eps, ost, R, K=K, eta=eta)
    assert np.abs(o_weight / eps[:, None] - 1).min() >= 1e-3
    assert 0 < o_mask.sum() < B * R
    st = GateState(B, R)
    first = start_state()
    st.delta.copy_(dev(first["delta"])); st.skip.copy_(dev(first["skip_count"])); st.prev.copy_(dev(first["prev_active"]))
    if via == "noalloc":
        status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        fd.fd_region_activity_noalloc(dev(z_cur), dev(z_prev), dev(labels), R, dev(eps), eta, K, st.delta, st.skip,
                                      st.prev, st.score, st.weight, st.mask, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
    else:
        wl = gen.workload("audio_small").replace(grid=(N,), B=B, R=R, D=D, L=1)
        ctx = make_ctx(wl, gen.block_weights(wl, 1, n_blocks=1), n_blocks=1, engine=fd.FD_ENGINE_SIMT, max_skip_k=K,
                       gate_eta=eta)
        fd.fd_region_activity(ctx, dev(z_cur), dev(z_prev), dev(labels), R, dev(eps), st.delta, st.skip, st.prev,
                              st.score, st.weight, st.mask)
        fd.fd_poll_status(ctx)
        assert fd.fd_destroy(ctx) == fd.FD_OK
    assert np.array_equal(host(st.mask), o_mask)
    np.testing.assert_allclose(host(st.score), o_score, rtol=1e-5, atol=0)
    np.testing.assert_allclose(host(st.weight), o_weight, rtol=1e-5, atol=0)
    assert np.array_equal(host(st.prev), ost["prev_active"])
    assert np.array_equal(host(st.skip), ost["skip_count"])


@pytest.mark.parametrize("name", ["tiny", "audio_small", "mmdit_small", "video_small"])
def test_compaction_bit_exact(name):
    from harness import StepBuffers, gpu_step
    wl = gen.workload(name)
    labels = labels_for(wl, 5)
    w = gen.block_weights(wl, 1, n_blocks=1)
    ctx = make_ctx(wl, w, n_blocks=1, engine=fd.FD_ENGINE_SIMT)
    inp = gen.step_inputs(wl, 5, labels)
    buf = StepBuffers(wl, 1)
    dt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    for fr in ([1.0] * wl.B, [0.5] * wl.B, [0.0] * wl.B, list(gen.request_fractions(wl, 3))):
        mask = gen.region_mask(wl, 11, fr)
        idx, cu = gpu_step(ctx, wl, dev(inp["x_cur"], dt), dev(inp["cond"], dt), dev(labels), dev(mask), buf)
        o_idx, o_cu = oracle.compact(mask, labels, wl.R)
        assert np.array_equal(cu, o_cu)
        assert np.array_equal(idx, o_idx)


def test_bad_label_is_reported_not_trapped():
    wl = gen.workload("audio_small")
    labels = gen.uniform_labels(wl).copy()
    labels[1, 7] = wl.R + 3
    lat = gen.latent_pair(wl, 1, gen.uniform_labels(wl), fractions=[0.5] * wl.B)
    ctx = _ctx(wl)
    st = GateState(wl.B, wl.R)
    fd.fd_region_activity(ctx, dev(lat["z_cur"]), dev(lat["z_prev"]), dev(labels), wl.R, dev(lat["eps"]), st.delta,
                          st.skip, st.prev, st.score, st.weight, st.mask)
    with pytest.raises(fd.FlashDiffError) as ei:
        fd.fd_poll_status(ctx)
    assert ei.value.status == fd.FD_ERR_STATE
    fd.fd_poll_status(ctx)          # cleared; the context stays usable
    # a status nobody polled for comes back from fd_destroy
    fd.fd_region_activity(ctx, dev(lat["z_cur"]), dev(lat["z_prev"]), dev(labels), wl.R, dev(lat["eps"]), st.delta,
                          st.skip, st.prev, st.score, st.weight, st.mask)
    assert fd.fd_destroy(ctx) == fd.FD_ERR_STATE
