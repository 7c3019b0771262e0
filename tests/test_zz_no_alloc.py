"""The allocation-free gate entry point against the regular one and against the CPU oracle.

fd_region_activity_noalloc serves callers that may not allocate device memory (a plug-in inside a
server with a frozen memory pool, a latency-critical thread, a process whose arena already owns
the whole GPU): it takes no context and no workspace, and keeps its accumulators in a fixed array
inside the library.  It must give what fd_region_activity gives, call after call, although all
calls share that array.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2607_12121_b200 as fd
from harness import dev, host, make_ctx

pytestmark = pytest.mark.gpu


class _State:
    def __init__(self, B, R):
        self.delta = torch.zeros((B, R), dtype=torch.float32, device="cuda")
        self.skip = torch.zeros((B, R), dtype=torch.int32, device="cuda")
        self.prev = torch.ones((B, R), dtype=torch.uint8, device="cuda")
        self.score = torch.full((B, R), -1.0, dtype=torch.float32, device="cuda")
        self.weight = torch.full((B, R), -1.0, dtype=torch.float32, device="cuda")
        self.mask = torch.full((B, R), 7, dtype=torch.uint8, device="cuda")


def test_noalloc_gate_matches_regular_gate_on_two_calls_in_a_row():
    wl = gen.workload("audio_small")
    labels_np = gen.uniform_labels(wl)
    K, eta = 3, 1e-12
    ctx = make_ctx(wl, gen.block_weights(wl, 1, n_blocks=1), n_blocks=1, engine=fd.FD_ENGINE_SIMT, max_skip_k=K,
                   gate_eta=eta)
    labels = dev(labels_np)
    ref, got = _State(wl.B, wl.R), _State(wl.B, wl.R)
    ost = oracle.initial_state(wl.B, wl.R)          # the oracle carries its own state through the same two calls
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    # two different problems back to back: the second call must not see the first call's sums
    for call, (seed, fr) in enumerate([(11, [0.25, 0.5, 0.75]), (12, [0.6, 0.3, 0.45])]):
        lat = gen.latent_pair(wl, seed, labels_np, fractions=fr)
        z_cur, z_prev, eps = dev(lat["z_cur"]), dev(lat["z_prev"]), dev(lat["eps"])
        fd.fd_region_activity(ctx, z_cur, z_prev, labels, wl.R, eps, ref.delta, ref.skip, ref.prev, ref.score,
                              ref.weight, ref.mask)
        fd.fd_poll_status(ctx)
        fd.fd_region_activity_noalloc(z_cur, z_prev, labels, wl.R, eps, eta, K, got.delta, got.skip, got.prev,
                                      got.score, got.weight, got.mask, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert np.array_equal(host(got.mask), host(ref.mask)), call
        np.testing.assert_allclose(host(got.score), host(ref.score), rtol=1e-5, atol=0)
        np.testing.assert_allclose(host(got.weight), host(ref.weight), rtol=1e-5, atol=0)
        assert np.array_equal(host(got.skip), host(ref.skip))
        assert np.array_equal(host(got.prev), host(ref.prev))
        assert np.array_equal(host(got.delta), host(got.score))
        o_score, o_weight, o_mask = oracle.activity_gate(lat["z_cur"], lat["z_prev"], labels_np, lat["eps"], ost, wl.R,
                                                         K=K, eta=eta)
        assert np.array_equal(host(got.mask), o_mask), call
        np.testing.assert_allclose(host(got.score), o_score, rtol=1e-5, atol=0)
        np.testing.assert_allclose(host(got.weight), o_weight, rtol=1e-5, atol=0)
        assert np.array_equal(host(got.skip), ost["skip_count"])
        assert 0 < host(got.mask).sum() < wl.B * wl.R


def test_noalloc_gate_refuses_oversized_problems():
    B, R = 3, fd.FD_NOALLOC_MAX_REGION_SLOTS // 3 + 1
    z = torch.zeros((B, R, 4), dtype=torch.float32, device="cuda")
    lab = torch.zeros((B, R), dtype=torch.int32, device="cuda")
    st = _State(B, R)
    eps = torch.zeros((B,), dtype=torch.float32, device="cuda")
    with pytest.raises(fd.FlashDiffError) as ei:
        fd.fd_region_activity_noalloc(z, z, lab, R, eps, 1e-12, 5, st.delta, st.skip, st.prev, st.score, st.weight,
                                      st.mask)
    assert ei.value.status == fd.FD_ERR_SHAPE
    assert (host(st.mask) == 7).all()          # nothing ran
