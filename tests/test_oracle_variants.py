"""Pins for the block variants of the oracle (QK-RMSNorm, rotary position embedding): what the mathematics fixes,
an independent restatement with complex numbers and library routines, and the two separately written C programs
against each other."""
import numpy as np
import pytest
import torch

import gen
import oracle

WL = gen.workload("tiny").replace(name="v", H=64, heads=2, head_dim=32, M=96, Hc=48, grid=(6, 8), B=2, R=6, D=8, L=2,
                                  labels="segments")
PROGRAMS = ("regional", "dense")


def _rows(seed, n=11, H=64):
    g = np.random.default_rng(seed)
    return g.standard_normal((n, H)).astype(np.float32) * 3, g.standard_normal((n, H)).astype(np.float32)


@pytest.mark.parametrize("program", PROGRAMS)
def test_rms_norm_gives_unit_rms_and_forgets_the_scale(program):
    q, k = _rows(1)
    ones = np.ones(32, np.float32)
    qn, kn = oracle.qk_variants(q, k, 2, q_norm_w=ones, k_norm_w=ones, qk_norm_eps=1e-12, program=program)
    for a in (qn, kn):
        rms = np.sqrt((a.reshape(-1, 2, 32).astype(np.float64) ** 2).mean(-1))
        np.testing.assert_allclose(rms, 1.0, rtol=1e-6)
    q2, _ = oracle.qk_variants(q * np.float32(7.5), k, 2, q_norm_w=ones, k_norm_w=ones, qk_norm_eps=1e-12, program=program)
    np.testing.assert_allclose(q2, qn, rtol=2e-6, atol=1e-7)          # scale invariance
    # the weight multiplies channel-wise, the same vector for every head; the key's weight does not touch the query
    gq = np.linspace(0.5, 2.0, 32).astype(np.float32)
    q3, k3 = oracle.qk_variants(q, k, 2, q_norm_w=gq, k_norm_w=ones, qk_norm_eps=1e-12, program=program)
    np.testing.assert_allclose(q3.reshape(-1, 2, 32), qn.reshape(-1, 2, 32) * gq, rtol=2e-6)
    assert np.array_equal(k3, kn)
    # eps sits under the root next to the mean square: a zero row stays zero, a tiny row is damped
    z, _ = oracle.qk_variants(np.zeros_like(q), k, 2, q_norm_w=ones, k_norm_w=ones, qk_norm_eps=1e-6, program=program)
    assert not z.any()
    t, _ = oracle.qk_variants(np.full_like(q, 1e-3), k, 2, q_norm_w=ones, k_norm_w=ones, qk_norm_eps=1e-6, program=program)
    np.testing.assert_allclose(t, 1e-3 / np.sqrt(1e-6 + 1e-6), rtol=1e-5)


@pytest.mark.parametrize("program", PROGRAMS)
def test_rope_is_a_rotation_that_depends_on_relative_position_only(program):
    wl = WL.replace(grid=(40,), B=1, R=5)
    tab = gen.block_variants(wl, 0, qk_norm=False)
    g = np.random.default_rng(2)
    a, b = g.standard_normal(64).astype(np.float32), g.standard_normal(64).astype(np.float32)
    # the same two vectors placed at every position
    q = np.broadcast_to(a, (40, 64)).copy()
    k = np.broadcast_to(b, (40, 64)).copy()
    qr, kr = oracle.qk_variants(q, k, 2, rope_cos=tab["rope_cos"], rope_sin=tab["rope_sin"], program=program)
    # norms of every channel pair are kept
    pair_norm = lambda x: np.hypot(x[..., 0::2], x[..., 1::2])
    np.testing.assert_allclose(pair_norm(qr), pair_norm(q), rtol=1e-6, atol=1e-7)
    # position 0 is the identity
    assert np.array_equal(qr[0], a) and np.array_equal(kr[0], b)
    # per head, <rot(a, m), rot(b, n)> is a function of m - n
    dots = np.einsum("mhc,nhc->hmn", qr.reshape(40, 2, 32).astype(np.float64), kr.reshape(40, 2, 32).astype(np.float64))
    for h in range(2):
        for d in (-7, 0, 3, 19):
            diag = np.diagonal(dots[h], offset=-d)          # entries (m, n) with m - n = d
            np.testing.assert_allclose(diag, diag[0], rtol=0, atol=2e-5)
    assert np.abs(np.diagonal(dots[0], offset=-3)[0] - np.diagonal(dots[0], offset=0)[0]) > 1e-2   # ... and not constant


@pytest.mark.parametrize("program", PROGRAMS)
def test_rope_and_norm_against_a_complex_number_restatement(program):
    wl = WL.replace(grid=(23,), B=1, R=1)
    tab = gen.block_variants(wl, 5)
    q, k = _rows(3, n=23)
    pos = np.random.default_rng(4).permutation(23).astype(np.int32)
    if program == "dense":
        pos = np.arange(23, dtype=np.int32)                    # the whole-matrix program takes row t at position t
    got_q, got_k = oracle.qk_variants(q, k, 2, pos=pos if program == "regional" else None, q_norm_w=tab["q_norm_w"][1],
                                      k_norm_w=tab["k_norm_w"][1], qk_norm_eps=1e-6, rope_cos=tab["rope_cos"],
                                      rope_sin=tab["rope_sin"], program=program)
    phase = np.exp(1j * (np.arange(23)[:, None] * 10000.0 ** (-2.0 * np.arange(16) / 32)))[pos][:, None, :]

    def restate(x, gamma):
        x = torch.from_numpy(x).double().view(23, 2, 32)
        x = x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + 1e-6) * torch.from_numpy(gamma).double()
        z = torch.view_as_complex(x.view(23, 2, 16, 2).contiguous()) * torch.from_numpy(phase)
        return torch.view_as_real(z).reshape(23, 64).numpy()

    np.testing.assert_allclose(got_q, restate(q, tab["q_norm_w"][1]), rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(got_k, restate(k, tab["k_norm_w"][1]), rtol=1e-5, atol=1e-6)


def test_the_two_programs_agree_bit_for_bit_on_the_variants():
    wl = WL.replace(grid=(19,), B=1, R=1)
    tab = gen.block_variants(wl, 6)
    q, k = _rows(7, n=19)
    kw = dict(q_norm_w=tab["q_norm_w"][0], k_norm_w=tab["k_norm_w"][0], rope_cos=tab["rope_cos"], rope_sin=tab["rope_sin"])
    a = oracle.qk_variants(q, k, 2, program="regional", **kw)
    b = oracle.qk_variants(q, k, 2, program="dense", **kw)
    assert np.array_equal(a[0].view(np.uint32), b[0].view(np.uint32)) and np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))


@pytest.mark.parametrize("which", ["both", "norm", "rope"])
def test_all_active_equals_dense_bit_for_bit_with_variants(which):
    w = gen.block_weights(WL, 3)
    labels = gen.uniform_labels(WL)
    inp = gen.step_inputs(WL, 3, labels)
    var = gen.block_variants(WL, 3, qk_norm=which != "rope", rope=which != "norm")
    B, N, H = inp["x_cur"].shape
    y_d, kv_d = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads, variants=var)
    kv = np.full((WL.L, B, 2, N, H), np.nan, np.float32)
    y = np.full((B, N, H), np.nan, np.float32)
    oracle.regional_step(inp["x_cur"], inp["cond"], labels, np.ones((B, WL.R), np.uint8), w, kv, y, WL.heads, WL.R,
                         variants=var)
    assert np.array_equal(y.view(np.uint32), y_d.view(np.uint32))
    assert np.array_equal(kv.view(np.uint32), kv_d.view(np.uint32))
    y_plain, _ = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads)
    assert np.abs(y_plain - y_d).max() > 1e-5                  # the variants do change the result


def test_identity_tables_switch_the_variants_off_bit_for_bit():
    """Zero angles (cos 1, sin 0) rotate nothing: the block with such tables equals the block without RoPE."""
    w = gen.block_weights(WL, 4)
    inp = gen.step_inputs(WL, 4, gen.uniform_labels(WL))
    N, dh = WL.N, WL.head_dim
    ident = {"rope_cos": np.ones((N, dh // 2), np.float32), "rope_sin": np.zeros((N, dh // 2), np.float32)}
    a, kva = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads, variants=ident)
    b, kvb = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32)) and np.array_equal(kva.view(np.uint32), kvb.view(np.uint32))


def test_dense_block_with_variants_against_torch_fp64():
    """Library restatement of the whole block with QK-RMSNorm and RoPE (complex multiplication), weights scaled up so
    that the attention is far from uniform; the cached key must be the normed, rotated one."""
    w = gen.block_weights(WL, 7)
    inp = gen.step_inputs(WL, 7, gen.uniform_labels(WL))
    var = gen.block_variants(WL, 7)
    B, N, H = inp["x_cur"].shape
    heads, dh = WL.heads, WL.head_dim
    w = {k: (v * 8).astype(np.float32) for k, v in w.items()}
    y, kv = oracle.dense_block(inp["x_cur"], inp["cond"], w, 1, heads, variants=var)
    t = lambda a: torch.from_numpy(np.asarray(a)).double()
    x, cond = t(inp["x_cur"]), t(inp["cond"])
    mod = torch.nn.functional.silu(cond) @ t(w["w_ada"][1]).T + t(w["b_ada"][1])
    sh_a, sc_a, g_a, sh_m, sc_m, g_m = [c[:, None, :] for c in mod.chunk(6, dim=1)]
    xh = torch.nn.functional.layer_norm(x, (H,), eps=1e-6) * (1 + sc_a) + sh_a
    q, k, v = (xh @ t(w["w_qkv"][1]).T + t(w["b_qkv"][1])).chunk(3, dim=-1)
    phase = torch.polar(torch.ones(N, dh // 2, dtype=torch.float64),
                        torch.arange(N, dtype=torch.float64)[:, None] * 10000.0 ** (-2.0 * torch.arange(dh // 2, dtype=torch.float64) / dh))

    def variant(a, gamma):
        a = a.view(B, N, heads, dh)
        a = a * torch.rsqrt(a.pow(2).mean(-1, keepdim=True) + 1e-6) * t(gamma)
        z = torch.view_as_complex(a.view(B, N, heads, dh // 2, 2).contiguous()) * phase[None, :, None, :]
        return torch.view_as_real(z).reshape(B, N, H)

    q, k = variant(q, var["q_norm_w"][1]), variant(k, var["k_norm_w"][1])
    sp = lambda a: a.view(B, N, heads, dh).transpose(1, 2)
    s = sp(q) @ sp(k).transpose(-1, -2) / np.sqrt(dh)
    assert s.std() > 0.5
    o = (torch.softmax(s, dim=-1) @ sp(v)).transpose(1, 2).reshape(B, N, H)
    r1 = x + g_a * (o @ t(w["w_o"][1]).T + t(w["b_o"][1]))
    m = torch.nn.functional.layer_norm(r1, (H,), eps=1e-6) * (1 + sc_m) + sh_m
    hmid = torch.nn.functional.gelu(m @ t(w["w_fc1"][1]).T + t(w["b_fc1"][1]), approximate="tanh")
    r2 = r1 + g_m * (hmid @ t(w["w_fc2"][1]).T + t(w["b_fc2"][1]))
    np.testing.assert_allclose(y, r2.numpy(), rtol=2e-5, atol=2e-5)
    np.testing.assert_allclose(kv[:, 0], k.numpy(), rtol=1e-5, atol=1e-5)
    np.testing.assert_allclose(kv[:, 1], v.numpy(), rtol=1e-5, atol=1e-5)
