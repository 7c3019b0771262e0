"""Pins for the cross-attention variant of the block oracle (between the self-attention update and the MLP every row
attends to a fixed context): closed forms, the two C programs against each other, and a library restatement."""
import numpy as np
import pytest
import torch

import gen
import oracle

WL = gen.workload("tiny").replace(name="x", H=64, heads=2, head_dim=32, M=96, Hc=48, grid=(6, 8), B=2, R=6, D=8, L=2,
                                  labels="segments")


def _setup(seed, n_ctx=11):
    w = gen.block_weights(WL, seed)
    labels = gen.uniform_labels(WL)
    inp = gen.step_inputs(WL, seed, labels)
    return w, labels, inp, {"cross": gen.cross_attention(WL, seed, n_ctx)}


def test_zero_out_projection_switches_it_off_bit_for_bit():
    w, labels, inp, var = _setup(1)
    var["cross"]["w_o"][:] = 0
    var["cross"]["b_o"][:] = 0
    a, kva = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads, variants=var)
    b, kvb = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32)) and np.array_equal(kva.view(np.uint32), kvb.view(np.uint32))


def test_one_context_token_adds_its_projected_value_to_every_row():
    """With a single context token the softmax is 1 whatever the query: the update is W_o v + b_o for every row, so
    with the MLP switched off (zero gate) and an identity-free check on the residual: y - y_without = W_o v + b_o."""
    w, labels, inp, var = _setup(2, n_ctx=1)
    H = WL.H
    w = {k: v.copy() for k, v in w.items()}
    for l in range(WL.L):               # MLP gate (chunk 5) off: the block output is r1 after the cross-attention
        w["w_ada"][l, 5 * H:6 * H] = 0
        w["b_ada"][l, 5 * H:6 * H] = 0
    y1, _ = oracle.dense_block(inp["x_cur"], inp["cond"], w, 0, WL.heads, variants=var)
    y0, _ = oracle.dense_block(inp["x_cur"], inp["cond"], w, 0, WL.heads)
    c = var["cross"]
    for b in range(WL.B):
        upd = c["w_o"][0].astype(np.float64) @ c["ctx_kv"][0, b, 1, 0].astype(np.float64) + c["b_o"][0]
        np.testing.assert_allclose(y1[b] - y0[b], np.broadcast_to(upd, y1[b].shape), rtol=1e-5, atol=2e-6)


def test_equal_context_keys_give_the_mean_context_value():
    w, labels, inp, var = _setup(3, n_ctx=7)
    H = WL.H
    c = var["cross"]
    c["ctx_kv"][:, :, 0] = c["ctx_kv"][:, :, 0, :1]              # all context keys of a request equal
    w = {k: v.copy() for k, v in w.items()}
    for l in range(WL.L):
        w["w_ada"][l, 5 * H:6 * H] = 0
        w["b_ada"][l, 5 * H:6 * H] = 0
    y1, _ = oracle.dense_block(inp["x_cur"], inp["cond"], w, 1, WL.heads, variants=var)
    y0, _ = oracle.dense_block(inp["x_cur"], inp["cond"], w, 1, WL.heads)
    for b in range(WL.B):
        upd = c["w_o"][1].astype(np.float64) @ c["ctx_kv"][1, b, 1].astype(np.float64).mean(0) + c["b_o"][1]
        np.testing.assert_allclose(y1[b] - y0[b], np.broadcast_to(upd, y1[b].shape), rtol=1e-5, atol=2e-6)


@pytest.mark.parametrize("n_ctx", [1, 11, 150])
def test_all_active_equals_dense_bit_for_bit_with_cross_attention(n_ctx):
    w, labels, inp, var = _setup(4, n_ctx=n_ctx)
    B, N, H = inp["x_cur"].shape
    y_d, kv_d = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads, variants=var)
    kv = np.full((WL.L, B, 2, N, H), np.nan, np.float32)
    y = np.full((B, N, H), np.nan, np.float32)
    oracle.regional_step(inp["x_cur"], inp["cond"], labels, np.ones((B, WL.R), np.uint8), w, kv, y, WL.heads, WL.R, variants=var)
    assert np.array_equal(y.view(np.uint32), y_d.view(np.uint32))
    assert np.array_equal(kv.view(np.uint32), kv_d.view(np.uint32))
    y_s, _ = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads)
    assert np.abs(y_s - y_d).max() > 1e-3


def test_skipped_rows_stay_untouched_with_cross_attention():
    w, labels, inp, var = _setup(5)
    y0, kv0 = oracle.dense_step(inp["x_prev"], inp["cond"], w, WL.heads, variants=var)
    mask = gen.region_mask(WL, 7, [0.5, 0.34])
    y, kv = y0.copy(), kv0.copy()
    idx, _ = oracle.regional_step(inp["x_cur"], inp["cond"], labels, mask, w, kv, y, WL.heads, WL.R, variants=var)
    act = np.zeros(WL.B * WL.N, bool)
    act[idx] = True
    act = act.reshape(WL.B, WL.N)
    assert np.array_equal(y[~act].view(np.uint32), y0[~act].view(np.uint32))
    for b in range(WL.B):
        assert np.array_equal(kv[:, b][:, :, ~act[b]].view(np.uint32), kv0[:, b][:, :, ~act[b]].view(np.uint32))
    assert np.abs(y[act] - y0[act]).max() > 1e-4


def test_dense_block_with_cross_attention_against_torch_fp64():
    w, labels, inp, var = _setup(6, n_ctx=13)
    w = {k: (v * 8).astype(np.float32) for k, v in w.items()}
    c = var["cross"]
    for k in ("w_q", "b_q", "w_o", "b_o"):
        c[k] = (c[k] * 8).astype(np.float32)
    B, N, H = inp["x_cur"].shape
    heads, dh = WL.heads, WL.head_dim
    y, kv = oracle.dense_block(inp["x_cur"], inp["cond"], w, 1, heads, variants=var)
    t = lambda a: torch.from_numpy(np.asarray(a)).double()
    x, cond = t(inp["x_cur"]), t(inp["cond"])
    mod = torch.nn.functional.silu(cond) @ t(w["w_ada"][1]).T + t(w["b_ada"][1])
    sh_a, sc_a, g_a, sh_m, sc_m, g_m = [ch[:, None, :] for ch in mod.chunk(6, dim=1)]
    xh = torch.nn.functional.layer_norm(x, (H,), eps=1e-6) * (1 + sc_a) + sh_a
    q, k, v = (xh @ t(w["w_qkv"][1]).T + t(w["b_qkv"][1])).chunk(3, dim=-1)
    sp = lambda a: a.view(B, -1, heads, dh).transpose(1, 2)
    o = torch.nn.functional.scaled_dot_product_attention(sp(q), sp(k), sp(v)).transpose(1, 2).reshape(B, N, H)
    r1 = x + g_a * (o @ t(w["w_o"][1]).T + t(w["b_o"][1]))
    qc = torch.nn.functional.layer_norm(r1, (H,), eps=1e-6) @ t(c["w_q"][1]).T + t(c["b_q"][1])
    kc, vc = t(c["ctx_kv"][1][:, 0]), t(c["ctx_kv"][1][:, 1])
    sc = sp(qc) @ sp(kc).transpose(-1, -2) / np.sqrt(dh)
    assert sc.std() > 0.3
    oc = (torch.softmax(sc, dim=-1) @ sp(vc)).transpose(1, 2).reshape(B, N, H)
    r1 = r1 + oc @ t(c["w_o"][1]).T + t(c["b_o"][1])
    m = torch.nn.functional.layer_norm(r1, (H,), eps=1e-6) * (1 + sc_m) + sh_m
    hmid = torch.nn.functional.gelu(m @ t(w["w_fc1"][1]).T + t(w["b_fc1"][1]), approximate="tanh")
    r2 = r1 + g_m * (hmid @ t(w["w_fc2"][1]).T + t(w["b_fc2"][1]))
    np.testing.assert_allclose(y, r2.numpy(), rtol=2e-5, atol=2e-5)
