"""Pins for the dual-stream form of the block oracle (joint text-image blocks: a token's stream selects the weights of
every per-token operation, the attention stays joint): reductions to the single-stream block, isolation properties the
structure implies, the two separately written C programs against each other, and a library restatement."""
import numpy as np
import pytest
import torch

import gen
import oracle

# 40 image tokens in 5 regions + 8 always-active text tokens (label R) at the end of every request
WL = gen.workload("tiny").replace(name="d", H=64, heads=2, head_dim=32, M=96, Hc=48, grid=(40,), n_text=8, B=2, R=5, D=8,
                                  L=2, labels="segments")


def _setup(seed):
    w = gen.block_weights(WL, seed)
    wt = gen.block_weights(WL, seed + 100)
    labels = gen.uniform_labels(WL)
    inp = gen.step_inputs(WL, seed, labels)
    return w, wt, labels, inp


def _dual(wt, **extra):
    return {"text": dict({"weights": wt, "n_text": WL.n_text}, **extra)}


def test_same_weights_in_both_streams_is_the_single_stream_block_bit_for_bit():
    w, _, labels, inp = _setup(1)
    y1, kv1 = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads)
    y2, kv2 = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads, variants=_dual(w))
    assert np.array_equal(y1.view(np.uint32), y2.view(np.uint32)) and np.array_equal(kv1.view(np.uint32), kv2.view(np.uint32))
    B, N, H = inp["x_cur"].shape
    mask = gen.region_mask(WL, 3, [0.6, 0.4])
    out = []
    for var in (None, _dual(w)):
        kv = kv1.copy()
        y = y1.copy()
        oracle.regional_step(inp["x_prev"], inp["cond"], labels, mask, w, kv, y, WL.heads, WL.R, variants=var)
        out.append((y, kv))
    assert np.array_equal(out[0][0].view(np.uint32), out[1][0].view(np.uint32))
    assert np.array_equal(out[0][1].view(np.uint32), out[1][1].view(np.uint32))


@pytest.mark.parametrize("with_variants", [False, True])
def test_all_active_equals_dense_bit_for_bit_with_two_streams(with_variants):
    w, wt, labels, inp = _setup(2)
    var = _dual(wt)
    if with_variants:
        var.update(gen.block_variants(WL, 2))
        var["text"].update({k: v for k, v in gen.block_variants(WL, 77, rope=False).items() if k.endswith("_w")})
    B, N, H = inp["x_cur"].shape
    y_d, kv_d = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads, variants=var)
    kv = np.full((WL.L, B, 2, N, H), np.nan, np.float32)
    y = np.full((B, N, H), np.nan, np.float32)
    oracle.regional_step(inp["x_cur"], inp["cond"], labels, np.ones((B, WL.R), np.uint8), w, kv, y, WL.heads, WL.R, variants=var)
    assert np.array_equal(y.view(np.uint32), y_d.view(np.uint32))
    assert np.array_equal(kv.view(np.uint32), kv_d.view(np.uint32))
    y_s, _ = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads)
    assert np.abs(y_s - y_d)[:, WL.n_grid:].max() > 1e-3          # the text rows really use other weights


def test_what_a_stream_can_and_cannot_see_of_the_other_within_one_block():
    """Inside one block a token's output depends on the other stream only through that stream's keys and values:
    changing the text stream's out-projection or MLP leaves every image row bit-identical (and vice versa), while
    changing its QKV projection moves the image rows too."""
    w, wt, labels, inp = _setup(4)
    x, cond = inp["x_cur"], inp["cond"]
    img = slice(0, WL.n_grid)
    txt = slice(WL.n_grid, WL.N)
    base, kv_base = oracle.dense_block(x, cond, w, 0, WL.heads, variants=_dual(wt))

    def bump(ws, keys):
        out = {k: v.copy() for k, v in ws.items()}
        for k in keys:
            out[k][0] = out[k][0] * np.float32(1.5) + np.float32(0.01)
        return out

    y, kv = oracle.dense_block(x, cond, w, 0, WL.heads, variants=_dual(bump(wt, ["w_o", "b_o", "w_fc1", "b_fc1", "w_fc2", "b_fc2"])))
    assert np.array_equal(y[:, img].view(np.uint32), base[:, img].view(np.uint32))
    assert np.array_equal(kv.view(np.uint32), kv_base.view(np.uint32))
    assert np.abs(y[:, txt] - base[:, txt]).max() > 1e-4
    y, kv = oracle.dense_block(x, cond, bump(w, ["w_o", "b_o", "w_fc1", "b_fc1", "w_fc2", "b_fc2"]), 0, WL.heads, variants=_dual(wt))
    assert np.array_equal(y[:, txt].view(np.uint32), base[:, txt].view(np.uint32))
    assert np.abs(y[:, img] - base[:, img]).max() > 1e-4
    y, kv = oracle.dense_block(x, cond, w, 0, WL.heads, variants=_dual(bump(wt, ["w_qkv", "b_qkv"])))
    assert np.array_equal(kv[:, :, img].view(np.uint32), kv_base[:, :, img].view(np.uint32))      # image K/V untouched
    assert np.abs(kv[:, :, txt] - kv_base[:, :, txt]).max() > 1e-4
    assert np.abs(y[:, img] - base[:, img]).max() > 1e-7                                            # ... but seen through attention


def test_no_text_tokens_means_one_stream():
    wl = WL.replace(n_text=0)
    w = gen.block_weights(wl, 5)
    wt = gen.block_weights(wl, 105)
    inp = gen.step_inputs(wl, 5, gen.uniform_labels(wl))
    a, kva = oracle.dense_step(inp["x_cur"], inp["cond"], w, wl.heads, variants={"text": {"weights": wt, "n_text": 0}})
    b, kvb = oracle.dense_step(inp["x_cur"], inp["cond"], w, wl.heads)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32)) and np.array_equal(kva.view(np.uint32), kvb.view(np.uint32))


def test_dual_stream_dense_block_against_torch_fp64():
    w, wt, labels, inp = _setup(6)
    w = {k: (v * 8).astype(np.float32) for k, v in w.items()}
    wt = {k: (v * 8).astype(np.float32) for k, v in wt.items()}
    B, N, H = inp["x_cur"].shape
    heads, dh, n_img = WL.heads, WL.head_dim, WL.n_grid
    y, kv = oracle.dense_block(inp["x_cur"], inp["cond"], w, 1, heads, variants=_dual(wt))
    t = lambda a: torch.from_numpy(np.asarray(a)).double()
    x, cond = t(inp["x_cur"]), t(inp["cond"])
    is_text = (torch.arange(N) >= n_img)[None, :, None]

    def per_stream(fn):                                   # evaluate with both weight sets on all rows, pick by stream
        return torch.where(is_text, fn(wt), fn(w))

    def mod_of(ws):
        return (torch.nn.functional.silu(cond) @ t(ws["w_ada"][1]).T + t(ws["b_ada"][1]))[:, None, :]

    chunk = lambda ws, i: mod_of(ws)[..., i * H:(i + 1) * H]
    ln = torch.nn.functional.layer_norm(x, (H,), eps=1e-6)
    qkv = per_stream(lambda ws: (ln * (1 + chunk(ws, 1)) + chunk(ws, 0)) @ t(ws["w_qkv"][1]).T + t(ws["b_qkv"][1]))
    q, k, v = qkv.chunk(3, dim=-1)
    sp = lambda a: a.view(B, N, heads, dh).transpose(1, 2)
    s = sp(q) @ sp(k).transpose(-1, -2) / np.sqrt(dh)
    assert s.std() > 0.5
    o = (torch.softmax(s, dim=-1) @ sp(v)).transpose(1, 2).reshape(B, N, H)
    r1 = x + per_stream(lambda ws: chunk(ws, 2) * (o @ t(ws["w_o"][1]).T + t(ws["b_o"][1])))
    ln2 = torch.nn.functional.layer_norm(r1, (H,), eps=1e-6)
    r2 = r1 + per_stream(lambda ws: chunk(ws, 5) * (torch.nn.functional.gelu(
        (ln2 * (1 + chunk(ws, 4)) + chunk(ws, 3)) @ t(ws["w_fc1"][1]).T + t(ws["b_fc1"][1]), approximate="tanh")
        @ t(ws["w_fc2"][1]).T + t(ws["b_fc2"][1])))
    np.testing.assert_allclose(y, r2.numpy(), rtol=2e-5, atol=2e-5)
    np.testing.assert_allclose(kv[:, 0], k.numpy(), rtol=1e-5, atol=1e-5)
    np.testing.assert_allclose(kv[:, 1], v.numpy(), rtol=1e-5, atol=1e-5)
