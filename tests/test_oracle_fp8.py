"""Pins for the FP8-operand variant of the block oracle: the two E4M3 quantisers (one arithmetic, one on the bit pattern)
against the format's definition, a library cast and each other; the 8-bit projection against exact cases and its error
bound; the two C block programs against each other and against a library restatement."""
import numpy as np
import pytest
import torch

import gen
import oracle

WL = gen.workload("tiny").replace(name="q", H=64, heads=2, head_dim=32, M=128, Hc=48, grid=(6, 8), B=2, R=6, D=8, L=2,
                                  labels="segments")


def _all_codes():
    """The 254 finite E4M3 values from the format's definition (sign, 4 exponent bits biased by 7, 3 mantissa bits;
    exponent field 0 is subnormal; 0x7f / 0xff are NaN)."""
    vals = []
    for code in range(256):
        if (code & 0x7f) == 0x7f:
            continue
        sgn = -1.0 if code & 0x80 else 1.0
        e, m = (code >> 3) & 0xf, code & 7
        vals.append(sgn * (m / 8.0 * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)))
    return np.array(sorted(set(vals)), np.float64)


@pytest.mark.parametrize("program", ["regional", "dense"])
def test_every_code_is_a_fixed_point_and_the_range_is_what_the_format_says(program):
    codes = _all_codes()
    assert codes.max() == 448.0 and np.abs(codes[codes != 0]).min() == 2.0 ** -9 and len(codes) == 253
    got = oracle.e4m3(codes.astype(np.float32), program)
    assert np.array_equal(got.astype(np.float64), codes)


@pytest.mark.parametrize("program", ["regional", "dense"])
def test_nearest_value_ties_to_even_and_saturation(program):
    codes = _all_codes()
    pos = codes[codes >= 0]
    mid = (pos[:-1] + pos[1:]) / 2                              # exactly representable in fp32
    got = oracle.e4m3(mid.astype(np.float32), program).astype(np.float64)
    # a tie goes to the neighbour whose mantissa (code) is even: codes alternate parity along the sorted values
    want = np.where(np.arange(len(mid)) % 2 == 0, pos[:-1], pos[1:])
    assert np.array_equal(got, want)
    assert np.array_equal(oracle.e4m3(-mid.astype(np.float32), program).astype(np.float64), -want)
    eps = np.float32(1e-3)
    below = oracle.e4m3((mid * (1 - eps)).astype(np.float32), program).astype(np.float64)
    above = oracle.e4m3((mid * (1 + eps)).astype(np.float32), program).astype(np.float64)
    assert np.array_equal(below, pos[:-1]) and np.array_equal(above, pos[1:])
    big = np.array([448.0, 449.0, 463.9, 464.0, 480.0, 1e4, 3e38, -500.0], np.float32)
    assert np.array_equal(oracle.e4m3(big, program), np.sign(big) * 448.0)


def test_quantisers_agree_with_each_other_and_with_the_library_cast():
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.standard_normal(200000) * s for s in (1e-3, 0.05, 1.0, 30.0, 150.0)]).astype(np.float32)
    x = np.concatenate([x, np.float32(2.0) ** rng.uniform(-12, 8.8, 100000).astype(np.float32)])
    a, b = oracle.e4m3(x, "regional"), oracle.e4m3(x, "dense")
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    inside = np.abs(x) <= 448
    lib = torch.from_numpy(x[inside]).to(torch.float8_e4m3fn).to(torch.float32).numpy()
    assert np.array_equal(a[inside], lib)
    # nearest: no representable value is closer
    codes = _all_codes()
    i = np.clip(np.searchsorted(codes, x.astype(np.float64)), 1, len(codes) - 1)
    best = np.minimum(np.abs(codes[i] - x), np.abs(codes[i - 1] - x))
    assert np.all(np.abs(a.astype(np.float64) - np.clip(x, -448, 448)) <= best + 1e-12)


def test_projection_is_exact_on_representable_operands():
    rng = np.random.default_rng(6)
    codes = _all_codes().astype(np.float32)
    small = codes[np.abs(codes) <= 8]
    K, O = 96, 40
    x8 = rng.choice(small, K)
    w8 = rng.choice(small, (O, K))
    s_w = rng.uniform(0.5, 2.0, O).astype(np.float32)
    bias = rng.standard_normal(O).astype(np.float32)
    a = np.float32(0.25)                                         # a power of two: x = a * x8 quantises back to x8 exactly
    y = oracle.linear_fp8(a * x8, float(a), w8, s_w, bias)
    want = (w8.astype(np.float64) @ x8.astype(np.float64)) * (np.float64(a) * s_w.astype(np.float64)) + bias
    assert np.array_equal(y, want.astype(np.float32))


def test_projection_error_stays_inside_the_rounding_bound():
    """|y - exact| <= sum_k |w_k| * |x_k - x8_k a| with |x_k - x8_k a| <= a * half a step of x8_k's binade (1/16 relative
    for normal values): the quantised weights are used as they are, so only the activation rounding contributes."""
    rng = np.random.default_rng(7)
    K, O = 256, 64
    x = rng.standard_normal(K).astype(np.float32) * 2
    w8 = oracle.e4m3(rng.standard_normal((O, K)).astype(np.float32) * 50)
    s_w = np.full(O, 0.01, np.float32)
    bias = np.zeros(O, np.float32)
    a = np.float32(0.03)
    y = oracle.linear_fp8(x, float(a), w8, s_w, bias).astype(np.float64)
    exact = (w8.astype(np.float64) * 0.01) @ x.astype(np.float64)
    step = np.maximum(np.abs(x.astype(np.float64)) / 16, a * 2.0 ** -10)
    bound = (np.abs(w8.astype(np.float64)) * 0.01) @ step
    err = np.abs(y - exact)
    assert np.all(err <= bound * 1.001 + 1e-6) and err.max() > 1e-4


def _setup(seed):
    w = gen.block_weights(WL, seed)
    labels = gen.uniform_labels(WL)
    inp = gen.step_inputs(WL, seed, labels)
    return w, labels, inp, {"fp8": gen.fp8_operands(WL, w, seed)}


def test_all_active_equals_dense_bit_for_bit_with_fp8_operands():
    w, labels, inp, var = _setup(4)
    B, N, H = inp["x_cur"].shape
    y_d, kv_d = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads, variants=var)
    kv = np.full((WL.L, B, 2, N, H), np.nan, np.float32)
    y = np.full((B, N, H), np.nan, np.float32)
    oracle.regional_step(inp["x_cur"], inp["cond"], labels, np.ones((B, WL.R), np.uint8), w, kv, y, WL.heads, WL.R, variants=var)
    assert np.array_equal(y.view(np.uint32), y_d.view(np.uint32)) and np.array_equal(kv.view(np.uint32), kv_d.view(np.uint32))
    y_s, _ = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL.heads)
    d = np.abs(y_s - y_d).max()
    assert 1e-4 < d < 0.2                                        # 8-bit operands move the result, a little


def test_dense_block_with_fp8_operands_against_torch_fp64():
    w, labels, inp, var = _setup(6)
    f = var["fp8"]
    B, N, H = inp["x_cur"].shape
    heads, dh = WL.heads, WL.head_dim
    y, kv = oracle.dense_block(inp["x_cur"], inp["cond"], w, 1, heads, variants=var)
    t = lambda a: torch.from_numpy(np.asarray(a)).double()

    def lin8(x, name, j):
        a = np.float32(f["a_scale"][1, j])
        xq = (x.float() * torch.tensor(np.float32(1.0) / a)).clamp(-448, 448).to(torch.float8_e4m3fn).double()
        return (xq @ t(f["w_" + name][1]).T) * (float(a) * t(f["s_" + name][1])) + t(w["b_" + name][1])

    x, cond = t(inp["x_cur"]), t(inp["cond"])
    mod = torch.nn.functional.silu(cond) @ t(w["w_ada"][1]).T + t(w["b_ada"][1])
    sh_a, sc_a, g_a, sh_m, sc_m, g_m = [ch[:, None, :] for ch in mod.chunk(6, dim=1)]
    xh = torch.nn.functional.layer_norm(x, (H,), eps=1e-6) * (1 + sc_a) + sh_a
    q, k, v = lin8(xh, "qkv", 0).chunk(3, dim=-1)
    sp = lambda a: a.reshape(B, -1, heads, dh).transpose(1, 2)
    o = torch.nn.functional.scaled_dot_product_attention(sp(q), sp(k), sp(v)).transpose(1, 2).reshape(B, N, H)
    r1 = x + g_a * (o @ t(w["w_o"][1]).T + t(w["b_o"][1]))
    m = torch.nn.functional.layer_norm(r1, (H,), eps=1e-6) * (1 + sc_m) + sh_m
    hmid = torch.nn.functional.gelu(lin8(m, "fc1", 1), approximate="tanh")
    r2 = r1 + g_m * lin8(hmid, "fc2", 2)
    # an activation that sits within an fp32 rounding of a quantisation tie may round the other way in the fp64
    # restatement: allow a handful of such elements, each worth one 8-bit step of one product
    err = np.abs(y - r2.numpy())
    assert np.quantile(err, 0.999) <= 2e-5 and err.max() <= 5e-3
    np.testing.assert_allclose(kv[:, 0], k.numpy(), rtol=0, atol=5e-3)
    assert np.quantile(np.abs(kv[:, 0] - k.numpy()), 0.999) <= 2e-5


# ---- FP8 operands with two streams: each stream has its own quantised weights and activation scales ----
WL2 = gen.workload("tiny").replace(name="q2", H=64, heads=2, head_dim=32, M=128, Hc=48, grid=(40,), n_text=8, B=2, R=5, D=8,
                                   L=2, labels="segments")


def _setup2(seed):
    w = gen.block_weights(WL2, seed)
    wt = gen.block_weights(WL2, seed + 100)
    labels = gen.uniform_labels(WL2)
    inp = gen.step_inputs(WL2, seed, labels)
    return w, wt, labels, inp


def test_same_fp8_operands_in_both_streams_is_the_single_stream_bit_for_bit():
    w, _, labels, inp = _setup2(8)
    f8 = gen.fp8_operands(WL2, w, 8)
    one = {"fp8": f8}
    two = {"fp8": f8, "text": {"weights": w, "n_text": WL2.n_text, "fp8": f8}}
    y1, kv1 = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL2.heads, variants=one)
    y2, kv2 = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL2.heads, variants=two)
    assert np.array_equal(y1.view(np.uint32), y2.view(np.uint32)) and np.array_equal(kv1.view(np.uint32), kv2.view(np.uint32))


def test_all_active_equals_dense_bit_for_bit_with_fp8_operands_in_two_streams():
    w, wt, labels, inp = _setup2(9)
    var = {"fp8": gen.fp8_operands(WL2, w, 9), "text": {"weights": wt, "n_text": WL2.n_text, "fp8": gen.fp8_operands(WL2, wt, 10)}}
    B, N, H = inp["x_cur"].shape
    y_d, kv_d = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL2.heads, variants=var)
    kv = np.full((WL2.L, B, 2, N, H), np.nan, np.float32)
    y = np.full((B, N, H), np.nan, np.float32)
    oracle.regional_step(inp["x_cur"], inp["cond"], labels, np.ones((B, WL2.R), np.uint8), w, kv, y, WL2.heads, WL2.R, variants=var)
    assert np.array_equal(y.view(np.uint32), y_d.view(np.uint32)) and np.array_equal(kv.view(np.uint32), kv_d.view(np.uint32))
    # the text rows really go through their own 8-bit operands: swapping the text stream's set changes them
    var2 = dict(var, text=dict(var["text"], fp8=gen.fp8_operands(WL2, wt, 11)))
    y_o, _ = oracle.dense_step(inp["x_cur"], inp["cond"], w, WL2.heads, variants=var2)
    assert np.abs(y_o - y_d)[:, WL2.n_grid:].max() > 1e-5


def test_one_streams_fp8_operands_without_the_others_are_refused():
    w, wt, labels, inp = _setup2(12)
    with pytest.raises(Exception):
        oracle.dense_step(inp["x_cur"], inp["cond"], w, WL2.heads,
                          variants={"fp8": gen.fp8_operands(WL2, w, 12), "text": {"weights": wt, "n_text": WL2.n_text}})
