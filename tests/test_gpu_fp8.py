"""GPU parity of the FP8-operand variant (QKV, fc1 and fc2 with E4M3 weights and activations, fp32 accumulation) against
the oracle, which quantises the same way: every head dim and tile width of the tensor-core engine, alone and with the
other block variants and the cross-attention, few CTAs, and the argument checks."""
import numpy as np
import pytest
import torch

import gen
import paper_2607_12121_b200 as fd
import oracle
from harness import StepBuffers, dev, gpu_step, host, labels_for, make_ctx, max_abs, rel_l2
from test_gpu_step import _run_sequence

pytestmark = pytest.mark.gpu


def _masks(wl):
    return [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 3, gen.request_fractions(wl, 3)),
            gen.region_mask(wl, 4, [0.34] * wl.B)]


@pytest.mark.parametrize("name", ["audio_tc", "image_tc", "video_tc", "wide_tc"])
def test_fp8_operands_match_the_oracle(name):
    wl = gen.workload(name)
    if wl.M % 192 and wl.M % 256:
        wl = wl.replace(M=768)                                   # the 8-bit kernels take 192- or 256-wide tiles
    _run_sequence(wl, 2, fd.FD_ENGINE_TC, _masks(wl), fp8=True)


def _buffer(ctx, which, dtype, cols, rows):
    ptr, nbytes = fd.fd_debug_buffer(ctx, which)
    off = ptr - ctx.workspace.data_ptr()
    flat = ctx.workspace[off:off + nbytes].view(dtype)
    return flat[:rows * cols].view(rows, cols)


def _codes_close(got, want, max_fraction):
    """E4M3 codes equal, except for a small share of values that sat within a rounding of a tie and landed on the
    neighbouring code (same sign, or the two zeros)."""
    diff = got != want
    assert diff.mean() <= max_fraction, diff.mean()
    g, w = got[diff].astype(np.int32), want[diff].astype(np.int32)
    near = (np.abs(g - w) == 1) | ((g & 0x7f) + (w & 0x7f) <= 1)
    assert near.all()


def _stage_workload(name):
    if name == "audio_width":                   # the audio configuration's width (hidden 1536, MLP 6144), 384 tokens
        return gen.workload("audio").replace(name=name, L=1, B=1, grid=(384,), R=24)
    if name == "video_width":                   # the video configuration's width (12 heads of 128, MLP 8960), 384 tokens
        return gen.workload("audio").replace(name=name, L=1, B=1, grid=(384,), R=24, heads=12, head_dim=128, M=8960)
    return gen.workload(name).replace(L=1)


@pytest.mark.parametrize("name", ["image_tc", "wide_tc", "audio_tc", "audio_width", "video_width"])
def test_fp8_projections_stage_by_stage(name):
    """One block, every row active, attention gate zero (the residual entering the MLP branch is then the block's input
    exactly): each 8-bit projection is checked against exact arithmetic on the library's own quantised operands, read
    from the step's intermediate buffers, so that no rounding decision taken upstream blurs the comparison."""
    wl = _stage_workload(name)
    seed = 11
    H, M = wl.H, wl.M
    labels = labels_for(wl, seed)
    w = {k: v.copy() for k, v in gen.block_weights(wl, seed, n_blocks=1).items()}
    w["w_ada"][0, 2 * H:3 * H] = 0
    w["b_ada"][0, 2 * H:3 * H] = 0
    inp = gen.step_inputs(wl, seed, labels)
    f8 = gen.fp8_operands(wl, w, seed, n_blocks=1)
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_TC, n_blocks=1)
    fd.fd_set_fp8_operands(ctx, dict({"w8_" + k: dev(f8["c_" + k]) for k in ("qkv", "fc1", "fc2")},
                                     **{"s_" + k: dev(f8["s_" + k]) for k in ("qkv", "fc1", "fc2")}, a_scale=f8["a_scale"]))
    buf = StepBuffers(wl, 1)
    mask = np.ones((wl.B, wl.R), np.uint8)
    idx, _ = gpu_step(ctx, wl, dev(inp["x_cur"], torch.bfloat16), dev(inp["cond"], torch.bfloat16), dev(labels), dev(mask), buf)
    rows = wl.B * wl.N
    assert np.array_equal(idx, np.arange(rows))
    m8 = _buffer(ctx, fd.FD_BUF_ACT, torch.uint8, H, rows)
    g8 = _buffer(ctx, fd.FD_BUF_HIDDEN, torch.uint8, M, rows)
    r2 = _buffer(ctx, fd.FD_BUF_RESID, torch.float32, H, rows).cpu().numpy()
    dec = lambda t: t.view(torch.float8_e4m3fn).to(torch.float64).cpu().numpy()
    a_qkv, a_fc1, a_fc2 = (np.float32(v) for v in f8["a_scale"][0])

    # QKV: the cache rows come straight out of the first 8-bit projection, whose input both sides quantise from the same values
    kv_ref = np.zeros((1, wl.B, 2, wl.N, H), np.float32)
    y_ref = np.zeros((wl.B, wl.N, H), np.float32)
    oracle.regional_step(inp["x_cur"], inp["cond"], labels, mask, w, kv_ref, y_ref, wl.heads, wl.R, n_blocks=1, variants={"fp8": f8})
    assert rel_l2(host(buf.kv), kv_ref) <= 2.5e-3 and max_abs(host(buf.kv), kv_ref) <= 3e-2        # bf16 storage of K and V

    # the MLP branch's input: LayerNorm of the block input, modulated, quantised
    x = inp["x_cur"].reshape(rows, H).astype(np.float64)
    cond = inp["cond"].astype(np.float64)
    mod = (cond / (1 + np.exp(-cond))) @ w["w_ada"][0].astype(np.float64).T + w["b_ada"][0]
    mod_r = np.repeat(mod, wl.N, axis=0)
    xn = (x - x.mean(1, keepdims=True)) / np.sqrt(x.var(1, keepdims=True) + 1e-6)
    m = (xn * (1 + mod_r[:, 4 * H:5 * H]) + mod_r[:, 3 * H:4 * H]).astype(np.float32)
    want = torch.from_numpy(oracle.e4m3(m * (np.float32(1) / a_fc1))).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    _codes_close(m8.cpu().numpy(), want, 2e-3)

    # fc1 + GELU on the library's own quantised input
    h = (dec(m8) @ f8["w_fc1"][0].astype(np.float64).T) * (np.float64(a_fc1) * f8["s_fc1"][0]) + w["b_fc1"][0]
    g = (0.5 * h * (1 + np.tanh(0.79788456080286535588 * (h + 0.044715 * h ** 3)))).astype(np.float32)
    want = torch.from_numpy(oracle.e4m3(g * (np.float32(1) / a_fc2))).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    _codes_close(g8.cpu().numpy(), want, 2e-2)

    # fc2 + gated residual on the library's own quantised hidden activations
    f = (dec(g8) @ f8["w_fc2"][0].astype(np.float64).T) * (np.float64(a_fc2) * f8["s_fc2"][0]) + w["b_fc2"][0]
    want = x + mod_r[:, 5 * H:6 * H] * f
    assert rel_l2(r2, want) <= 1e-5 and max_abs(r2, want) <= 2e-4
    assert fd.fd_destroy(ctx) == fd.FD_OK


def test_fp8_operands_with_variants_and_cross_attention():
    wl = gen.workload("audio_tc")
    _run_sequence(wl, 3, fd.FD_ENGINE_TC, _masks(wl), fp8=True, variants=gen.block_variants(wl, 9), n_ctx=77, qk_gain=4.0)


@pytest.mark.parametrize("n_text,B", [(154, 2), (300, 2), (5, 4)])
def test_fp8_operands_with_two_streams(n_text, B):
    """Each stream with its own 8-bit weights and activation scales; text segments shorter and longer than a row tile,
    several requests per tile."""
    wl = gen.workload("mmdit_tc").replace(n_text=n_text, B=B)
    _run_sequence(wl, 6, fd.FD_ENGINE_TC, _masks(wl), fp8=True, text_seed=91)


def test_fp8_operands_few_ctas(monkeypatch):
    monkeypatch.setenv("FD_TC_MAX_CTAS", "6")                  # every CTA pair walks many tiles: rings and accumulators wrap
    wl = gen.workload("audio_tc")
    _run_sequence(wl, 4, fd.FD_ENGINE_TC, _masks(wl), fp8=True)


def test_fp8_operands_without_the_bulk_residual_reduction(monkeypatch):
    monkeypatch.setenv("FD_TMA_RESID", "0")
    wl = gen.workload("audio_tc")
    _run_sequence(wl, 5, fd.FD_ENGINE_TC, _masks(wl), fp8=True)


def test_fp8_argument_checks_and_switch_off(monkeypatch):
    wl = gen.workload("audio_tc").replace(L=1)
    w = gen.block_weights(wl, 2)
    f8 = gen.fp8_operands(wl, w, 2)
    args = dict({"w8_" + k: dev(f8["c_" + k]) for k in ("qkv", "fc1", "fc2")},
                **{"s_" + k: dev(f8["s_" + k]) for k in ("qkv", "fc1", "fc2")}, a_scale=f8["a_scale"])
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_SIMT)
    with pytest.raises(fd.FlashDiffError) as ei:                # CUDA-core engine: refused
        fd.fd_set_fp8_operands(ctx, args)
    assert ei.value.status == fd.FD_ERR_UNSUPPORTED
    fd.fd_destroy(ctx)
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_TC)
    with pytest.raises(fd.FlashDiffError):                      # a non-positive activation scale
        fd.fd_set_fp8_operands(ctx, dict(args, a_scale=np.zeros_like(f8["a_scale"])))
    fd.fd_set_text_stream(ctx, {k: dev(v, torch.bfloat16) for k, v in gen.block_weights(wl, 80).items()})
    fd.fd_set_fp8_operands(ctx, args)
    labels = gen.uniform_labels(wl)
    inp = gen.step_inputs(wl, 2, labels)
    buf = StepBuffers(wl, 1)
    with pytest.raises(fd.FlashDiffError) as ei:                # a second stream without 8-bit operands of its own
        gpu_step(ctx, wl, dev(inp["x_cur"], torch.bfloat16), dev(inp["cond"], torch.bfloat16), dev(labels),
                 dev(np.ones((wl.B, wl.R), np.uint8)), buf)
    assert ei.value.status == fd.FD_ERR_UNSUPPORTED
    fd.fd_set_fp8_operands(ctx, args, text_stream=True)
    gpu_step(ctx, wl, dev(inp["x_cur"], torch.bfloat16), dev(inp["cond"], torch.bfloat16), dev(labels),
             dev(np.ones((wl.B, wl.R), np.uint8)), buf)
    fd.fd_set_fp8_operands(ctx, None, text_stream=True)
    fd.fd_set_text_stream(ctx, None)
    fd.fd_set_fp8_operands(ctx, None)
    assert fd.fd_destroy(ctx) == fd.FD_OK
    _run_sequence(wl, 2, fd.FD_ENGINE_TC, _masks(wl))           # without it the block is what it was
    monkeypatch.setenv("FD_TC_PAIR", "0")                       # the single-CTA kernels have no 8-bit form: refused
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_TC)
    with pytest.raises(fd.FlashDiffError) as ei:
        fd.fd_set_fp8_operands(ctx, args)
    assert ei.value.status == fd.FD_ERR_UNSUPPORTED


def test_empty_mask_with_fp8_operands_and_variants_touches_nothing():
    """No active row at all (device-side row count zero): every kernel of the step, the 8-bit projections and the
    fused variants included, finds nothing to do and leaves y and the cache as they were."""
    wl = gen.workload("audio_tc")
    labels = gen.uniform_labels(wl)
    w = gen.block_weights(wl, 8)
    inp = gen.step_inputs(wl, 8, labels)
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_TC)
    f8 = gen.fp8_operands(wl, w, 8)
    fd.fd_set_fp8_operands(ctx, dict({"w8_" + k: dev(f8["c_" + k]) for k in ("qkv", "fc1", "fc2")},
                                     **{"s_" + k: dev(f8["s_" + k]) for k in ("qkv", "fc1", "fc2")}, a_scale=f8["a_scale"]))
    var = gen.block_variants(wl, 9)
    fd.fd_set_block_variants(ctx, **{k: (dev(v, torch.bfloat16 if k.endswith("_w") else None) if isinstance(v, np.ndarray) else v)
                                     for k, v in var.items()})
    buf = StepBuffers(wl, wl.L)
    buf.y.fill_(1.5)
    buf.kv.fill_(-2.0)
    idx, cu = gpu_step(ctx, wl, dev(inp["x_cur"], torch.bfloat16), dev(inp["cond"], torch.bfloat16), dev(labels),
                       dev(np.zeros((wl.B, wl.R), np.uint8)), buf)
    assert idx.size == 0 and not cu.any()
    assert (host(buf.y) == 1.5).all() and (host(buf.kv) == -2.0).all()
    assert fd.fd_destroy(ctx) == fd.FD_OK
