"""GPU parity of the regional step against the oracle, element by element."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2607_12121_b200 as fd
from harness import StepBuffers, dev, gpu_step, host, labels_for, make_ctx, max_abs, rel_l2, tdtype

pytestmark = pytest.mark.gpu

BF16_MAX_ABS, BF16_REL_L2 = 3e-2, 1e-2      # bf16 block outputs vs the fp32 oracle
F32_MAX_ABS, F32_REL_L2 = 1e-4, 1e-5        # fp32 CUDA-core path vs the oracle


def _tol(wl):
    return (BF16_MAX_ABS, BF16_REL_L2) if wl.dtype == "bf16" else (F32_MAX_ABS, F32_REL_L2)


def _check_step(wl, y, kv, y_ref, kv_ref, y_before, kv_before, idx, widen=(0.0, 0.0), widen_kv=(0.0, 0.0)):
    """Active rows within tolerance; every other row of y and kv bit-identical to before.  `widen`, `widen_kv`: added to
    the (max-abs, relative-L2) bounds of y and of the cache rows (FP8 operands: a share of the change the 8-bit rounding
    itself makes)."""
    B, N, H = wl.B, wl.N, wl.H
    ma, rl = _tol(wl)
    ma_kv, rl_kv = ma + widen_kv[0], rl + widen_kv[1]
    ma, rl = ma + widen[0], rl + widen[1]
    act = np.zeros(B * N, bool)
    act[idx] = True
    yf, yr = y.reshape(B * N, H), y_ref.reshape(B * N, H)
    assert max_abs(yf[act], yr[act]) <= ma
    assert rel_l2(yf[act], yr[act]) <= rl
    assert np.array_equal(yf[~act], y_before.reshape(B * N, H)[~act])
    L = kv.shape[0]
    a2 = act.reshape(B, N)
    for l in range(L):
        for s in range(2):
            got, ref, old = kv[l][:, s], kv_ref[l][:, s], kv_before[l][:, s]
            assert max_abs(got[a2], ref[a2]) <= ma_kv
            assert rel_l2(got[a2], ref[a2]) <= rl_kv
            assert np.array_equal(got[~a2], old[~a2])


def _run_sequence(wl, seed, engine, masks, n_blocks=None, qk_gain=1.0, variants=None, text_seed=None, n_ctx=None,
                  fp8=False):
    """Warm-up (all active) on the previous step's tokens, then gated steps; both sides start
    from the same zero caches and carry their own state forward.  `variants`: inputs of the block variants
    (QK-RMSNorm weights, rotary tables) handed to both sides.  `text_seed`: dual stream, the always-active tokens
    (label R) get a second weight set drawn from this seed.  `n_ctx`: cross-attention to a context of that many tokens.
    `fp8`: the QKV, fc1 and fc2 projections take E4M3 operands quantised from the same weights."""
    L = wl.L if n_blocks is None else n_blocks
    labels = labels_for(wl, seed)
    w = gen.block_weights(wl, seed, n_blocks=L)
    if qk_gain != 1.0:          # a power of two keeps the weights exact in bf16
        w["w_qkv"][:, :wl.H] *= np.float32(qk_gain)       # query rows only: K/V keep their magnitude
        w["b_qkv"][:, :wl.H] *= np.float32(qk_gain)
    inp = gen.step_inputs(wl, seed, labels)
    ctx = make_ctx(wl, w, engine=engine, n_blocks=L)
    buf = StepBuffers(wl, L)
    dt = tdtype(wl)
    variants = dict(variants) if variants is not None else None
    if text_seed is not None:
        wt = gen.block_weights(wl, text_seed, n_blocks=L)
        if qk_gain != 1.0:
            wt["w_qkv"][:, :wl.H] *= np.float32(qk_gain)
            wt["b_qkv"][:, :wl.H] *= np.float32(qk_gain)
        fd.fd_set_text_stream(ctx, {k: dev(v[:L], dt) for k, v in wt.items()})
        text = {"weights": wt, "n_text": wl.n_text}
        if variants is not None and "q_norm_w" in variants:     # the second stream normalises with weights of its own
            tv = gen.block_variants(wl, text_seed, n_blocks=L, rope=False)
            text.update(q_norm_w=tv["q_norm_w"], k_norm_w=tv["k_norm_w"])
    if variants is not None:
        kw = {k: (dev(v, dt if k.endswith("_w") else None) if isinstance(v, np.ndarray) else v) for k, v in variants.items()}
        if text_seed is not None and "q_norm_w" in variants:
            kw.update(q_norm_w_text=dev(text["q_norm_w"], dt), k_norm_w_text=dev(text["k_norm_w"], dt))
        fd.fd_set_block_variants(ctx, **kw)
    if text_seed is not None:
        variants = dict(variants or {}, text=text)
    if n_ctx is not None:
        cross = gen.cross_attention(wl, seed, n_ctx, n_blocks=L)
        cross["w_q"] *= np.float32(qk_gain)
        cross["b_q"] *= np.float32(qk_gain)
        fd.fd_set_cross_attention(ctx, {k: dev(v, dt) for k, v in cross.items()})
        variants = dict(variants or {}, cross=cross)
    if fp8:
        f8 = gen.fp8_operands(wl, w, seed, n_blocks=L)
        fd.fd_set_fp8_operands(ctx, dict({"w8_" + k: dev(f8["c_" + k]) for k in ("qkv", "fc1", "fc2")},
                                         **{"s_" + k: dev(f8["s_" + k]) for k in ("qkv", "fc1", "fc2")}, a_scale=f8["a_scale"]))
        variants = dict(variants or {}, fp8=f8)
        if text_seed is not None:                                # the second stream quantises with operands of its own
            f8t = gen.fp8_operands(wl, wt, text_seed, n_blocks=L)
            fd.fd_set_fp8_operands(ctx, dict({"w8_" + k: dev(f8t["c_" + k]) for k in ("qkv", "fc1", "fc2")},
                                             **{"s_" + k: dev(f8t["s_" + k]) for k in ("qkv", "fc1", "fc2")},
                                             a_scale=f8t["a_scale"]), text_stream=True)
            variants["text"] = dict(variants["text"], fp8=f8t)
    B, N, H = wl.B, wl.N, wl.H
    kv_ref = np.zeros((L, B, 2, N, H), np.float32)
    y_ref = np.zeros((B, N, H), np.float32)
    rng = np.random.default_rng(seed)
    x_np = inp["x_prev"]
    for step, mask in enumerate(masks):
        if step == 1:
            x_np = inp["x_cur"]
        elif step > 1:
            x_np = (x_np + np.float32(0.01) * rng.standard_normal(x_np.shape).astype(np.float32))
            x_np = gen.round_bf16(x_np) if wl.dtype == "bf16" else x_np.astype(np.float32)
        y_before, kv_before = host(buf.y), host(buf.kv)
        idx, cu = gpu_step(ctx, wl, dev(x_np, dt), dev(inp["cond"], dt), dev(labels), dev(mask), buf)
        widen = widen_kv = (0.0, 0.0)
        if fp8:
            # Two E4M3 roundings sit between the attention branch and the block output, and a rounding turns a relative
            # difference d between the two sides' inputs into sqrt(d * step) of the value (a share d / step of the
            # values lands on the neighbouring code, a whole step away): the bf16 path's 1e-4 becomes 3e-3 after the
            # first and 1.6e-2 after the second, that is up to ~0.6 of the rounding noise the format itself adds.  So
            # the bounds widen by 0.6 of what FP8 changes in the oracle (same state, same inputs, operands unquantised).
            plain = {k: v for k, v in (variants or {}).items() if k != "fp8"}
            if "text" in plain:
                plain["text"] = {k: v for k, v in plain["text"].items() if k != "fp8"}
            kv_p, y_p = kv_ref.copy(), y_ref.copy()
            oracle.regional_step(x_np, inp["cond"], labels, mask, w, kv_p, y_p, wl.heads, wl.R, n_blocks=L, variants=plain or None)
        o_idx, o_cu = oracle.regional_step(x_np, inp["cond"], labels, mask, w, kv_ref, y_ref, wl.heads, wl.R,
                                           n_blocks=L, variants=variants)
        assert np.array_equal(idx, o_idx) and np.array_equal(cu, o_cu)
        if fp8:
            act = np.zeros(B * N, bool)
            act[idx] = True
            ya, yp = y_ref.reshape(B * N, H)[act], y_p.reshape(B * N, H)[act]
            widen = (0.6 * max_abs(ya, yp), 0.6 * rel_l2(yp, ya))
            sel = act.reshape(B, N)[:, None].repeat(2, 1)                    # [B, 2, N]: the fresh K and V rows
            widen_kv = (0.6 * max_abs(kv_ref[:, sel], kv_p[:, sel]), 0.6 * rel_l2(kv_p[:, sel], kv_ref[:, sel]))
        if variants and "q_norm_w" in variants and wl.dtype == "bf16":
            # Normalised keys are of order one with tails of 4-5: storing such a value in bf16 costs up to |k| 2^-9,
            # and where the variants run in a kernel of their own behind the projection the key is rounded twice
            # (before and after the normalisation), so the absolute bound carries 2 |k| 2^-9 of the largest stored key.
            widen_kv = (widen_kv[0] + float(np.abs(kv_ref).max()) * 2.0 ** -8, widen_kv[1])
        _check_step(wl, host(buf.y), host(buf.kv), y_ref, kv_ref, y_before, kv_before, idx, widen, widen_kv)
    return ctx


def test_tiny_fp32_eight_steps_fixed_schedule():
    wl = gen.workload("tiny")
    masks = gen.mask_schedule(wl, 0, 8)
    _run_sequence(wl, 0, fd.FD_ENGINE_SIMT, masks)


@pytest.mark.parametrize("name", ["audio_small", "image_small", "mmdit_small", "video_small"])
def test_small_twins_simt_engine(name):
    wl = gen.workload(name)
    masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 3, gen.request_fractions(wl, 3)),
             gen.region_mask(wl, 4, [0.34] * wl.B)]
    _run_sequence(wl, 2, fd.FD_ENGINE_SIMT, masks)


def test_all_active_step_equals_dense_oracle():
    wl = gen.workload("audio_small")
    labels = gen.uniform_labels(wl)
    w = gen.block_weights(wl, 6)
    inp = gen.step_inputs(wl, 6, labels)
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_SIMT)
    buf = StepBuffers(wl, wl.L)
    dt = tdtype(wl)
    gpu_step(ctx, wl, dev(inp["x_cur"], dt), dev(inp["cond"], dt), dev(labels), dev(np.ones((wl.B, wl.R), np.uint8)), buf)
    y_d, kv_d = oracle.dense_step(inp["x_cur"], inp["cond"], w, wl.heads)
    assert max_abs(host(buf.y), y_d) <= BF16_MAX_ABS and rel_l2(host(buf.y), y_d) <= BF16_REL_L2
    assert max_abs(host(buf.kv), kv_d) <= BF16_MAX_ABS and rel_l2(host(buf.kv), kv_d) <= BF16_REL_L2


def test_empty_mask_touches_nothing():
    wl = gen.workload("audio_small")
    labels = gen.uniform_labels(wl)
    w = gen.block_weights(wl, 8)
    inp = gen.step_inputs(wl, 8, labels)
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_SIMT)
    buf = StepBuffers(wl, wl.L)
    buf.y.fill_(1.5)
    buf.kv.fill_(-2.0)
    dt = tdtype(wl)
    idx, cu = gpu_step(ctx, wl, dev(inp["x_cur"], dt), dev(inp["cond"], dt), dev(labels),
                       dev(np.zeros((wl.B, wl.R), np.uint8)), buf)
    assert idx.size == 0 and not cu.any()
    assert (host(buf.y) == 1.5).all() and (host(buf.kv) == -2.0).all()


def test_host_side_argument_errors():
    wl = gen.workload("audio_small")
    w = gen.block_weights(wl, 1, n_blocks=1)
    ctx = make_ctx(wl, w, n_blocks=1, engine=fd.FD_ENGINE_SIMT)
    buf = StepBuffers(wl, 1)
    dt = tdtype(wl)
    x = torch.zeros((wl.B + 1, wl.N, wl.H), dtype=dt, device="cuda")
    with pytest.raises(fd.FlashDiffError) as ei:
        fd.fd_regional_step(ctx, x, x, x, x, wl.R, buf.kv, buf.y, buf.active_idx, buf.cu_active)
    assert ei.value.status == fd.FD_ERR_SHAPE
    # more regions than tokens; misaligned index arrays: refused on the host, nothing launched
    small = torch.zeros((1, 8, wl.H), dtype=dt, device="cuda")
    lab = torch.zeros((wl.B * wl.N + 1,), dtype=torch.int32, device="cuda")
    n0 = ctx.launches
    with pytest.raises(fd.FlashDiffError) as ei:
        fd.fd_regional_step(ctx, small, small, lab, lab, 9, buf.kv, buf.y, buf.active_idx, buf.cu_active)
    assert ei.value.status == fd.FD_ERR_SHAPE
    xs = torch.zeros((wl.B, wl.N, wl.H), dtype=dt, device="cuda")
    odd = lab.view(torch.uint8)[1:1 + 4 * wl.B * wl.N]          # an int32 array that starts on an odd byte
    for args in ((odd, buf.active_idx, buf.cu_active), (lab, odd, buf.cu_active), (lab, buf.active_idx, odd)):
        with pytest.raises(fd.FlashDiffError) as ei:
            fd.fd_regional_step(ctx, xs, xs, args[0], lab, wl.R, buf.kv, buf.y, args[1], args[2])
        assert ei.value.status == fd.FD_ERR_INVALID_ARG
    assert ctx.launches == n0
    assert fd.fd_destroy(ctx) == fd.FD_OK
    bad = fd.make_config(wl.replace(H=250))
    assert fd.fd_workspace_bytes(bad) == 0


@pytest.mark.parametrize("name", ["audio_tc", "mmdit_tc", "video_tc", "wide_tc", "image_tc"])
def test_small_twins_tensor_core_engine(name):
    wl = gen.workload(name)
    masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 3, gen.request_fractions(wl, 3)),
             gen.region_mask(wl, 4, [0.34] * wl.B)]
    _run_sequence(wl, 2, fd.FD_ENGINE_TC, masks)


@pytest.mark.parametrize("name,n_tok", [("audio_tc", None), ("audio_tc", 130), ("audio_tc", 100), ("image_tc", None),
                                        ("wide_tc", None), ("mmdit_tc", None), ("audio_tc", 520)])
def test_tensor_core_engine_few_ctas_walk_many_tiles(monkeypatch, name, n_tok):
    """Two persistent CTAs process every tile: the shared-memory rings and both TMEM accumulator
    stages wrap around many times, and every attention CTA runs many items back to back (with four, two
    and one key tiles per item: the hand-over of an item's statistics and accumulators to the epilogue
    warps, and of the score / P buffers between items, at every key-loop length).  Three and five key tiles per
    item: at head dim 64 the softmax warpgroups own the tiles of one parity of the CTA-wide tile counter, so the
    parity an item starts on alternates from item to item."""
    monkeypatch.setenv("FD_TC_MAX_CTAS", "2")
    wl = gen.workload(name)
    if n_tok is not None:
        wl = wl.replace(grid=(n_tok,), R=10, L=1)
    masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 5, [0.6] * wl.B)]
    _run_sequence(wl, 3, fd.FD_ENGINE_TC, masks)


@pytest.mark.parametrize("name,n_tok,max_ctas", [("audio_tc", None, None), ("audio_tc", 700, "8"), ("mmdit_tc", None, "8"),
                                                 ("image_tc", None, None), ("image_tc", 520, "8"), ("wide_tc", None, "8"),
                                                 ("audio_tc", 100, None)])
def test_attention_items_cut_along_the_keys(monkeypatch, name, n_tok, max_ctas):
    """The items of the last, partly filled round of attention CTAs are cut into pieces along the key sequence (forced
    here at every length; by default only long sequences are cut) and a second kernel puts the pieces together: with
    all SMs (every item is cut: fewer items than CTAs) and with 8 CTAs (whole rounds first, then 2 to 8 pieces per
    left-over item), pieces of one key tile (one softmax warpgroup idle at head dim 64) and of several."""
    monkeypatch.setenv("FD_ATT_SPLIT", "2")
    if max_ctas:
        monkeypatch.setenv("FD_TC_MAX_CTAS", max_ctas)
    wl = gen.workload(name)
    if n_tok is not None:
        wl = wl.replace(grid=(n_tok,), R=10, L=1)
    masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 6, [0.6] * wl.B)]
    cut = _run_sequence(wl, 4, fd.FD_ENGINE_TC, masks).launches
    monkeypatch.setenv("FD_ATT_SPLIT", "0")
    whole = _run_sequence(wl, 4, fd.FD_ENGINE_TC, masks).launches
    assert cut == whole + len(masks) * wl.L                     # the second kernel ran behind every attention launch


@pytest.mark.parametrize("switch", ["FD_TMA_RESID", "FD_TC_PAIR", "FD_PDL"])
def test_tensor_core_engine_switched_off_variants(monkeypatch, switch):
    """The library's switches select older forms of a kernel (per-thread residual reductions instead of the bulk
    tensor reduction, single-CTA instead of CTA-pair GEMM tiles, fully serialized launches); they stay correct."""
    monkeypatch.setenv(switch, "0")
    wl = gen.workload("mmdit_tc")
    masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 8, [0.5] * wl.B)]
    _run_sequence(wl, 6, fd.FD_ENGINE_TC, masks)


@pytest.mark.parametrize("name,engine,gain", [("audio_tc", fd.FD_ENGINE_TC, 64.0), ("video_tc", fd.FD_ENGINE_TC, 64.0),
                                              ("image_tc", fd.FD_ENGINE_TC, 16.0), ("audio_tc", fd.FD_ENGINE_SIMT, 64.0)])
def test_peaked_attention_exercises_running_max(name, engine, gain):
    """Query weights scaled up: scores spread over many e-folds, so the running maximum moves
    between key tiles and the accumulated output has to be rescaled.  (The image twin has the full hidden width
    1152, so its queries are larger to begin with: a gain of 16 gives it the score spread 64 gives the 256-wide
    twins; beyond that the softmax is one-hot and a bf16-rounded query flips near ties.)"""
    wl = gen.workload(name)
    masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 6, [0.5] * wl.B)]
    _run_sequence(wl, 4, engine, masks, qk_gain=gain)


@pytest.mark.parametrize("name,n_tok,max_ctas,gain", [("image_tc", 520, "8", 8.0), ("image_tc", None, None, 8.0),
                                                      ("audio_tc", 700, "8", 64.0), ("wide_tc", 520, "8", 16.0)])
def test_peaked_attention_with_items_cut_along_the_keys(monkeypatch, name, n_tok, max_ctas, gain):
    """Peaked softmax and forced key cuts together: the pieces of an item hold very different running maxima, so the
    second kernel's rescaling of every piece decides the result (head dims 72, 64 and 128)."""
    monkeypatch.setenv("FD_ATT_SPLIT", "2")
    if max_ctas:
        monkeypatch.setenv("FD_TC_MAX_CTAS", max_ctas)
    wl = gen.workload(name)
    if n_tok is not None:
        wl = wl.replace(grid=(n_tok,), R=10, L=1)
    masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 6, [0.6] * wl.B)]
    _run_sequence(wl, 4, fd.FD_ENGINE_TC, masks, qk_gain=gain)


def test_bounded_wait_reports_timeout_and_context_stays_usable():
    """A device-side wait that nothing satisfies gives up after its limit: the kernel returns, the status
    word says FD_ERR_TIMEOUT, and the same context then runs a normal step."""
    wl = gen.workload("audio_tc")
    labels = gen.uniform_labels(wl)
    w = gen.block_weights(wl, 9)
    inp = gen.step_inputs(wl, 9, labels)
    ctx = make_ctx(wl, w)
    fd.fd_selftest_bounded_wait(ctx)
    with pytest.raises(fd.FlashDiffError) as ei:
        fd.fd_poll_status(ctx)
    assert ei.value.status == fd.FD_ERR_TIMEOUT
    buf = StepBuffers(wl, wl.L)
    dt = tdtype(wl)
    idx, cu = gpu_step(ctx, wl, dev(inp["x_cur"], dt), dev(inp["cond"], dt), dev(labels),
                       dev(np.ones((wl.B, wl.R), np.uint8)), buf)
    assert idx.size == wl.B * wl.N
    y_d, _ = oracle.dense_step(inp["x_cur"], inp["cond"], w, wl.heads)
    assert max_abs(host(buf.y), y_d) <= BF16_MAX_ABS and rel_l2(host(buf.y), y_d) <= BF16_REL_L2


@pytest.mark.parametrize("n_tok,regions,heads,head_dim", [(40, 5, 4, 64), (64, 4, 4, 64), (130, 13, 4, 64),
                                                        (200, 8, 4, 64), (40, 5, 2, 128), (130, 13, 2, 128),
                                                        (1, 1, 4, 64)])
def test_tensor_core_engine_ragged_key_counts(n_tok, regions, heads, head_dim):
    """Key counts around the 128-key tile and its 64-key halves: a single partial tile, a tile whose second
    half has no valid key, a last tile with two keys, and a single token."""
    wl = gen.workload("audio_tc").replace(grid=(n_tok,), R=regions, B=2, heads=heads, head_dim=head_dim, L=1)
    masks = [np.ones((wl.B, wl.R), np.uint8)]
    if regions > 1:
        masks.append(gen.region_mask(wl, 7, [0.6, 0.4]))
    _run_sequence(wl, 5, fd.FD_ENGINE_TC, masks, qk_gain=16.0)


@pytest.mark.parametrize("case", ["twins", "ragged", "cut", "peaked", "few_ctas"])
def test_head_dim_128_on_cta_pairs(monkeypatch, case):
    """The CTA-pair attention kernel (two CTAs share every key tile through cta_group::2 products; switched on with
    FD_ATT_PAIR=1): the same parity cases as the single-CTA kernel, including items whose second CTA has few or no
    rows, a single token, forced key cuts with the pair combine kernel, and a peaked softmax."""
    monkeypatch.setenv("FD_ATT_PAIR", "1")
    if case == "twins":
        for name in ("video_tc", "wide_tc"):
            wl = gen.workload(name)
            masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 3, gen.request_fractions(wl, 3)),
                     gen.region_mask(wl, 4, [0.34] * wl.B)]
            n = _run_sequence(wl, 2, fd.FD_ENGINE_TC, masks).launches
        monkeypatch.setenv("FD_ATT_PAIR", "0")
        assert _run_sequence(wl, 2, fd.FD_ENGINE_TC, masks).launches == n      # same number of kernels either way
    elif case == "ragged":
        for n_tok, regions in ((40, 5), (130, 13), (300, 10), (1, 1)):
            wl = gen.workload("audio_tc").replace(grid=(n_tok,), R=regions, B=2, heads=2, head_dim=128, L=1)
            masks = [np.ones((wl.B, wl.R), np.uint8)]
            if regions > 1:
                masks.append(gen.region_mask(wl, 7, [0.6, 0.4]))
            _run_sequence(wl, 5, fd.FD_ENGINE_TC, masks, qk_gain=16.0)
    elif case == "cut":
        monkeypatch.setenv("FD_ATT_SPLIT", "2")
        for max_ctas in (None, "8"):
            if max_ctas:
                monkeypatch.setenv("FD_TC_MAX_CTAS", max_ctas)
            wl = gen.workload("wide_tc").replace(grid=(520,), R=10, L=1)
            masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 6, [0.6] * wl.B)]
            cut = _run_sequence(wl, 4, fd.FD_ENGINE_TC, masks, qk_gain=16.0).launches
        monkeypatch.setenv("FD_ATT_SPLIT", "0")
        whole = _run_sequence(wl, 4, fd.FD_ENGINE_TC, masks, qk_gain=16.0).launches
        assert cut == whole + len(masks) * wl.L                  # the pair combine kernel ran behind every attention launch
    elif case == "peaked":
        wl = gen.workload("video_tc")
        masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 6, [0.5] * wl.B)]
        _run_sequence(wl, 4, fd.FD_ENGINE_TC, masks, qk_gain=64.0)
    else:
        monkeypatch.setenv("FD_TC_MAX_CTAS", "2")                # one cluster walks every item: rings and barriers wrap many times
        wl = gen.workload("wide_tc").replace(grid=(700,), R=10, L=1)
        masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 5, [0.6] * wl.B)]
        _run_sequence(wl, 3, fd.FD_ENGINE_TC, masks)
