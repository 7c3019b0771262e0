"""GPU parity of the cross-attention variant (every block attends, between its self-attention update and its MLP, to a
fixed context whose keys and values the caller supplies) against the oracle: both engines, context lengths below one key
tile, ragged and spanning several tiles, alone and together with the other block variants and the dual stream."""
import numpy as np
import pytest
import torch

import gen
import paper_2607_12121_b200 as fd
from harness import StepBuffers, dev, gpu_step, make_ctx
from test_gpu_step import _run_sequence

pytestmark = pytest.mark.gpu


def _masks(wl):
    return [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 3, gen.request_fractions(wl, 3)),
            gen.region_mask(wl, 4, [0.34] * wl.B)]


@pytest.mark.parametrize("name,engine", [("tiny", fd.FD_ENGINE_SIMT), ("audio_small", fd.FD_ENGINE_SIMT),
                                         ("video_small", fd.FD_ENGINE_SIMT)])
@pytest.mark.parametrize("n_ctx", [1, 37])
def test_cross_attention_simt_engine(name, engine, n_ctx):
    wl = gen.workload(name)
    _run_sequence(wl, 2, engine, _masks(wl), n_ctx=n_ctx)


@pytest.mark.parametrize("name", ["audio_tc", "image_tc", "video_tc"])          # head dims 64, 72, 128
@pytest.mark.parametrize("n_ctx", [1, 77, 128, 300])
def test_cross_attention_tensor_core_engine(name, n_ctx):
    wl = gen.workload(name)
    _run_sequence(wl, 2, fd.FD_ENGINE_TC, _masks(wl), n_ctx=n_ctx, qk_gain=4.0)


def test_cross_attention_with_variants_and_dual_stream():
    wl = gen.workload("mmdit_tc")
    _run_sequence(wl, 3, fd.FD_ENGINE_TC, _masks(wl), n_ctx=226, variants=gen.block_variants(wl, 9), text_seed=77)


def test_cross_attention_few_ctas_and_single_cta_gemms(monkeypatch):
    monkeypatch.setenv("FD_TC_MAX_CTAS", "5")
    monkeypatch.setenv("FD_TC_PAIR", "0")
    wl = gen.workload("audio_tc")
    _run_sequence(wl, 4, fd.FD_ENGINE_TC, _masks(wl), n_ctx=150, qk_gain=4.0)


def test_cross_attention_argument_checks_and_switch_off():
    wl = gen.workload("audio_tc").replace(L=1)
    w = gen.block_weights(wl, 2)
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_TC)
    cross = {k: dev(v, torch.bfloat16) for k, v in gen.cross_attention(wl.replace(B=wl.B + 1), 5, 16).items()}
    with pytest.raises(fd.FlashDiffError):                      # more requests in the context than the engine holds
        fd.fd_set_cross_attention(ctx, cross)
    bad = dict(cross, ctx_kv=cross["ctx_kv"][:, :1].contiguous())
    fd.fd_set_cross_attention(ctx, bad)
    labels = gen.uniform_labels(wl)
    inp = gen.step_inputs(wl, 2, labels)
    buf = StepBuffers(wl, 1)
    if wl.B != 1:
        with pytest.raises(fd.FlashDiffError):                  # a step whose batch differs from the context's
            gpu_step(ctx, wl, dev(inp["x_cur"], torch.bfloat16), dev(inp["cond"], torch.bfloat16), dev(labels),
                     dev(np.ones((wl.B, wl.R), np.uint8)), buf)
    fd.fd_set_cross_attention(ctx, None)
    assert fd.fd_destroy(ctx) == fd.FD_OK
    _run_sequence(wl, 2, fd.FD_ENGINE_TC, _masks(wl))           # without it the block is what it was
