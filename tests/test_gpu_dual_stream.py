"""GPU parity of the dual-stream blocks (the always-active tokens with label R run through a second weight set,
the attention stays joint) against the oracle: both engines, with and without the other block variants, with row tiles
that hold both streams, only one of them, and requests whose image tokens are all skipped."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2607_12121_b200 as fd
from harness import dev, make_ctx
from test_gpu_step import _run_sequence

pytestmark = pytest.mark.gpu


def _masks(wl):
    return [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 3, gen.request_fractions(wl, 3)),
            gen.region_mask(wl, 4, [0.34] * wl.B)]


@pytest.mark.parametrize("name,engine", [("mmdit_small", fd.FD_ENGINE_SIMT), ("mmdit_tc", fd.FD_ENGINE_TC)])
@pytest.mark.parametrize("with_variants", [False, True])
def test_dual_stream_matches_the_oracle(name, engine, with_variants):
    wl = gen.workload(name)
    var = gen.block_variants(wl, 9) if with_variants else None
    _run_sequence(wl, 2, engine, _masks(wl), qk_gain=4.0, variants=var, text_seed=77)


@pytest.mark.parametrize("n_text,B", [(200, 3), (300, 2), (5, 4)])
def test_dual_stream_row_tile_lists(n_text, B):
    """Text segments longer than a row tile, shorter than one, and several requests per tile: the second launch of every
    projection walks exactly the tiles that hold text rows (a missed tile leaves rows unwritten, which the parity check
    sees: both sides start from zero caches)."""
    wl = gen.workload("mmdit_tc").replace(n_text=n_text, B=B, L=1)
    masks = [np.ones((wl.B, wl.R), np.uint8), gen.region_mask(wl, 5, [0.5] * wl.B), np.zeros((wl.B, wl.R), np.uint8)]
    _run_sequence(wl, 3, fd.FD_ENGINE_TC, masks, text_seed=78)


def test_dual_stream_grouped_launch_with_few_ctas(monkeypatch):
    monkeypatch.setenv("FD_TC_MAX_CTAS", "4")                  # two CTA pairs walk every tile of both groups in turn
    wl = gen.workload("mmdit_tc").replace(n_text=300, B=3)
    _run_sequence(wl, 8, fd.FD_ENGINE_TC, _masks(wl), variants=gen.block_variants(wl, 9), text_seed=83)


def test_dual_stream_as_two_launches_per_projection(monkeypatch):
    monkeypatch.setenv("FD_TC_GROUPED", "0")                   # not the grouped launch: one launch per stream
    wl = gen.workload("mmdit_tc")
    _run_sequence(wl, 5, fd.FD_ENGINE_TC, _masks(wl), variants=gen.block_variants(wl, 9), text_seed=81)


def test_dual_stream_with_single_cta_gemm_tiles(monkeypatch):
    monkeypatch.setenv("FD_TC_PAIR", "0")                      # the 128-row tile list
    wl = gen.workload("mmdit_tc").replace(L=1)
    _run_sequence(wl, 4, fd.FD_ENGINE_TC, _masks(wl), text_seed=79)


def test_text_stream_can_be_switched_off_again():
    wl = gen.workload("mmdit_tc").replace(L=1)
    w = gen.block_weights(wl, 2)
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_TC)
    wt = {k: dev(v, torch.bfloat16) for k, v in gen.block_weights(wl, 80).items()}
    fd.fd_set_text_stream(ctx, wt)
    fd.fd_set_text_stream(ctx, None)
    assert fd.fd_destroy(ctx) == fd.FD_OK
    _run_sequence(wl, 2, fd.FD_ENGINE_TC, _masks(wl))          # single stream is what it was
