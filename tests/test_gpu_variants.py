"""GPU parity of the block variants (QK-RMSNorm, rotary position embedding) against the oracle: the normalised,
rotated keys in the cache, the block outputs, and skipped rows left bit-identical, on both engines and at every
head dim the tensor-core attention kernel has (64, 72 stored as 80, 128)."""
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


_CONFIGS = [("tiny", fd.FD_ENGINE_SIMT), ("audio_small", fd.FD_ENGINE_SIMT), ("image_small", fd.FD_ENGINE_SIMT),
            ("audio_tc", fd.FD_ENGINE_TC), ("image_tc", fd.FD_ENGINE_TC), ("wide_tc", fd.FD_ENGINE_TC),
            ("mmdit_tc", fd.FD_ENGINE_TC), ("video_tc", fd.FD_ENGINE_TC)]
# both variants together everywhere; each one alone on three configurations
_CASES = [(n, e, "both") for n, e in _CONFIGS] + [(n, e, w) for n, e in _CONFIGS if n in ("audio_small", "audio_tc", "image_tc")
                                                   for w in ("norm", "rope")]


@pytest.mark.parametrize("name,engine,which", _CASES)
def test_variants_match_the_oracle(name, engine, which):
    wl = gen.workload(name)
    var = gen.block_variants(wl, 9, qk_norm=which != "rope", rope=which != "norm")
    masks = _masks(wl) if name != "tiny" else list(gen.mask_schedule(wl, 0, 3))
    # larger query / key weights: the variants then change the attention visibly (weights stay exact in bf16)
    _run_sequence(wl, 2, engine, masks, qk_gain=4.0, variants=var)


@pytest.mark.parametrize("name", ["audio_tc", "wide_tc", "mmdit_tc"])
def test_variants_in_their_own_kernel_behind_the_projection(monkeypatch, name):
    """Head dims 64 and 128 normally get the variants inside the QKV epilogue; the separate kernel (what head dim 72 and
    the CUDA-core engine use) on the same shapes."""
    monkeypatch.setenv("FD_QK_FUSED", "0")
    wl = gen.workload(name)
    _run_sequence(wl, 7, fd.FD_ENGINE_TC, _masks(wl), qk_gain=4.0, variants=gen.block_variants(wl, 9))


def test_variants_can_be_switched_off_again_and_bad_arguments_are_refused():
    wl = gen.workload("audio_tc")
    w = gen.block_weights(wl, 2)
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_TC)
    var = gen.block_variants(wl, 9)
    qn = dev(var["q_norm_w"], torch.bfloat16)
    with pytest.raises(fd.FlashDiffError) as ei:
        fd.fd_set_block_variants(ctx, q_norm_w=qn)                       # key weights missing
    assert ei.value.status == fd.FD_ERR_INVALID_ARG
    with pytest.raises(fd.FlashDiffError) as ei:
        fd.fd_set_block_variants(ctx, rope_cos=dev(var["rope_cos"]))     # sine table missing
    assert ei.value.status == fd.FD_ERR_INVALID_ARG
    fd.fd_set_block_variants(ctx, q_norm_w=qn, k_norm_w=qn)
    fd.fd_set_block_variants(ctx)                                        # all off again
    assert fd.fd_destroy(ctx) == fd.FD_OK
    # with the variants off the plain parity run is what it was
    _run_sequence(wl, 2, fd.FD_ENGINE_TC, _masks(wl))
