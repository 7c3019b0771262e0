"""GPU parity of the partitioner: region labels bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2607_12121_b200 as fd
from harness import dev, host, make_ctx

pytestmark = pytest.mark.gpu


def _ctx_for(B, N, R):
    wl = gen.workload("tiny").replace(B=B, grid=(N,), R=R, H=64, heads=1, head_dim=64, M=64, Hc=64, L=1)
    return make_ctx(wl, gen.block_weights(wl, 0), engine=fd.FD_ENGINE_SIMT)


def _gpu_partition(amap, R, m_min, m_max, cols=None):
    B, N, T = amap.shape
    ctx = _ctx_for(B, N, R)
    labels = torch.full((B, N), -1, dtype=torch.int32, device="cuda")
    sizes = torch.full((B, R), -1, dtype=torch.int32, device="cuda")
    fd.fd_partition_regions(ctx, dev(amap), R, labels, sizes, None if cols is None else dev(cols), m_min, m_max)
    fd.fd_poll_status(ctx)
    return host(labels), host(sizes)


@pytest.mark.parametrize("name", ["image_small", "mmdit_small", "video_small", "image", "mmdit"])
def test_partition_labels_bit_exact(name):
    wl = gen.workload(name)
    amap = gen.saliency_map(wl, 7)
    o_lab, o_sizes = oracle.partition(amap, None, wl.R, wl.m_min, wl.m_max)
    lab, sizes = _gpu_partition(amap, wl.R, wl.m_min, wl.m_max)
    assert np.array_equal(lab, o_lab)
    assert np.array_equal(sizes, o_sizes)


def test_partition_video_full_size():
    wl = gen.workload("video")
    amap = gen.saliency_map(wl, 3)
    o_lab, o_sizes = oracle.partition(amap, None, wl.R, wl.m_min, wl.m_max)
    lab, sizes = _gpu_partition(amap, wl.R, wl.m_min, wl.m_max)
    assert np.array_equal(lab, o_lab)
    assert np.array_equal(sizes, o_sizes)
    assert sizes.min() >= wl.m_min and sizes.max() <= wl.m_max


def test_partition_unbounded_salient_columns_and_fallbacks():
    rng = np.random.default_rng(5)
    # several columns, a subset of them salient
    amap = rng.random((2, 333, 7)).astype(np.float32)
    cols = np.array([5, 0, 3], np.int32)
    o_lab, o_sizes = oracle.partition(amap, cols, 9)
    lab, sizes = _gpu_partition(amap, 9, 1, 0, cols)
    assert np.array_equal(lab, o_lab) and np.array_equal(sizes, o_sizes)
    # constant map: no threshold exists, the fallback chops in token order
    amap = np.full((1, 50, 1), 0.25, np.float32)
    o_lab, _ = oracle.partition(amap, None, 7)
    lab, _ = _gpu_partition(amap, 7, 1, 0)
    assert np.array_equal(lab, o_lab)
    # few distinct levels with many ties, and bounds that force fallbacks deeper in the tree
    amap = (rng.integers(0, 4, size=(2, 200, 1)) / 4.0).astype(np.float32)
    o_lab, _ = oracle.partition(amap, None, 16, 4, 40)
    lab, _ = _gpu_partition(amap, 16, 4, 40)
    assert np.array_equal(lab, o_lab)
    # R = 1 and R = N
    amap = rng.random((1, 40, 1)).astype(np.float32)
    for R in (1, 40):
        o_lab, _ = oracle.partition(amap, None, R)
        lab, _ = _gpu_partition(amap, R, 1, 0)
        assert np.array_equal(lab, o_lab)


def test_partition_argument_errors():
    ctx = _ctx_for(1, 64, 8)
    amap = torch.zeros((1, 64, 1), dtype=torch.float32, device="cuda")
    labels = torch.zeros((1, 64), dtype=torch.int32, device="cuda")
    with pytest.raises(fd.FlashDiffError) as ei:
        fd.fd_partition_regions(ctx, amap, 9, labels)          # R beyond max_regions
    assert ei.value.status == fd.FD_ERR_SHAPE
