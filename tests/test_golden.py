"""The oracle still gives the answers frozen under tests/golden/ (written by make_golden.py, which calls
only the oracle; the paper prints no worked example to store instead)."""
import os
import sys

import numpy as np

HERE = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
sys.path.insert(0, HERE)
import make_golden  # noqa: E402


def _load(name, dtype):
    return np.loadtxt(os.path.join(HERE, name), dtype=dtype, ndmin=2)


def test_partition_golden():
    labels, sizes = make_golden.partition_case()
    assert np.array_equal(labels, _load("partition_image_small_seed42_labels.txt", np.int64))
    assert np.array_equal(sizes, _load("partition_image_small_seed42_sizes.txt", np.int64))


def test_gate_golden():
    score, mask = make_golden.gate_case()
    np.testing.assert_allclose(score, _load("gate_audio_small_seed42_score.txt", np.float64), rtol=1e-7)
    assert np.array_equal(mask, _load("gate_audio_small_seed42_mask.txt", np.int64))
