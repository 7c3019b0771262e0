"""Writes the stored expected values under tests/golden/ by calling ONLY the CPU oracle.

The paper prints no worked numeric example for the gate or the partitioner, so there are no
paper values to store; these files freeze the oracle's own answers on two small seeded inputs so
that an accidental change of its arithmetic shows up as a diff.  Run from the repository root:

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import gen      # noqa: E402
import oracle   # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))


def partition_case():
    wl = gen.workload("image_small")
    amap = gen.saliency_map(wl, 42)
    labels, sizes = oracle.partition(amap, None, wl.R, wl.m_min, wl.m_max)
    return labels, sizes


def gate_case():
    wl = gen.workload("audio_small")
    labels = gen.uniform_labels(wl)
    lat = gen.latent_pair(wl, 42, labels, fractions=[0.25, 0.5, 0.75])
    st = oracle.initial_state(wl.B, wl.R)
    score, weight, mask = oracle.activity_gate(lat["z_cur"], lat["z_prev"], labels, lat["eps"], st, wl.R)
    return score, mask


def main():
    labels, sizes = partition_case()
    np.savetxt(os.path.join(HERE, "partition_image_small_seed42_labels.txt"), labels, fmt="%d",
               header="oracle.partition on gen.saliency_map(image_small, 42): labels [B,N] (paper Sec. 4.1, Appendix A.3)")
    np.savetxt(os.path.join(HERE, "partition_image_small_seed42_sizes.txt"), sizes, fmt="%d",
               header="region sizes [B,R] of the same case")
    score, mask = gate_case()
    np.savetxt(os.path.join(HERE, "gate_audio_small_seed42_score.txt"), score, fmt="%.9e",
               header="oracle.activity_gate on gen.latent_pair(audio_small, 42, fractions 0.25/0.5/0.75): RMS change per region [B,R] (paper Sec. 4.2, Appendix A.1)")
    np.savetxt(os.path.join(HERE, "gate_audio_small_seed42_mask.txt"), mask, fmt="%d",
               header="active-region mask [B,R] of the same case")


if __name__ == "__main__":
    main()
