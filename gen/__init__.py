"""Seeded synthetic inputs for the region-selective DiT step.

This package only *draws inputs* (weights, latents, saliency maps, masks,
uniform label grids).  It holds none of the method's arithmetic: no activity
score, no gate, no partition rule, no transformer math.  Both the CPU oracle's
tests and the CUDA library's tests/bench feed from here, so the two sides see
identical arrays without sharing any code of the method itself.
"""
from .workloads import (  # noqa: F401
    Workload, WORKLOADS, workload, round_bf16, block_weights, step_inputs,
    uniform_labels, latent_pair, saliency_map, region_mask, mask_schedule,
    region_sigma, request_fractions, sampler_weights, latent_sequence, block_variants, cross_attention, fp8_operands,
)
