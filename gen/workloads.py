"""Workload shapes and seeded input draws.

Shapes follow the five benchmark configurations (tiny fp32 block, 1-D audio
latent, DiT-XL/2 image, 1024px joint text-image, 480p video).  Everything is
drawn from ``numpy.random.Generator(PCG64)`` with explicit seeds.  Nothing in
this file evaluates the method: thresholds handed to the gate are derived from
the generator's own noise scales, never from a computed score.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, Optional, Sequence, Tuple

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str                 # "f32" | "bf16": storage type of weights/activations
    L: int                     # transformer blocks
    H: int                     # hidden width
    heads: int
    head_dim: int
    M: int                     # MLP width
    Hc: int                    # conditioning width
    grid: Tuple[int, ...]      # latent token grid (product = image/audio/video tokens)
    n_text: int                # always-active tokens appended after the grid tokens
    B: int                     # concurrent requests
    R: int                     # regions per request
    D: int                     # latent channels per token seen by the gate
    labels: str                # "blocks2d" | "segments" | "partition"
    n_cells: int = 0           # Voronoi cells of the synthetic saliency map
    t_group: int = 0           # frames per temporal group (3-D maps only)
    m_min: int = 1             # region size bounds handed to the partitioner
    m_max: int = 0             # 0 = unbounded (N)

    @property
    def n_grid(self) -> int:
        return int(np.prod(self.grid))

    @property
    def N(self) -> int:
        return self.n_grid + self.n_text

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


WORKLOADS: Dict[str, Workload] = {
    # config 0: tiny fp32 block, 16x16 patches, 16 regions of 4x4 patches
    "tiny": Workload("tiny", "f32", 1, 256, 4, 64, 1024, 256, (16, 16), 0, 1, 16, 256, "blocks2d"),
    # config 1: audio latent, 1024 tokens x 64 channels, 16-token segments, 8 ragged requests
    "audio": Workload("audio", "bf16", 24, 1536, 24, 64, 6144, 1536, (1024,), 0, 8, 64, 64, "segments"),
    # config 2: DiT-XL/2 image, 32x32 tokens, 64 irregular regions of 8..32 tokens
    "image": Workload("image", "bf16", 28, 1152, 16, 72, 4608, 1152, (32, 32), 0, 4, 64, 16,
                      "partition", n_cells=64, m_min=8, m_max=32),
    # config 3: joint text-image at 1024px, 64x64 image tokens + 154 text tokens
    "mmdit": Workload("mmdit", "bf16", 24, 1536, 24, 64, 6144, 1536, (64, 64), 154, 2, 128, 64,
                      "partition", n_cells=128, m_min=8, m_max=128),
    # config 4: 480p video, 21 x 30 x 52 tokens, 256 spatio-temporal tubes
    "video": Workload("video", "bf16", 30, 1536, 12, 128, 8960, 1536, (21, 30, 52), 0, 1, 256, 64,
                      "partition", n_cells=37, t_group=3, m_min=32, m_max=512),
}

# scaled-down twins with the same structure, small enough for the CPU oracle
WORKLOADS["audio_small"] = WORKLOADS["audio"].replace(
    name="audio_small", L=2, H=256, heads=4, M=512, Hc=256, grid=(416,), B=3, R=26, D=16)
WORKLOADS["image_small"] = WORKLOADS["image"].replace(
    name="image_small", L=2, H=288, heads=4, M=576, Hc=288, grid=(12, 16), B=2, R=12,
    n_cells=12, m_min=8, m_max=32)
WORKLOADS["mmdit_small"] = WORKLOADS["mmdit"].replace(
    name="mmdit_small", L=2, H=256, heads=4, M=512, Hc=256, grid=(16, 20), n_text=27, B=2, R=16,
    n_cells=16, m_min=8, m_max=64, D=16)
WORKLOADS["video_small"] = WORKLOADS["video"].replace(
    name="video_small", L=2, H=256, heads=2, M=640, Hc=256, grid=(6, 10, 14), B=1, R=24,
    n_cells=12, m_min=8, m_max=128, D=16)


# twins whose widths fit the tensor-core tiles (multiples of 128)
WORKLOADS["audio_tc"] = WORKLOADS["audio"].replace(
    name="audio_tc", L=2, H=256, heads=4, M=512, Hc=256, grid=(416,), B=3, R=26, D=16)
WORKLOADS["mmdit_tc"] = WORKLOADS["mmdit"].replace(
    name="mmdit_tc", L=2, H=384, heads=6, M=768, Hc=384, grid=(16, 20), n_text=27, B=2, R=16,
    n_cells=16, m_min=8, m_max=64, D=16)
WORKLOADS["video_tc"] = WORKLOADS["video"].replace(
    name="video_tc", L=2, H=256, heads=2, M=640, Hc=256, grid=(6, 10, 14), B=1, R=24,
    n_cells=12, m_min=8, m_max=128, D=16)
# config 4's scaled-down twin for full-depth, multi-step parity: all 30 blocks, 3136 keys (long enough for the
# attention's default cut-and-combine path), 32 spatio-temporal regions
WORKLOADS["video_twin"] = WORKLOADS["video"].replace(
    name="video_twin", H=256, heads=2, M=640, Hc=256, grid=(7, 16, 28), B=1, R=32,
    n_cells=6, m_min=16, m_max=256, D=16)
WORKLOADS["image_tc"] = WORKLOADS["image"].replace(
    name="image_tc", L=1, grid=(12, 16), B=2, R=12, n_cells=12, m_min=8, m_max=32)
WORKLOADS["wide_tc"] = WORKLOADS["audio"].replace(
    name="wide_tc", L=1, H=1024, heads=8, head_dim=128, M=3072, Hc=256, grid=(208,), B=2, R=13, D=16)


def workload(name: str) -> Workload:
    return WORKLOADS[name]


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence(list(key))))


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bfloat16 (ties to even), returned as fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    lsb = (bits >> 16) & 1
    rounded = ((bits + 0x7FFF + lsb) >> 16) << 16
    return rounded.astype(np.uint32).view(np.float32).reshape(a.shape)


def _store(wl: Workload, a: np.ndarray) -> np.ndarray:
    a = a.astype(np.float32)
    return round_bf16(a) if wl.dtype == "bf16" else a


def block_weights(wl: Workload, seed: int, n_blocks: Optional[int] = None,
                  std: float = 0.02) -> Dict[str, np.ndarray]:
    """Weights and biases ~N(0, std) for ``n_blocks`` blocks, rounded to the storage type.

    Block ``l`` is drawn from its own stream, so a shorter stack is a prefix of a longer one.
    Layout (row-major, input dimension contiguous): w_qkv [L,3H,H], w_o [L,H,H],
    w_fc1 [L,M,H], w_fc2 [L,H,M], w_ada [L,6H,Hc]; biases [L,out].
    """
    L = wl.L if n_blocks is None else n_blocks
    H, M, Hc = wl.H, wl.M, wl.Hc
    shapes = {
        "w_qkv": (3 * H, H), "b_qkv": (3 * H,), "w_o": (H, H), "b_o": (H,),
        "w_fc1": (M, H), "b_fc1": (M,), "w_fc2": (H, M), "b_fc2": (H,),
        "w_ada": (6 * H, Hc), "b_ada": (6 * H,),
    }
    out = {k: np.empty((L,) + s, dtype=np.float32) for k, s in shapes.items()}
    for l in range(L):
        g = _rng(seed, 101, l)
        for k, s in shapes.items():
            out[k][l] = _store(wl, g.standard_normal(s, dtype=np.float32) * np.float32(std))
    return out


def sampler_weights(wl: Workload, seed: int) -> Dict[str, np.ndarray]:
    """Patch embedding (D -> H, bias, positional table) and final layer (H -> D, bias), rounded to the
    storage type: w_in [H,D], b_in [H], pos [N,H], w_out [D,H], b_out [D]."""
    g = _rng(seed, 909)
    H, D, N = wl.H, wl.D, wl.N
    return {
        "w_in": _store(wl, g.standard_normal((H, D), dtype=np.float32) / np.float32(np.sqrt(D))),
        "b_in": _store(wl, g.standard_normal((H,), dtype=np.float32) * np.float32(0.1)),
        "pos": _store(wl, g.standard_normal((N, H), dtype=np.float32) * np.float32(0.5)),
        "w_out": _store(wl, g.standard_normal((D, H), dtype=np.float32) / np.float32(np.sqrt(H))),
        "b_out": _store(wl, g.standard_normal((D,), dtype=np.float32) * np.float32(0.1)),
    }


def uniform_labels(wl: Workload) -> np.ndarray:
    """Caller-written partitions: 2-D square blocks or contiguous 1-D segments. int32 [B,N]."""
    if wl.labels == "blocks2d":
        h, w = wl.grid
        side = int(round(np.sqrt(wl.R)))
        assert side * side == wl.R and h % side == 0 and w % side == 0
        bh, bw = h // side, w // side
        yy, xx = np.meshgrid(np.arange(h), np.arange(w), indexing="ij")
        lab = ((yy // bh) * side + (xx // bw)).reshape(-1)
    elif wl.labels == "segments":
        n = wl.n_grid
        assert n % wl.R == 0
        lab = np.arange(n) // (n // wl.R)
    else:
        raise ValueError("labels of this workload come from the partitioner")
    lab = np.concatenate([lab, np.full(wl.n_text, wl.R)]).astype(np.int32)
    return np.ascontiguousarray(np.broadcast_to(lab, (wl.B, wl.N)))


def saliency_map(wl: Workload, seed: int, noise: float = 0.05) -> np.ndarray:
    """Block-structured early-step attention map, fp32 [B, n_grid, 1].

    Random Voronoi cells on the token grid (per temporal group for 3-D grids), each cell with
    one level out of an evenly spaced, seeded permutation of [0,1], plus N(0, noise).
    """
    out = np.empty((wl.B, wl.n_grid, 1), dtype=np.float32)
    grid = wl.grid
    coords = np.stack(np.meshgrid(*[np.arange(g) for g in grid], indexing="ij"), -1)
    coords = coords.reshape(-1, len(grid)).astype(np.float64)
    for b in range(wl.B):
        g = _rng(seed, 202, b)
        if len(grid) == 3 and wl.t_group > 0:
            n_groups = (grid[0] + wl.t_group - 1) // wl.t_group
            cell = np.empty(wl.n_grid, dtype=np.int64)
            tgrp = (coords[:, 0] // wl.t_group).astype(np.int64)
            for q in range(n_groups):
                sites = g.random((wl.n_cells, 2)) * np.array(grid[1:], dtype=np.float64)
                sel = np.nonzero(tgrp == q)[0]
                d2 = ((coords[sel, None, 1:] - sites[None]) ** 2).sum(-1)
                cell[sel] = q * wl.n_cells + np.argmin(d2, axis=1)
            n_total = n_groups * wl.n_cells
        else:
            sites = g.random((wl.n_cells, len(grid))) * np.array(grid, dtype=np.float64)
            d2 = ((coords[:, None, :] - sites[None]) ** 2).sum(-1)
            cell = np.argmin(d2, axis=1)
            n_total = wl.n_cells
        levels = np.linspace(0.0, 1.0, n_total)[g.permutation(n_total)]
        s = levels[cell] + noise * g.standard_normal(wl.n_grid)
        out[b, :, 0] = s.astype(np.float32)
    return out


def step_inputs(wl: Workload, seed: int, labels: np.ndarray,
                sigma: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Hidden tokens of two neighbouring steps and the conditioning vectors.

    x_cur[B,N,H] ~ N(0,1); x_prev = x_cur + sigma[b, region] * N(0,1) (text tokens, label R,
    get the median sigma); cond[B,Hc] ~ N(0,1).  All rounded to the storage type.
    """
    g = _rng(seed, 303)
    B, N, H = wl.B, wl.N, wl.H
    x_cur = g.standard_normal((B, N, H), dtype=np.float32)
    if sigma is None:
        sigma = region_sigma(wl, seed)
    sig_tok = _sigma_per_token(wl, labels, sigma)
    x_prev = x_cur + sig_tok[..., None] * g.standard_normal((B, N, H), dtype=np.float32)
    cond = g.standard_normal((B, wl.Hc), dtype=np.float32)
    return {"x_cur": _store(wl, x_cur), "x_prev": _store(wl, x_prev), "cond": _store(wl, cond)}


def region_sigma(wl: Workload, seed: int, lo: float = 1e-4, hi: float = 1e-1) -> np.ndarray:
    """Per-region noise scale, log-uniform in [lo, hi]. fp64 [B,R]."""
    g = _rng(seed, 404)
    return np.exp(g.uniform(np.log(lo), np.log(hi), size=(wl.B, wl.R)))


def _sigma_per_token(wl: Workload, labels: np.ndarray, sigma: np.ndarray) -> np.ndarray:
    ext = np.concatenate([sigma, np.median(sigma, axis=1, keepdims=True)], axis=1)  # label R
    return np.take_along_axis(ext, labels.astype(np.int64), axis=1).astype(np.float32)


def latent_pair(wl: Workload, seed: int, labels: np.ndarray,
                fractions: Optional[Sequence[float]] = None,
                eps_fixed: Optional[float] = None) -> Dict[str, np.ndarray]:
    """Latents of two neighbouring steps plus the gate threshold of each request.

    z_cur[B,N,D] ~ N(0,1) fp32; z_prev = z_cur + sigma_r * N(0,1) per region (label-R tokens
    unchanged).  Either ``fractions`` (one target active-region fraction per request) or
    ``eps_fixed`` selects the threshold:

    * fractions: the k = round(f*R) largest sigmas are pushed up by sqrt(2) and the others
      down by sqrt(2), and eps = sqrt(sigma_(k) * sigma_(k+1)) / sum(sigma): the cut sits in
      a gap of at least 2x in noise scale, far more than the sampling spread of a region's
      measured change, so exactly k regions end up above it.  f = 1 gives eps = 0.
    * eps_fixed: sigmas are re-drawn until every sigma_r / sum(sigma) is at least 15 % away
      from eps_fixed.

    Returns z_cur, z_prev, eps [B] fp32, sigma [B,R] fp64, n_loud [B] (expected active regions).
    """
    B, N, D, R = wl.B, wl.N, wl.D, wl.R
    sigma = None
    for attempt in range(1000):
        g = _rng(seed, 505, attempt)
        sigma = np.exp(g.uniform(np.log(1e-4), np.log(1e-1), size=(B, R)))
        if eps_fixed is None:
            break
        rel = sigma / sigma.sum(axis=1, keepdims=True) / eps_fixed
        if np.all(np.abs(rel - 1.0) >= 0.15):
            break
    else:  # pragma: no cover
        raise RuntimeError("could not draw sigmas away from the threshold")
    eps = np.empty(B, dtype=np.float32)
    n_loud = np.empty(B, dtype=np.int64)
    if eps_fixed is not None:
        eps[:] = eps_fixed
        n_loud[:] = (sigma / sigma.sum(axis=1, keepdims=True) >= eps_fixed).sum(axis=1)
    else:
        assert fractions is not None and len(fractions) == B
        for b in range(B):
            k = int(round(float(fractions[b]) * R))
            k = min(max(k, 1), R)
            order = np.argsort(-sigma[b], kind="stable")
            sigma[b, order[:k]] *= np.sqrt(2.0)
            sigma[b, order[k:]] /= np.sqrt(2.0)
            n_loud[b] = k
            if k == R:
                eps[b] = 0.0
            else:
                cut = np.sqrt(sigma[b, order[k - 1]] * sigma[b, order[k]])
                eps[b] = np.float32(cut / sigma[b].sum())
    g = _rng(seed, 606)
    z_cur = g.standard_normal((B, N, D), dtype=np.float32)
    sig_tok = np.take_along_axis(np.concatenate([sigma, np.zeros((B, 1))], axis=1),
                                 labels.astype(np.int64), axis=1).astype(np.float32)
    z_prev = z_cur + sig_tok[..., None] * g.standard_normal((B, N, D), dtype=np.float32)
    return {"z_cur": z_cur, "z_prev": z_prev.astype(np.float32), "eps": eps,
            "sigma": sigma, "n_loud": n_loud}


def region_mask(wl: Workload, seed: int, fractions: Sequence[float]) -> np.ndarray:
    """Active-region mask with round(f_b * R) regions switched on per request. uint8 [B,R]."""
    g = _rng(seed, 707)
    mask = np.zeros((wl.B, wl.R), dtype=np.uint8)
    for b in range(wl.B):
        k = min(max(int(round(float(fractions[b]) * wl.R)), 0), wl.R)
        mask[b, g.permutation(wl.R)[:k]] = 1
    return mask


def mask_schedule(wl: Workload, seed: int, steps: int, fraction: float = 0.5) -> np.ndarray:
    """Fixed mask schedule: step 0 dense (warm-up), then ``fraction`` of regions per step.
    uint8 [steps,B,R]."""
    out = np.zeros((steps, wl.B, wl.R), dtype=np.uint8)
    out[0] = 1
    for s in range(1, steps):
        out[s] = region_mask(wl, seed * 131 + s, [fraction] * wl.B)
    return out


def request_fractions(wl: Workload, seed: int, lo: float = 0.2, hi: float = 0.8) -> np.ndarray:
    """Per-request active fraction ~U[lo,hi] (requests at different denoising steps)."""
    return _rng(seed, 808).uniform(lo, hi, size=wl.B)


def latent_sequence(wl: Workload, seed: int, labels: np.ndarray,
                    fractions_per_step: Sequence[Sequence[float]]):
    """Latents of a run of neighbouring steps with a target active fraction per step and request.

    z_0 ~ N(0,1); step t moves every region by its own noise scale, z_t = z_{t-1} + sigma_t[region] * N(0,1), where
    sigma_t and the threshold eps_t are drawn exactly as in ``latent_pair`` for the fractions of step t (a fresh
    log-uniform draw per step, the k loudest pushed up and the others down by sqrt(2), eps in the gap).  Regions
    a gate keeps frozen carry older magnitudes, so the measured fraction of a step need not equal its target.
    Returns a list of dicts with z_cur, z_prev, eps (one per step).
    """
    B, N, D, R = wl.B, wl.N, wl.D, wl.R
    g = _rng(seed, 1212)
    z = g.standard_normal((B, N, D), dtype=np.float32)
    out = []
    for t, fractions in enumerate(fractions_per_step):
        assert len(fractions) == B
        sigma = np.exp(g.uniform(np.log(1e-4), np.log(1e-1), size=(B, R)))
        eps = np.empty(B, dtype=np.float32)
        for b in range(B):
            k = min(max(int(round(float(fractions[b]) * R)), 1), R)
            order = np.argsort(-sigma[b], kind="stable")
            sigma[b, order[:k]] *= np.sqrt(2.0)
            sigma[b, order[k:]] /= np.sqrt(2.0)
            eps[b] = 0.0 if k == R else np.float32(np.sqrt(sigma[b, order[k - 1]] * sigma[b, order[k]]) / sigma[b].sum())
        sig_tok = np.take_along_axis(np.concatenate([sigma, np.zeros((B, 1))], axis=1),
                                     labels.astype(np.int64), axis=1).astype(np.float32)
        z_next = (z + sig_tok[..., None] * g.standard_normal((B, N, D), dtype=np.float32)).astype(np.float32)
        out.append({"z_cur": z_next, "z_prev": z, "eps": eps})
        z = z_next
    return out


def block_variants(wl: Workload, seed: int, n_blocks: Optional[int] = None, qk_norm: bool = True, rope: bool = True,
                   rope_base: float = 10000.0) -> Dict[str, np.ndarray]:
    """Inputs of the block variants: QK-RMSNorm weights ~ 1 + N(0, 0.1) per block and head channel
    (q_norm_w, k_norm_w [L, head_dim], rounded to the storage type) and rotary tables for positions 0..N-1 with the
    usual frequencies base^(-2i/d) (rope_cos, rope_sin [N, head_dim/2] fp32).  Only draws and tabulates inputs."""
    L = wl.L if n_blocks is None else n_blocks
    dh = wl.head_dim
    out: Dict[str, np.ndarray] = {}
    if qk_norm:
        g = _rng(seed, 1313)
        out["q_norm_w"] = _store(wl, 1.0 + 0.1 * g.standard_normal((L, dh), dtype=np.float32))
        out["k_norm_w"] = _store(wl, 1.0 + 0.1 * g.standard_normal((L, dh), dtype=np.float32))
        out["qk_norm_eps"] = 1e-6
    if rope:
        freq = rope_base ** (-2.0 * np.arange(dh // 2, dtype=np.float64) / dh)
        ang = np.arange(wl.N, dtype=np.float64)[:, None] * freq[None, :]
        out["rope_cos"] = np.cos(ang).astype(np.float32)
        out["rope_sin"] = np.sin(ang).astype(np.float32)
    return out


def cross_attention(wl: Workload, seed: int, n_ctx: int, n_blocks: Optional[int] = None, std: float = 0.02) -> Dict[str, np.ndarray]:
    """Inputs of the cross-attention variant: query / out projections ~N(0, std) per block (w_q, w_o [L,H,H]; b_q, b_o
    [L,H]) and the context's keys and values ~N(0, 0.5) (ctx_kv [L,B,2,n_ctx,H]; they stand for a text encoder's states
    already projected by the caller), rounded to the storage type."""
    L = wl.L if n_blocks is None else n_blocks
    H = wl.H
    g = _rng(seed, 1414)
    out = {k: _store(wl, g.standard_normal(s, dtype=np.float32) * np.float32(std))
           for k, s in (("w_q", (L, H, H)), ("b_q", (L, H)), ("w_o", (L, H, H)), ("b_o", (L, H)))}
    out["ctx_kv"] = _store(wl, g.standard_normal((L, wl.B, 2, n_ctx, H), dtype=np.float32) * np.float32(0.5))
    return out


def fp8_operands(wl: Workload, w: Dict[str, np.ndarray], seed: int, n_blocks: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Inputs of the FP8-operand variant from a weight set: the QKV, fc1 and fc2 matrices quantised per output row to
    E4M3 (scale s = max|row| / 448, fp32; codes by the library's float8 cast of row / s), and per-block activation
    scales drawn per tensor (the normalised inputs of QKV and fc1 ~U[0.02, 0.04], the GELU output ~U[0.01, 0.02]; an
    activation beyond 448 scales saturates on both sides alike).  Returns, per matrix, the codes c_* (uint8), their
    values w_* (float32) and the scales s_*, and a_scale [L, 3]."""
    import torch
    L = wl.L if n_blocks is None else n_blocks
    out: Dict[str, np.ndarray] = {}
    for name in ("qkv", "fc1", "fc2"):
        W = torch.from_numpy(np.ascontiguousarray(w["w_" + name][:L], dtype=np.float32))
        s = (W.abs().amax(dim=-1) / 448.0).clamp_min(1e-12)
        q = (W / s[..., None]).to(torch.float8_e4m3fn)
        out["c_" + name] = q.view(torch.uint8).numpy().copy()
        out["w_" + name] = q.to(torch.float32).numpy().copy()
        out["s_" + name] = s.numpy().astype(np.float32)
    g = _rng(seed, 1515)
    a = np.empty((L, 3), np.float32)
    a[:, 0:2] = g.uniform(0.02, 0.04, (L, 2))
    a[:, 2] = g.uniform(0.01, 0.02, L)
    out["a_scale"] = a
    return out
