"""TEST INFRASTRUCTURE -- CPU oracle of the sampler closure around the regional step.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import this.
Shares no code with the CUDA library.

Update rule (Appendix A.1, Eq. sf-update): at step n every patch moves along a drift,

    x_{n+1}^(i) = x_n^(i) + h * f^(i)(x_n, t_n)     if patch i is active,
    x_{n+1}^(i) = x_n^(i) + h * c_n^(i)              if it is skipped,

where c_n^(i) is the drift the patch had at its most recent active step.  The drift of a token
is read off the block stack's output row by a final layer (LayerNorm without affine, then a
linear map H -> D); the token rows enter the block stack through a linear patch embedding
D -> H plus a positional table.  Both maps are per token, so "patch i" is simply the set of
tokens carrying label i.

fp64 arithmetic on fp32-stored inputs.
"""
from __future__ import annotations

import numpy as np


def embed(z: np.ndarray, w_in: np.ndarray, b_in: np.ndarray, pos: np.ndarray) -> np.ndarray:
    """x[b, j, :] = z[b, j, :] @ w_in^T + b_in + pos[j, :].   z [B,N,D], w_in [H,D], pos [N,H]."""
    B, N, D = z.shape
    H = w_in.shape[0]
    x = np.empty((B, N, H), np.float64)
    w = w_in.astype(np.float64)
    for b in range(B):
        for j in range(N):
            x[b, j] = w @ z[b, j].astype(np.float64) + b_in.astype(np.float64) + pos[j].astype(np.float64)
    return x.astype(np.float32)


def token_drift(y_row: np.ndarray, w_out: np.ndarray, b_out: np.ndarray, ln_eps: float) -> np.ndarray:
    """Final layer of one token: LayerNorm (no affine) over the H outputs, then H -> D."""
    v = y_row.astype(np.float64)
    mean = v.sum() / v.size
    var = ((v - mean) ** 2).sum() / v.size
    u = (v - mean) / np.sqrt(var + ln_eps)
    return w_out.astype(np.float64) @ u + b_out.astype(np.float64)


def update(z: np.ndarray, y: np.ndarray, active_idx: np.ndarray, w_out: np.ndarray, b_out: np.ndarray,
           h: np.ndarray, drift: np.ndarray, ln_eps: float = 1e-6) -> np.ndarray:
    """One application of Eq. sf-update.

    z [B,N,D] fp32 latent; y [B,N,H] block-stack output (rows of skipped tokens are whatever
    they were, they are not read); active_idx ascending global token ids b*N+j of the active
    tokens; h [B] step sizes; drift [B,N,D] fp32 cache, updated in place for the active
    tokens.  Returns z_next [B,N,D] fp32.
    """
    B, N, D = z.shape
    for g in np.asarray(active_idx, np.int64):
        b, j = divmod(int(g), N)
        drift[b, j] = token_drift(y[b, j], w_out, b_out, ln_eps).astype(np.float32)   # fresh drift, cached
    z_next = np.empty_like(z)
    for b in range(B):
        hb = float(h[b])
        for j in range(N):
            z_next[b, j] = (z[b, j].astype(np.float64) + hb * drift[b, j].astype(np.float64)).astype(np.float32)
    return z_next
