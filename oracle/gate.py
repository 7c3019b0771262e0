"""TEST INFRASTRUCTURE -- CPU oracle of the Patch Gate and of the active-token compaction.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import this.
Shares no code with the CUDA library.

Gate (paper Sec. 4.2; Appendix A.1 "Patch Gate notation", Eq. gate-weight, Eq.
forced-reactivation).  The raw per-patch signal is the change of the latent between two
neighbouring steps (root mean square over the patch's tokens and channels); everything
after it is the paper's rule:

* a patch executed at the previous step gets a fresh change magnitude, a skipped patch keeps
  its cached one;
* w_i = (delta_i + eta) / D with D = sum_j (delta_j + eta);
* the patch is skipped iff w_i < eps, unless it has already been skipped K steps in a row,
  in which case it is forced back on.

fp64 arithmetic on fp32-stored inputs; the change magnitude is stored in fp32.
"""
from __future__ import annotations

from typing import Dict

import numpy as np


def initial_state(B: int, R: int) -> Dict[str, np.ndarray]:
    """Gate state right after the dense warm-up steps: everything ran, nothing skipped yet."""
    return {"delta": np.zeros((B, R), np.float32),
            "skip_count": np.zeros((B, R), np.int32),
            "prev_active": np.ones((B, R), np.uint8)}


def activity_gate(z_cur: np.ndarray, z_prev: np.ndarray, labels: np.ndarray, eps: np.ndarray,
                  state: Dict[str, np.ndarray], R: int, K: int = 5, eta: float = 1e-12):
    """One gate evaluation for B requests.

    z_cur, z_prev [B,N,D] fp32; labels [B,N] with values in [0,R) (R = always-active tokens,
    outside the gate); eps [B].  ``state`` is updated in place.
    Returns score [B,R] f32, weight [B,R] f32, mask [B,R] u8.
    """
    B, N, D = z_cur.shape
    delta, skip, prev = state["delta"], state["skip_count"], state["prev_active"]
    weight = np.zeros((B, R), np.float32)
    mask = np.zeros((B, R), np.uint8)
    for b in range(B):
        # Eq. delta-i with the latent-change signal: fresh only where the patch ran last step
        for i in range(R):
            if not prev[b, i]:
                continue                      # frozen at its last-active value
            tok = np.nonzero(labels[b] == i)[0]
            if tok.size == 0:
                delta[b, i] = 0.0
                continue
            acc = 0.0
            for j in tok:                     # ascending token, ascending channel
                d = z_cur[b, j].astype(np.float64) - z_prev[b, j].astype(np.float64)
                acc += float(np.dot(d, d))
            delta[b, i] = np.float32(np.sqrt(acc / (tok.size * D)))
        # Eq. gate-weight
        dn = 0.0
        for i in range(R):
            dn += float(delta[b, i]) + eta
        for i in range(R):
            num = float(delta[b, i]) + eta
            weight[b, i] = np.float32(num / dn) if dn > 0.0 else np.float32(1.0 / R)
            gate_on = (num >= float(eps[b]) * dn) if dn > 0.0 else True   # w_i >= eps
            forced = skip[b, i] >= K          # Eq. forced-reactivation
            mask[b, i] = 1 if (gate_on or forced) else 0
        for i in range(R):
            skip[b, i] = 0 if mask[b, i] else skip[b, i] + 1
            prev[b, i] = mask[b, i]
    return delta.copy(), weight, mask


def compact(mask: np.ndarray, labels: np.ndarray, R: int):
    """Ascending list of active global token ids b*N + j and per-request offsets.

    A token is active iff its patch is in the active set (Algorithm 1, PatchGate output) or
    its label is R (always active).  Returns active_idx int32 [A], cu_active int32 [B+1].
    """
    B, N = labels.shape
    idx = []
    cu = [0]
    for b in range(B):
        for j in range(N):
            lab = int(labels[b, j])
            if lab == R or mask[b, lab]:
                idx.append(b * N + j)
        cu.append(len(idx))
    return np.asarray(idx, np.int32), np.asarray(cu, np.int32)
