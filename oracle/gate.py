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


def attention_mass(q_rows: np.ndarray, k_cache: np.ndarray, labels: np.ndarray, active_idx: np.ndarray,
                   heads: int, R: int) -> np.ndarray:
    """Own-region self-attention mass of the active queries (paper Sec. 4.2, the sum inside R_i).

    q_rows [A,H]: queries of the active tokens (one block), k_cache [B,N,H]: keys of ALL tokens of
    every request as the attention of that block saw them (fresh rows for active tokens, cached
    rows for skipped ones).  SA is the softmax attention matrix averaged over heads; the result
    is mass[b,i] = sum over active queries u of region i, and over keys v of region i, of
    SA[u,v].  Tokens with label R (always active, outside the gate) contribute to no region.
    """
    B, N, H = k_cache.shape
    d = H // heads
    mass = np.zeros((B, R), np.float64)
    for a, g in enumerate(np.asarray(active_idx, np.int64)):
        b, j = divmod(int(g), N)
        i = int(labels[b, j])
        if i >= R:
            continue
        same = labels[b] == i
        own = 0.0
        for hd in range(heads):
            qv = q_rows[a, hd * d:(hd + 1) * d].astype(np.float64)
            s = k_cache[b, :, hd * d:(hd + 1) * d].astype(np.float64) @ qv / np.sqrt(d)
            p = np.exp(s - s.max())
            p /= p.sum()
            own += p[same].sum()
        mass[b, i] += own / heads
    return mass


def attention_gate(mass: np.ndarray, region_sizes: np.ndarray, eps: np.ndarray, state: Dict[str, np.ndarray], R: int,
                   K: int = 5, eta: float = 1e-12):
    """Patch Gate on the paper's own signal (Sec. 4.2): R_i = mass_i / |A_i|^2 for the patches that were
    executed at the step that produced ``mass``; for those, Delta_i = |R_i - Rbar_i| and Rbar_i <- R_i;
    a skipped patch keeps its Delta_i.  The weights, the threshold and the forced reactivation are
    those of ``activity_gate``.  ``state`` additionally holds ``rbar`` [B,R] fp32 (updated in place).
    Returns importance [B,R] f32 (R_i where fresh, Rbar_i otherwise), weight [B,R] f32, mask [B,R] u8.
    """
    B = mass.shape[0]
    delta, skip, prev, rbar = state["delta"], state["skip_count"], state["prev_active"], state["rbar"]
    weight = np.zeros((B, R), np.float32)
    mask = np.zeros((B, R), np.uint8)
    for b in range(B):
        for i in range(R):
            if not prev[b, i]:
                continue                                      # skipped: Delta_i and Rbar_i stay
            n = float(region_sizes[b, i])
            r_i = np.float32(float(mass[b, i]) / (n * n)) if n > 0 else np.float32(0.0)
            delta[b, i] = np.float32(abs(float(r_i) - float(rbar[b, i])))
            rbar[b, i] = r_i
        dn = 0.0
        for i in range(R):
            dn += float(delta[b, i]) + eta
        for i in range(R):
            num = float(delta[b, i]) + eta
            weight[b, i] = np.float32(num / dn) if dn > 0.0 else np.float32(1.0 / R)
            gate_on = (num >= float(eps[b]) * dn) if dn > 0.0 else True
            mask[b, i] = 1 if (gate_on or skip[b, i] >= K) else 0
        for i in range(R):
            skip[b, i] = 0 if mask[b, i] else skip[b, i] + 1
            prev[b, i] = mask[b, i]
    return rbar.copy(), weight, mask


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
