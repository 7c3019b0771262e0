"""TEST INFRASTRUCTURE -- CPU oracle of the Patch Partitioner.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import this.
Shares no code with the CUDA library.

Follows paper Sec. 4.1 ("Capturing Patch Coherence and Complexity", "Recursive Load-Aware
Patch Partitioning") and Appendix A.3 (Eq. otsu, hierarchical-extension remark):

1. saliency S_j = mean over the salient prompt tokens of the attention map's columns;
2. the map is min-max normalised and put on a 16-bit integer scale, so that every later
   decision is exact integer arithmetic (Python integers here);
3. a node is bisected at the threshold maximising the between-class variance
   omega_f omega_c (mu_f - mu_c)^2 (focus: value >= theta);
4. the node's region budget is shared by r_f = argmin_r |r - R n_f / (n_f + n_c)|;
5. both halves are split again until R regions exist.

Conventions where the paper is silent: ties go to the lowest threshold / smallest r; a cut
must leave each side between m_min and m_max tokens per region it has to host; a node with
no admissible cut is chopped in token order into equal chunks; regions are numbered by
their smallest token index.
"""
from __future__ import annotations

from typing import List, Optional, Tuple

import numpy as np


def saliency(attn_map: np.ndarray, salient_cols: Optional[np.ndarray]) -> np.ndarray:
    """S_j for one request: attn_map [N,T] -> fp32 [N] (fp64 accumulation in column order)."""
    N, T = attn_map.shape
    cols = list(range(T)) if salient_cols is None else [int(c) for c in salient_cols]
    out = np.empty(N, np.float32)
    for j in range(N):
        acc = 0.0
        for t in cols:
            acc += float(attn_map[j, t])
        out[j] = np.float32(acc / len(cols))
    return out


def quantise(S: np.ndarray) -> np.ndarray:
    """16-bit codes floor((S - min) / (max - min) * 65535 + 0.5), each step rounded to fp32."""
    S = S.astype(np.float32)
    lo, hi = np.float32(S.min()), np.float32(S.max())
    if hi == lo:
        return np.zeros(S.shape, np.int64)
    t = (S - lo).astype(np.float32)
    t = (t / np.float32(hi - lo)).astype(np.float32)
    t = (t * np.float32(65535.0)).astype(np.float32)
    t = (t + np.float32(0.5)).astype(np.float32)
    return np.floor(t).astype(np.int64)


def allocate(n_f: int, n_c: int, R: int) -> int:
    """r_f = argmin over r in 1..R-1 of |r - R n_f/(n_f+n_c)|, in integers; ties -> smaller r.

    |r n - R n_f| is convex in r with its minimum at R n_f / n, so only the two integers
    around that point (clamped to 1..R-1) can win; the tests compare this with the full scan.
    """
    n = n_f + n_c
    lo = (R * n_f) // n
    best_r, best_d = None, None
    for r in (lo, lo + 1):
        r = min(max(r, 1), R - 1)
        d = abs(r * n - R * n_f)
        if best_d is None or d < best_d:
            best_r, best_d = r, d
    return best_r


def best_cut(q_sorted: List[int], R_node: int, m_min: int, m_max: int
             ) -> Optional[Tuple[int, int]]:
    """Position p (context = first p sorted tokens) of the admissible cut with the largest
    between-class variance, and its r_f.  None if no cut is admissible."""
    n = len(q_sorted)
    total = sum(q_sorted)
    best = None           # (num, den, p, r_f)
    pre = 0
    for p in range(1, n):
        pre += q_sorted[p - 1]
        if q_sorted[p - 1] == q_sorted[p]:
            continue       # a threshold cannot separate equal values
        n_c, n_f = p, n - p
        s_c, s_f = pre, total - pre
        r_f = allocate(n_f, n_c, R_node)
        r_c = R_node - r_f
        if not (m_min * r_f <= n_f <= m_max * r_f and m_min * r_c <= n_c <= m_max * r_c):
            continue
        num = (n_c * s_f - n_f * s_c) ** 2      # sigma_B^2 * n^2 * n_f * n_c
        den = n_f * n_c
        if best is None or num * best[1] > best[0] * den:
            best = (num, den, p, r_f)
    return None if best is None else (best[2], best[3])


def _split(tokens: List[int], q: np.ndarray, R_node: int, m_min: int, m_max: int,
           leaves: List[List[int]]) -> None:
    if R_node == 1:
        leaves.append(tokens)
        return
    order = sorted(tokens, key=lambda j: (int(q[j]), j))
    cut = best_cut([int(q[j]) for j in order], R_node, m_min, m_max)
    if cut is None:
        by_index = sorted(tokens)
        n = len(by_index)
        base, extra = divmod(n, R_node)
        pos = 0
        for r in range(R_node):
            size = base + (1 if r < extra else 0)
            leaves.append(by_index[pos:pos + size])
            pos += size
        return
    p, r_f = cut
    _split(order[p:], q, r_f, m_min, m_max, leaves)            # focus: value >= theta
    _split(order[:p], q, R_node - r_f, m_min, m_max, leaves)   # context


def partition_request(S: np.ndarray, R: int, m_min: int = 1, m_max: int = 0) -> np.ndarray:
    """Labels int32 [N] in [0,R) for one request from its saliency map."""
    N = S.shape[0]
    if not (1 <= R <= N):
        raise ValueError("need 1 <= R <= N")
    if m_max <= 0:
        m_max = N
    q = quantise(S)
    leaves: List[List[int]] = []
    _split(list(range(N)), q, R, m_min, m_max, leaves)
    leaves = [lf for lf in leaves]
    leaves.sort(key=lambda lf: min(lf) if lf else N)
    labels = np.full(N, -1, np.int32)
    for i, lf in enumerate(leaves):
        labels[lf] = i
    return labels


def partition(attn_map: np.ndarray, salient_cols: Optional[np.ndarray], R: int,
              m_min: int = 1, m_max: int = 0):
    """attn_map [B,N,T] -> labels int32 [B,N], region_sizes int32 [B,R]."""
    B, N, _ = attn_map.shape
    labels = np.empty((B, N), np.int32)
    sizes = np.zeros((B, R), np.int32)
    for b in range(B):
        labels[b] = partition_request(saliency(attn_map[b], salient_cols), R, m_min, m_max)
        sizes[b] = np.bincount(labels[b], minlength=R)[:R]
    return labels, sizes
