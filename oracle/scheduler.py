"""TEST INFRASTRUCTURE -- CPU oracle of the host-side batch former (patch monotasks, Sec. 4.3).

Only tests may import this.  Shares no code with the library.

Two policies of the paper's Patch Scheduler, restated for requests that share one device step:

``pack``        the least-maximum-load rule (Sec. 4.3, the equation of "Maximizing Goodput with
                Monotask Packing"): an incoming monotask j of cost w_j goes to

                    g* = argmin_g  max_g' ( L_g' + w_j  if g' == g  else  L_g' )

                written out literally: for every candidate g the maximum over all g' is formed and
                the candidate with the smallest maximum wins.  Readings where the paper is silent:
                among candidates that tie on that maximum the monotask's *home* (the device that
                already holds patches of the same request; Sec. 4.3 "Monotask Packing" asks for
                placement that respects locality) wins if it is one of them, otherwise the candidate with the smallest own
                load, otherwise the smallest index.  A warm-up monotask has no home, so it goes to
                the least loaded device, which is what the paper states for the warm-up phase.

``form_batch``  which requests run the next step on one device.  Every request's step is one unit
                (its active patch monotasks run together: intra-step execution is atomic and a
                request's step ends only when all of its active patches have run), queued under
                the request's priority; switching happens at step boundaries only, i.e. exactly
                when this function is called.  Requests are visited in the order (priority
                descending, arrival number ascending, index ascending); a request is taken if its
                active tokens still fit into the token budget and its state is resident or a
                residency slot is free (then it takes the slot); a request that does not fit is
                passed over and lower-priority ones may use the leftover (Sec. 4.3 "Efficient Patch
                Switching with Monotasks": spare capacity goes to the best-ranked waiting
                monotask).  The paper's
                worker keeps at most two requests' state; here the bound is a parameter.  A
                request without active tokens costs nothing and is taken if it is resident (its
                step is a pure cached-drift update).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np


def pack(load: Sequence[float], cost: Sequence[float], home: Sequence[int]) -> Tuple[np.ndarray, np.ndarray]:
    """Assign monotasks one after another in the given order.  Returns (assign [n] int32, load [G] f64)."""
    L = [float(v) for v in load]
    G = len(L)
    assign = np.empty(len(cost), np.int32)
    for j, w in enumerate(cost):
        w = float(w)
        worst = []                                       # worst[g] = the step's straggler load if j went to g
        for g in range(G):
            worst.append(max((L[gp] + w) if gp == g else L[gp] for gp in range(G)))
        best = min(worst)
        cands = [g for g in range(G) if worst[g] == best]
        h = int(home[j])
        if h in cands:
            g_star = h
        else:
            g_star = min(cands, key=lambda g: (L[g], g))
        assign[j] = g_star
        L[g_star] += w
    return assign, np.asarray(L, np.float64)


def form_batch(priority: Sequence[int], arrival: Sequence[int], active_tokens: Sequence[int],
               resident: Sequence[int], token_budget: int, max_resident: int) -> Tuple[np.ndarray, np.ndarray]:
    """Returns (chosen [n] uint8, resident_after [n] uint8)."""
    n = len(priority)
    order: List[int] = sorted(range(n), key=lambda i: (-int(priority[i]), int(arrival[i]), i))
    res = [1 if r else 0 for r in resident]
    slots = max_resident - sum(res)
    left = int(token_budget)
    chosen = np.zeros(n, np.uint8)
    for i in order:
        t = int(active_tokens[i])
        if t > left:
            continue
        if not res[i]:
            if t == 0 or slots <= 0:
                continue
            res[i] = 1
            slots -= 1
        chosen[i] = 1
        left -= t
    return chosen, np.asarray(res, np.uint8)


# ---------------------------------------------------------------------------------------------
# Adaptive patch granularity (Sec. 4.1, "Adaptive Patch Granularity")
# ---------------------------------------------------------------------------------------------
# The paper: performance as a function of the number of patches R is unimodal, and R is tuned online by a
# bounded binary search on observed performance -- while a larger R improves performance the search keeps
# refining, when performance degrades it comes back.  Reading (the paper gives no more than that): a search
# state (accepted R with its observed performance, a direction, a step).  The first observation belongs to
# the starting R.  Every later observation belongs to the candidate proposed last: better than the accepted
# one -> the candidate becomes the accepted R and the search continues in the same direction with the same
# step; not better -> the direction flips and the step halves (never below 1).  A candidate is the accepted
# R plus direction * step, clamped to [r_min, r_max]; a candidate equal to the accepted R counts as "not
# better" without being run.  Two failures in a row at step 1 (both neighbours are no better) end the
# search: the accepted R is returned from then on.  The initial step is half the range, rounded up.
class RSearch:
    def __init__(self, r_min: int, r_max: int, r_start: int):
        assert r_min <= r_start <= r_max
        self.r_min, self.r_max = int(r_min), int(r_max)
        self.accepted = int(r_start)
        self.candidate = int(r_start)
        self.step = max(1, (self.r_max - self.r_min + 1) // 2)
        self.dir = 1
        self.ref = None
        self.fails_at_one = 0
        self.converged = self.r_min == self.r_max

    def _propose(self) -> int:
        while not self.converged:
            c = min(self.r_max, max(self.r_min, self.accepted + self.dir * self.step))
            if c != self.accepted:
                self.candidate = c
                return c
            self._fail()                                  # clamped onto the accepted R: nothing to run
        self.candidate = self.accepted
        return self.accepted

    def _fail(self):
        if self.step == 1:
            self.fails_at_one += 1
            if self.fails_at_one >= 2:
                self.converged = True
        self.dir = -self.dir
        self.step = max(1, self.step // 2)

    def update(self, perf: float) -> int:
        """Reports the performance (higher is better) observed with the R returned last; returns the next R."""
        if self.converged:
            return self.accepted
        if self.ref is None:
            self.ref = float(perf)
        elif float(perf) > self.ref:
            self.accepted, self.ref = self.candidate, float(perf)
            self.fails_at_one = 0
        else:
            self._fail()
        return self._propose()
