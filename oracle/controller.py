"""Algorithm 1 ("Pilot-Commit") as a plain simulation over epochs and sampling batches, given the pilot success rate of
every (prompt, step).  TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

    R <- {} ; t <- 0
    for each epoch, for each sampling batch B of D with |B| = b_g:
        pilot: p_hat(q) for q in B
        B' <- {q : p_lower <= p_hat(q) <= p_upper}            filter
        D  <- D \\ {q : p_hat(q) >= p_solve}                    evict solved prompts (for later epochs)
        R  <- R u B'                                           buffer survivors
        while fewer than b_t selected and R not empty: take q from R, draw n_commit rollouts
        train on pilot + commit rollouts of the selected prompts
        remove entries of R older than d steps ; t <- t + 1

Readings (the same as the host controller's, stated there): survivors are taken oldest first in arrival order, a taken
prompt leaves R.  Section 4.2 states d as the maximum delay between a prompt's pilot and its commit, so an entry whose
pilot ran at step b may commit at steps b .. b + d; the clean-up at the end of step t therefore removes the entries that
the next step could no longer use (t - b >= d), which is "older than d steps" on the next step's clock.
"""
from __future__ import annotations

from typing import Callable, Dict, List


def simulate(dataset: List[int], n_epochs: int, b_g: int, b_t: int, n_pilot: int, n_commit: int, p_lower: float,
             p_upper: float, p_solve: float, d: int, p_hat: Callable[[int, int], float]) -> List[Dict]:
    R: List[tuple] = []
    t = 0
    D = list(dataset)
    log = []
    for _ in range(n_epochs):
        pool = list(D)                                    # evictions take effect from the next epoch on
        for b0 in range(0, len(pool), b_g):
            B = pool[b0:b0 + b_g]
            if not B:
                continue
            ph = {q: p_hat(q, t) for q in B}
            survivors = [q for q in B if p_lower <= ph[q] <= p_upper]
            solved = [q for q in B if ph[q] >= p_solve]
            D = [q for q in D if q not in solved]
            R = R + [(q, t) for q in survivors]
            selected = R[:b_t]
            R = R[len(selected):]
            stale = [q for (q, born) in R if t - born >= d]
            R = [(q, born) for (q, born) in R if t - born < d]
            log.append(dict(step=t, batch=B, selected=selected, solved=solved, stale=stale, buffered=len(R),
                            rollouts=len(B) * n_pilot + len(selected) * n_commit))
            t += 1
    return log
