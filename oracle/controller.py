"""Multi-step bookkeeping of Pilot-Commit (Algorithm 1; Section 3.4 "Replay buffer for pilot survivors" and "Evicting
solved prompts"; Section 6.3 for the second sampling round), as a plain simulation driven by the pilot success rate of
every (prompt, step).  TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

The state is kept as events rather than as containers that are edited in place: every pilot survivor is one record
(prompt, step its pilot ran, step it was committed or dropped), and every question the method asks -- who is waiting at
step t, who is too old, who is solved -- is answered by filtering those records.

Readings (the same as the host controller's, stated there): waiting survivors are taken oldest first, in arrival order;
a taken prompt stops waiting; d is the largest delay between a prompt's pilot and its commit (Section 4.2), so after the
commits of step t the survivors whose pilot ran at step t - d or earlier stop waiting (the next step could not use them
within the delay); a prompt whose pilot success rate reaches p_solve is left out of the sampling pool from the next
epoch on; when a step's first sampling batch leaves fewer than b_t prompts selected and `max_rounds` allows it, the next
sampling batch of the epoch is drawn within the same training step (Section 6.3, "second sampling round").
"""
from __future__ import annotations

import dataclasses
from typing import Callable, Dict, List, Optional


@dataclasses.dataclass
class _Survivor:
    prompt: int
    born: int                      # training step whose pilot stage kept it
    order: int                     # arrival order (ties between survivors of one batch)
    taken_at: Optional[int] = None
    dropped_at: Optional[int] = None

    def waiting(self) -> bool:
        return self.taken_at is None and self.dropped_at is None


def simulate(dataset: List[int], n_epochs: int, b_g: int, b_t: int, n_pilot: int, n_commit: int, p_lower: float,
             p_upper: float, p_solve: float, d: int, p_hat: Callable[[int, int], float], max_rounds: int = 1) -> List[Dict]:
    """One record per training step: step, batch (the prompts piloted in it, all rounds), rounds, selected [(prompt, born)],
    solved, stale, buffered (survivors still waiting after the step), rollouts (Section 4.3's count, every round's pilots
    included)."""
    survivors: List[_Survivor] = []
    solved_at: Dict[int, int] = {}             # prompt -> epoch in which it was found solved
    log: List[Dict] = []
    step = 0
    for epoch in range(n_epochs):
        pool = [q for q in dataset if q not in solved_at or solved_at[q] >= epoch]     # solved in an EARLIER epoch: left out
        cursor = 0
        while cursor < len(pool):
            piloted, solved_now, taken = [], [], []
            rounds = 0
            while cursor < len(pool) and rounds < max_rounds and (rounds == 0 or len(taken) < b_t):
                batch = pool[cursor:cursor + b_g]
                cursor += len(batch)
                rounds += 1
                piloted += batch
                for q in batch:
                    ph = p_hat(q, step)
                    if ph >= p_solve:
                        solved_now.append(q)
                        solved_at.setdefault(q, epoch)
                    if p_lower <= ph <= p_upper:
                        survivors.append(_Survivor(q, step, len(survivors)))
                for s in sorted((s for s in survivors if s.waiting()), key=lambda s: (s.born, s.order)):
                    if len(taken) == b_t:
                        break
                    s.taken_at = step
                    taken.append((s.prompt, s.born))
            stale = []
            for s in survivors:
                if s.waiting() and step - s.born >= d:
                    s.dropped_at = step
                    stale.append(s.prompt)
            log.append(dict(step=step, batch=piloted, rounds=rounds, selected=taken, solved=solved_now, stale=stale,
                            buffered=sum(1 for s in survivors if s.waiting()),
                            rollouts=len(piloted) * n_pilot + len(taken) * n_commit))
            step += 1
    return log
