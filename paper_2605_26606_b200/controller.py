"""Host-side bookkeeping of Pilot-Commit across training steps (Section 3.4; Algorithm 1): the replay buffer of pilot
survivors with its maximum age d, the per-step choice of the b_t prompts that receive commit rollouts, and the set of
solved prompts evicted from later epochs.

The per-prompt decisions (filter, eviction flag) come from the device (`pc_allocate` called with b_t = batch size, so
that every survivor is reported as kept); this class only remembers them between steps.  It holds no tensors.

Readings where Algorithm 1 leaves a choice: survivors are committed oldest first (ties in arrival order) -- the
algorithm leaves the draw from the buffer unspecified; a committed prompt leaves the buffer; d is the maximum delay
between a prompt's pilot and its commit (Section 4.2), so after the commits of step t the entries whose pilot ran at
step t - d or earlier are dropped: the next step could not use them within the delay.  A training step may take more
than one sampling batch: when the first one leaves fewer than b_t prompts selected, Section 6.3 speaks of a second
sampling round to fill the training batch; `begin_step` / `add_round` / `end_step` expose that, `step` is the
single-round form.
"""
from __future__ import annotations

import collections
import dataclasses
from typing import Deque, Iterable, List, Sequence, Set, Tuple


@dataclasses.dataclass
class StepPlan:
    step: int
    committed: List[Tuple[int, int]]     # (prompt id, step its pilot rollouts were drawn), oldest first
    newly_evicted: List[int]
    dropped_stale: List[int]
    buffered_after: int
    rollouts_sampled: int                # pilots of every round + |committed| n_commit  (Section 4.3)
    rounds: int = 1                      # sampling batches this training step consumed (Section 6.3)


class PilotCommitController:
    def __init__(self, n_pilot: int, n_commit: int, b_t: int, max_delay: int):
        if min(n_pilot, b_t) <= 0 or n_commit < 0 or max_delay < 0:
            raise ValueError("n_pilot and b_t must be positive, n_commit and max_delay non-negative")
        self.n_pilot, self.n_commit, self.b_t, self.d = n_pilot, n_commit, b_t, max_delay
        self.t = 0
        self.buffer: Deque[Tuple[int, int]] = collections.deque()     # (prompt id, birth step), in arrival order
        self.evicted: Set[int] = set()

    def sampling_pool(self, dataset: Iterable[int]) -> List[int]:
        """The prompts still eligible for pilot rollouts (solved ones stay out of later epochs)."""
        return [q for q in dataset if q not in self.evicted]

    def begin_step(self) -> None:
        self._selected: List[Tuple[int, int]] = []
        self._newly: List[int] = []
        self._rounds = 0
        self._piloted = 0

    @property
    def need_more(self) -> bool:
        """True while the training batch of the current step is not full."""
        return len(self._selected) < self.b_t

    def add_round(self, batch_ids: Sequence[int], kept: Sequence[int], evict: Sequence[int]) -> List[Tuple[int, int]]:
        """One sampling batch whose pilot results are in.  Returns the prompts this round adds to the training batch.

        kept[i] / evict[i]: the pilot filter and the eviction rule for batch_ids[i] (non-zero = true)."""
        if not (len(batch_ids) == len(kept) == len(evict)):
            raise ValueError("batch_ids, kept and evict must have the same length")
        for q, k, e in zip(batch_ids, kept, evict):
            if e and q not in self.evicted:
                self.evicted.add(q)
                self._newly.append(q)
            if k:
                self.buffer.append((q, self.t))
        take = min(self.b_t - len(self._selected), len(self.buffer))
        added = [self.buffer.popleft() for _ in range(take)]
        self._selected += added
        self._rounds += 1
        self._piloted += len(batch_ids)
        return added

    def end_step(self) -> StepPlan:
        stale = [q for q, born in self.buffer if self.t - born >= self.d]
        if stale:
            self.buffer = collections.deque((q, born) for q, born in self.buffer if self.t - born < self.d)
        plan = StepPlan(self.t, self._selected, self._newly, stale, len(self.buffer),
                        self._piloted * self.n_pilot + len(self._selected) * self.n_commit, self._rounds)
        self.t += 1
        return plan

    def step(self, batch_ids: Sequence[int], kept: Sequence[int], evict: Sequence[int]) -> StepPlan:
        """One iteration of Algorithm 1's inner loop with a single sampling batch."""
        if not (len(batch_ids) == len(kept) == len(evict)):
            raise ValueError("batch_ids, kept and evict must have the same length")
        self.begin_step()
        self.add_round(batch_ids, kept, evict)
        return self.end_step()
