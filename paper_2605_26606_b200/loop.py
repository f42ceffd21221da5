"""Several consecutive Pilot-Commit training steps on one GPU (Algorithm 1; Section 3.4): the host controller (replay
buffer, delay d, eviction, second sampling round) drives the rollout engine.

What stays resident between passes: the prompt KV and the last-position logits of every prompt that is still waiting for
its commit rollouts (a pool of slot ranges in one persistent prompt arena -- nothing is copied or evaluated twice), and the
token cells of its pilot rollouts, so that the union of pilot and commit rollouts is complete when the prompt commits.

With `bind=True` a pass holds the commit rollouts of the prompts selected in the previous round together with the pilot
rollouts of the next sampling batch (Section 3.4, "Binding pilot and commit"); otherwise every round is a pilot pass
followed by a commit pass.  Rollouts are keyed by (seed, dataset prompt id, rollout, step), so neither choice changes a
token.  Only driver code lives here: every computation is a call into the library.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

from . import binding as B
from .controller import PilotCommitController, StepPlan
from .engine import RolloutEngine
from .workloads import Batch, Workload


class SlotPool:
    """First-fit allocator of contiguous slot ranges (host bookkeeping for the persistent prompt arena)."""

    def __init__(self, capacity: int):
        self.free: List[Tuple[int, int]] = [(0, capacity)]        # (start, length), sorted by start

    def alloc(self, n: int) -> int:
        for j, (s, l) in enumerate(self.free):
            if l >= n:
                if l == n:
                    self.free.pop(j)
                else:
                    self.free[j] = (s + n, l - n)
                return s
        raise MemoryError("prompt arena exhausted")

    def release(self, start: int, n: int) -> None:
        self.free.append((start, n))
        self.free.sort()
        merged: List[Tuple[int, int]] = []
        for s, l in self.free:
            if merged and merged[-1][0] + merged[-1][1] == s:
                merged[-1] = (merged[-1][0], merged[-1][1] + l)
            else:
                merged.append((s, l))
        self.free = merged


@dataclasses.dataclass
class StepRecord:
    plan: StepPlan
    batches: List[List[int]]                       # dataset ids piloted, per round
    pilot_success: Dict[int, int]                  # dataset id -> successes among its pilot rollouts
    tokens: Dict[Tuple[int, int], np.ndarray]      # (dataset id, rollout) -> tokens of every rollout that finished in this step
    rewards: Dict[Tuple[int, int], float]
    advantages: Dict[int, np.ndarray]              # committed prompt -> advantages over its union group [G]
    passes: int


class RolloutLoop:
    def __init__(self, eng: RolloutEngine, wl: Workload, dataset: Batch, b_g: int, b_t: int, max_delay: int, max_rounds: int = 1,
                 bind: bool = True, max_resident_prompts: Optional[int] = None, prompt_slots: Optional[int] = None):
        """dataset: one Batch holding every prompt of the data set (prompt q = its entry q); wl gives G, k, seeds, thresholds."""
        self.eng, self.wl, self.data = eng, wl, dataset
        self.b_g, self.b_t, self.bind, self.max_rounds = b_g, b_t, bind, max_rounds
        G, k = wl.group_size, wl.n_pilot
        self.ctl = PilotCommitController(k, G - k, b_t, max_delay)
        dev = eng.device
        # room for one sampling batch per round plus everything that may wait in the buffer
        R = max_resident_prompts or (b_g * (max_rounds + 1) + b_t * (max_delay + 2))
        self.R = R
        max_len = int(dataset.prompt_lens.max())
        self.slots = SlotPool(prompt_slots or R * max_len)
        self.capacity_slots = prompt_slots or R * max_len
        self.free_rows = list(range(R))[::-1]
        self.row_of: Dict[int, int] = {}                 # dataset id -> pool row
        self.slot_of: Dict[int, Tuple[int, int]] = {}
        # engine state shaped for R resident prompts; run_stage indexes prompts by pool row
        eng.wl = dataclasses.replace(wl, n_prompts=R)
        eng.batch = Batch(np.zeros(R, np.int32), np.zeros(R + 1, np.int32), np.zeros(0, np.int32), np.zeros(R), np.zeros(R, np.int32),
                          np.ones((R, G), np.int32))
        eng.prompt_kv = eng.kv_arena(self.capacity_slots, "prompt")
        eng.total_prompt_tokens = self.capacity_slots
        eng.tokens = torch.full((R * G * wl.max_new,), -1, dtype=torch.int32, device=dev)
        eng.logprobs = None
        B.pc_set_logprob_buffer(eng.ctx, None)
        B.pc_set_index_bounds(eng.ctx, R, R * G * wl.max_new)
        eng.last_logits = torch.zeros((R, eng.model.vocab), dtype=torch.float32, device=dev)
        eng.prompt_key_host = np.zeros(R, np.int32)
        eng.kv_start_host = np.zeros((R, G), np.int64)
        eng.rewards = torch.zeros(R * G, dtype=torch.float32, device=dev)
        eng.adv = torch.zeros(R * G, dtype=torch.float32, device=dev)
        self.group_start = torch.arange(R, dtype=torch.int32, device=dev) * G
        self.passes = 0

    # -- residency ---------------------------------------------------------------------------------------------
    def _admit(self, ids: Sequence[int]) -> None:
        """Prefills the prompts `ids` into free ranges of the persistent arena (one pc_prefill_shared call)."""
        eng, d, dev = self.eng, self.data, self.eng.device
        rows, lens, starts, toks = [], [], [], []
        for q in ids:
            r = self.free_rows.pop()
            L = int(d.prompt_lens[q])
            s = self.slots.alloc(L)
            self.row_of[q], self.slot_of[q] = r, (s, L)
            rows.append(r); lens.append(L); starts.append(s)
            toks.append(d.prompt_tokens[d.prompt_offsets[q]:d.prompt_offsets[q + 1]])
            eng.batch.prompt_lens[r] = L
            eng.batch.caps[r] = d.caps[q]
            eng.batch.reward_threshold[r] = d.reward_threshold[q]
            eng.prompt_key_host[r] = q
        eng.tokens.view(self.R, -1)[torch.tensor(rows, device=dev)] = -1
        offsets = np.zeros(len(ids) + 1, np.int32)
        offsets[1:] = np.cumsum(lens)
        logits = torch.empty((len(ids), eng.model.vocab), dtype=torch.float32, device=dev)
        B.pc_prefill_shared(eng.ctx, len(ids), torch.from_numpy(np.concatenate(toks).astype(np.int32)).to(dev),
                            torch.from_numpy(offsets).to(dev), int(offsets[-1]), int(max(lens)), eng.prompt_kv, self.capacity_slots,
                            torch.tensor(starts, dtype=torch.int64, device=dev), logits)
        eng.last_logits[torch.tensor(rows, device=dev)] = logits
        self._upload_prompt_tables()

    def _upload_prompt_tables(self) -> None:
        eng, dev = self.eng, self.eng.device
        starts = np.zeros(self.R, np.int64)
        for q, r in self.row_of.items():
            starts[r] = self.slot_of[q][0]
        eng.prompt_len = torch.from_numpy(eng.batch.prompt_lens.astype(np.int32)).to(dev)
        eng.prompt_kv_start = torch.from_numpy(starts).to(dev)
        eng.prompt_key_dev = torch.from_numpy(eng.prompt_key_host.astype(np.int32)).to(dev)
        B.pc_set_prompt_keys(eng.ctx, eng.prompt_key_dev)
        eng.thresholds = torch.from_numpy(np.repeat(eng.batch.reward_threshold, self.wl.group_size).astype(np.int32)).to(dev)
        caps = eng.batch.caps.astype(np.int64).reshape(-1)
        eng.last_index = torch.from_numpy(np.arange(caps.shape[0], dtype=np.int64) * self.wl.max_new + caps - 1).to(dev)

    def _release(self, q: int) -> None:
        r = self.row_of.pop(q)
        s, L = self.slot_of.pop(q)
        self.slots.release(s, L)
        self.free_rows.append(r)

    # -- one inference pass ------------------------------------------------------------------------------------
    def _run_pass(self, items: List[Tuple[int, int]]) -> None:
        """Decodes the rollouts `items` = (dataset id, rollout) to completion in one decode batch."""
        if not items:
            return
        eng = self.eng
        rows = np.array([self.row_of[q] for q, _ in items], dtype=np.int64)
        rolls = np.array([i for _, i in items], dtype=np.int64)
        order = np.lexsort((rolls, rows))
        rows, rolls = rows[order], rolls[order]
        caps = eng.batch.caps[rows, rolls].astype(np.int64)
        start = np.zeros(len(items), np.int64)
        start[1:] = np.cumsum(caps)[:-1]
        eng.kv_start_host[rows, rolls] = start
        eng.suffix_slots = int(caps.sum())
        eng.suffix_kv = eng.kv_arena(eng.suffix_slots, "suffix")
        eng.run_stage(rows, rolls)
        self.passes += 1

    def _pilot_results(self, ids: Sequence[int]):
        """Rewards, group statistics and the pilot filter / eviction flags of the prompts `ids` (device calls, host copies)."""
        eng, G, k = self.eng, self.wl.group_size, self.wl.n_pilot
        dev = eng.device
        rows = torch.tensor([self.row_of[q] for q in ids], dtype=torch.int64, device=dev)
        n = len(ids)
        B.pc_reward_last_token(self.R * G, eng.tokens, eng.last_index, eng.thresholds, eng.rewards)
        start = self.group_start[rows].contiguous()
        cnt = torch.full((n,), k, dtype=torch.int32, device=dev)
        i32 = lambda: torch.zeros(n, dtype=torch.int32, device=dev)
        f32 = lambda: torch.zeros(n, dtype=torch.float32, device=dev)
        pn, pm, mean, var = i32(), i32(), f32(), f32()
        B.pc_group_stats(n, eng.rewards, start, cnt, pn, pm, mean, var)
        status, extra, evict = i32(), i32(), i32()
        nsel, total = torch.zeros(1, dtype=torch.int32, device=dev), torch.zeros(1, dtype=torch.int64, device=dev)
        w = self.wl
        # b_t = batch size: every survivor is reported as kept; how many commit when is the controller's decision
        B.pc_allocate(n, pm, pn, B.AllocParams(w.p_lower, w.p_upper, w.p_solve, G - k, n), status, extra, evict, nsel, total)
        return pm.cpu().numpy(), status.cpu().numpy() == B.PC_STATUS_COMMIT, evict.cpu().numpy()

    def _finish_committed(self, committed: Sequence[int], rec: StepRecord) -> None:
        """Union statistics and advantages of prompts whose commit rollouts are done; copies their rollouts out, frees them."""
        if not committed:
            return
        eng, G = self.eng, self.wl.group_size
        dev = eng.device
        rows = torch.tensor([self.row_of[q] for q in committed], dtype=torch.int64, device=dev)
        n = len(committed)
        B.pc_reward_last_token(self.R * G, eng.tokens, eng.last_index, eng.thresholds, eng.rewards)
        start = self.group_start[rows].contiguous()
        cnt = torch.full((n,), G, dtype=torch.int32, device=dev)
        B.pc_grpo_advantage(n, eng.rewards, start, cnt, None, eng.adv)
        toks = eng.tokens.view(self.R, G, -1).cpu().numpy()
        rew, adv = eng.rewards.view(self.R, G).cpu().numpy(), eng.adv.view(self.R, G).cpu().numpy()
        for q in committed:
            r = self.row_of[q]
            for i in range(G):
                rec.tokens[(q, i)] = toks[r, i, :eng.batch.caps[r, i]].copy()
                rec.rewards[(q, i)] = float(rew[r, i])
            rec.advantages[q] = adv[r].copy()
            self._release(q)

    # -- the loop ----------------------------------------------------------------------------------------------
    def run(self, dataset_ids: Sequence[int], n_epochs: int, max_steps: Optional[int] = None) -> List[StepRecord]:
        G, k = self.wl.group_size, self.wl.n_pilot
        out: List[StepRecord] = []
        pending: List[int] = []                 # selected prompts whose commit rollouts ride on the next pass (bind)
        pending_rec: Optional[StepRecord] = None
        for _ in range(n_epochs):
            pool = self.ctl.sampling_pool(dataset_ids)
            cursor = 0
            while cursor < len(pool) and (max_steps is None or len(out) < max_steps):
                self.ctl.begin_step()
                rec = StepRecord(None, [], {}, {}, {}, {}, 0)
                p0 = self.passes
                while cursor < len(pool) and self.ctl._rounds < self.max_rounds and (self.ctl._rounds == 0 or self.ctl.need_more):
                    batch = list(pool[cursor:cursor + self.b_g])
                    cursor += len(batch)
                    rec.batches.append(batch)
                    self._admit(batch)
                    items = [(q, i) for q in batch for i in range(k)]
                    if self.bind and pending:
                        items += [(q, i) for q in pending for i in range(k, G)]
                    self._run_pass(items)
                    if self.bind and pending:
                        self._finish_committed(pending, pending_rec)
                        pending, pending_rec = [], None
                    pm, kept, evict = self._pilot_results(batch)
                    for q, m in zip(batch, pm):
                        rec.pilot_success[q] = int(m)
                    added = [q for q, _ in self.ctl.add_round(batch, kept, evict)]
                    for q, keep in zip(batch, kept):               # prompts the filter dropped leave at once
                        if not keep:
                            self._copy_out_pilot(q, rec)
                            self._release(q)
                    if self.bind:
                        pending += added
                        pending_rec = rec
                    else:
                        self._run_pass([(q, i) for q in added for i in range(k, G)])
                        self._finish_committed(added, rec)
                rec.plan = self.ctl.end_step()
                for q in rec.plan.dropped_stale:
                    self._copy_out_pilot(q, rec)
                    self._release(q)
                rec.passes = self.passes - p0
                out.append(rec)
        if pending:                                                # commit rollouts of the last round
            self._run_pass([(q, i) for q in pending for i in range(k, G)])
            self._finish_committed(pending, pending_rec)
            pending_rec.passes += 1
        self.eng.check_error_flag()
        return out

    def _copy_out_pilot(self, q: int, rec: StepRecord) -> None:
        eng, k = self.eng, self.wl.n_pilot
        r = self.row_of[q]
        toks = eng.tokens.view(self.R, self.wl.group_size, -1)[r, :k].cpu().numpy()
        rew = eng.rewards.view(self.R, self.wl.group_size)[r, :k].cpu().numpy()
        for i in range(k):
            rec.tokens[(q, i)] = toks[i, :eng.batch.caps[r, i]].copy()
            rec.rewards[(q, i)] = float(rew[i])
