"""Thin driver of one Pilot-Commit step on one GPU (Section 3.3; Algorithm 1, one iteration).

It only owns device memory (torch tensors), lays out the weights the way the C ABI
wants them, decides which rollouts are live at which step (known in advance: the
synthetic workloads end a rollout at its length cap, there is no end-of-sequence
token) and calls the library: pc_prefill_shared once per batch, then for the pilot
and for the commit stage pc_sample for the first token, pc_decode_step per step,
pc_reward_last_token, pc_group_stats, pc_allocate, pc_grpo_advantage.  No arithmetic
of the method happens here.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np
import torch

from . import binding as B
from .workloads import DTYPE_BF16, DTYPE_F32, Batch, ModelShape, Weights, Workload


def _dev_matrix(w: Weights, names: List[str], model: ModelShape, device, interleave: bool = False, half: bool = False) -> torch.Tensor:
    """Concatenates (or row-interleaves) matrices and uploads them in the model's storage type.

    half: a bf16 model's matrix is uploaded as IEEE half instead (same two bytes; a storage-format conversion of the
    bfloat16 value, exact unless the value is below 2^-14 in magnitude)."""
    if model.dtype == DTYPE_BF16 and half:
        parts = [torch.from_numpy((w.bits(n).astype(np.uint32) << 16).view(np.float32).astype(np.float16).view(np.int16)) for n in names]
    elif model.dtype == DTYPE_BF16:
        parts = [torch.from_numpy(w.bits(n).view(np.int16)) for n in names]
    else:
        parts = [torch.from_numpy(w[n]) for n in names]
    if interleave:
        assert len(parts) == 2
        t = torch.stack(parts, dim=1).reshape(-1, parts[0].shape[1])
    else:
        t = torch.cat(parts, dim=0) if len(parts) > 1 else parts[0]
    t = t.contiguous().to(device)
    return t.view(torch.bfloat16) if model.dtype == DTYPE_BF16 else t


STEP_DESC_DTYPE = np.dtype([("n_rows", np.int32), ("n_groups", np.int32), ("max_group_rows", np.int32), ("reserved", np.int32),
                            ("row_offset", np.int64), ("group_offset", np.int64)])


@dataclasses.dataclass
class StageSchedule:
    """Which rollouts are live at every decode step of one stage, flattened over steps and uploaded once."""
    n_steps: int
    rows_per_step: np.ndarray         # [n_steps]
    row_off: np.ndarray               # [n_steps] offset of the step's rows in the flat row arrays
    groups_per_step: np.ndarray       # [n_steps]
    group_off: np.ndarray             # [n_steps] offset in the flat group_row_start array
    max_group_rows: np.ndarray        # [n_steps]
    row_prompt: torch.Tensor
    row_rollout: torch.Tensor
    row_step: torch.Tensor
    row_kv_start: torch.Tensor
    row_tok_index: torch.Tensor
    group_row_start: torch.Tensor
    total_rows: int
    steps_host: np.ndarray            # [n_steps] records laid out like the C pc_step_desc
    steps_dev: torch.Tensor           # the same bytes on the device


class RolloutEngine:
    def __init__(self, model: ModelShape, weights: Weights, max_rows: int, max_prefill_tokens: int, device="cuda:0",
                 half_gemm: Optional[bool] = None):
        """half_gemm: hand the GEMM matrices of a bf16 model to the library as IEEE half (pc_model_desc.half_gemm); default
        on for bf16 models: the synthetic weights N(0, 0.02) and the unit-scale GEMM inputs sit well inside half's range."""
        self.model = model
        self.half_gemm = (model.dtype == DTYPE_BF16) if half_gemm is None else bool(half_gemm)
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        m, dev = model, self.device
        f32 = lambda n: torch.from_numpy(np.ascontiguousarray(weights[n], dtype=np.float32)).to(dev)
        L = range(m.n_layers)
        self.embed = _dev_matrix(weights, ["embed"], m, dev)
        hg = self.half_gemm
        lm_name = "embed" if m.tied_embed else "lm_head"
        self.lm_head = None if (m.tied_embed and not hg) else _dev_matrix(weights, [lm_name], m, dev, half=hg)
        self.final_norm = f32("final_norm")
        self.attn_norm = [f32(f"layers.{l}.attn_norm") for l in L]
        self.mlp_norm = [f32(f"layers.{l}.mlp_norm") for l in L]
        self.wqkv = [_dev_matrix(weights, [f"layers.{l}.wq", f"layers.{l}.wk", f"layers.{l}.wv"], m, dev, half=hg) for l in L]
        self.bqkv = [torch.cat([f32(f"layers.{l}.bq"), f32(f"layers.{l}.bk"), f32(f"layers.{l}.bv")]) for l in L] \
            if m.qkv_bias else None
        self.q_norm = [f32(f"layers.{l}.q_norm") for l in L] if m.qk_norm else None
        self.k_norm = [f32(f"layers.{l}.k_norm") for l in L] if m.qk_norm else None
        self.wo = [_dev_matrix(weights, [f"layers.{l}.wo"], m, dev, half=hg) for l in L]
        self.w_gate_up = [_dev_matrix(weights, [f"layers.{l}.w_gate", f"layers.{l}.w_up"], m, dev, interleave=True, half=self.half_gemm)
                          for l in L]
        self.w_down = [_dev_matrix(weights, [f"layers.{l}.w_down"], m, dev, half=self.half_gemm) for l in L]
        desc = B.ModelDesc(m.n_layers, m.d_model, m.n_q_heads, m.n_kv_heads, m.head_dim, m.d_ff, m.vocab, m.rms_eps,
                           m.rope_theta, m.dtype, int(m.tied_embed), int(m.qk_norm), int(m.qkv_bias), int(self.half_gemm))
        self.ctx = B.pc_create(desc, self.embed, self.lm_head, self.final_norm, self.attn_norm, self.wqkv, self.bqkv,
                               self.q_norm, self.k_norm, self.wo, self.mlp_norm, self.w_gate_up, self.w_down)
        self.max_rows, self.max_prefill = max_rows, max_prefill_tokens
        nbytes = B.pc_workspace_bytes(self.ctx, max_rows, max_prefill_tokens)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        self.err_flag = torch.zeros(1, dtype=torch.int32, device=dev)
        B.pc_set_workspace(self.ctx, self.workspace, max_rows, max_prefill_tokens, self.err_flag)
        self.kv_dtype = torch.float32 if m.dtype == DTYPE_F32 else torch.bfloat16
        # measurement: every `profile_every`-th decode step, time the operations of one layer and of the step's tail
        self._arenas: Dict[str, Optional[torch.Tensor]] = {}
        self.profile_every = 0
        self.use_graphs = True
        self.prompt_key_host: Optional[np.ndarray] = None    # sampling-key id per prompt (None: the prompt's index)
        self.collect_logprobs = False       # also keep log pi(o_t) of every sampled token (Eq. 2's denominator)
        self.record_pilot_logits: Optional[dict] = None     # {decode step: None} -> filled during the pilot stage
        self.record_commit_logits: Optional[dict] = None    # the same for the commit stage
        self.record_rows: Optional[set] = None              # keep only the logits rows of these (prompt, rollout) pairs
        self.profile_layer = m.n_layers // 2
        self.stage_rows_per_step: List[np.ndarray] = []      # live rows of every decode step, one array per stage run so far
        self.profile_samples: List[tuple] = []      # (events at the marks of binding.PROFILE_MARKS, rows, suffix slots read per row)

    # ------------------------------------------------------------------------------------------
    def kv_arena(self, n_slots: int, which: str) -> torch.Tensor:
        """An arena of n_slots slots; the previous arena of the same role is reused when it has the same size
        (two 75 GB arenas must never be alive together)."""
        m = self.model
        shape = (m.n_layers, 2, m.n_kv_heads, max(n_slots, 1), m.head_dim)
        old = self._arenas.get(which)
        if old is not None and tuple(old.shape) == shape:
            return old
        self._arenas[which] = None
        del old
        t = torch.empty(shape, dtype=self.kv_dtype, device=self.device)
        self._arenas[which] = t
        return t

    def check_error_flag(self) -> None:
        code = int(self.err_flag.item())
        if code != 0:
            raise RuntimeError(f"device error flag = {code}")

    # ------------------------------------------------------------------------------------------
    def load_batch(self, wl: Workload, batch: Batch, host_inputs: Optional[Dict[str, torch.Tensor]] = None) -> None:
        """Uploads the batch and allocates the KV arenas and every output buffer of the step."""
        dev, P, G = self.device, wl.n_prompts, wl.group_size
        self.wl, self.batch = wl, batch
        up = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dev, dtype=dt, non_blocking=True)
        if host_inputs is not None:           # pinned host buffers prepared by the caller (end-to-end timing)
            self.prompt_tokens = host_inputs["prompt_tokens"].to(dev, non_blocking=True)
            self.prompt_offsets = host_inputs["prompt_offsets"].to(dev, non_blocking=True)
        else:
            self.prompt_tokens = up(batch.prompt_tokens, torch.int32)
            self.prompt_offsets = up(batch.prompt_offsets, torch.int32)
        self.prompt_len = up(batch.prompt_lens, torch.int32)
        self.prompt_kv_start = up(batch.prompt_offsets[:-1].astype(np.int64), torch.int64)
        self.total_prompt_tokens = int(batch.prompt_offsets[-1])
        self.prompt_kv = self.kv_arena(self.total_prompt_tokens, "prompt")
        # every rollout (p, i) owns caps[p, i] suffix slots and max_new token cells
        caps = batch.caps.astype(np.int64)
        kv_start = np.zeros(P * G, dtype=np.int64)
        kv_start[1:] = np.cumsum(caps.reshape(-1))[:-1]
        self.kv_start_host = kv_start.reshape(P, G)
        self.suffix_slots = int(caps.sum())
        self.prompt_kv = self.prompt_kv
        self.suffix_kv = None
        self.suffix_kv = self.kv_arena(self.suffix_slots, "suffix")
        self.tokens = torch.full((P * G * wl.max_new,), -1, dtype=torch.int32, device=dev)
        self.logprobs = torch.zeros(P * G * wl.max_new, dtype=torch.float32, device=dev) if self.collect_logprobs else None
        B.pc_set_logprob_buffer(self.ctx, self.logprobs)
        B.pc_set_index_bounds(self.ctx, P, P * G * wl.max_new)
        self.prompt_key_host = None
        self.prompt_key_dev = None
        B.pc_set_prompt_keys(self.ctx, None)
        self.last_logits = torch.empty((P, self.model.vocab), dtype=torch.float32, device=dev)
        self.rewards = torch.zeros(P * G, dtype=torch.float32, device=dev)
        self.adv = torch.zeros(P * G, dtype=torch.float32, device=dev)
        self.thresholds = up(np.repeat(batch.reward_threshold, G), torch.int32)
        self.last_index = up((np.arange(P * G, dtype=np.int64) * wl.max_new + caps.reshape(-1) - 1), torch.int64)
        self.group_start = up(np.arange(P, dtype=np.int32) * G, torch.int32)
        i32 = lambda: torch.zeros(P, dtype=torch.int32, device=dev)
        f32 = lambda: torch.zeros(P, dtype=torch.float32, device=dev)
        self.pilot_n, self.pilot_success, self.pilot_mean, self.pilot_var = i32(), i32(), f32(), f32()
        self.union_n, self.union_success, self.union_mean, self.union_var = i32(), i32(), f32(), f32()
        self.status, self.extra, self.evict = i32(), i32(), i32()
        self.n_selected = torch.zeros(1, dtype=torch.int32, device=dev)
        self.total_rollouts = torch.zeros(1, dtype=torch.int64, device=dev)

    def prefill(self) -> None:
        b = self.batch
        B.pc_prefill_shared(self.ctx, self.wl.n_prompts, self.prompt_tokens, self.prompt_offsets, self.total_prompt_tokens,
                            int(b.prompt_lens.max()), self.prompt_kv, self.total_prompt_tokens, self.prompt_kv_start,
                            self.last_logits)

    # ------------------------------------------------------------------------------------------
    def build_schedule(self, prompts: np.ndarray, rollouts: np.ndarray) -> StageSchedule:
        """Rollouts (prompts[j], rollouts[j]), sorted by (prompt, rollout), all starting together.

        A rollout with cap c takes part in decode steps 0 .. c-2 (its c-th token needs no further forward)."""
        wl, dev = self.wl, self.device
        caps = self.batch.caps[prompts, rollouts].astype(np.int64)
        rid = prompts.astype(np.int64) * wl.group_size + rollouts
        kv0 = self.kv_start_host[prompts, rollouts]
        n_steps = int(max(caps.max() - 1, 0)) if len(caps) else 0
        rp, rr, rs, rk, rt, gs = [], [], [], [], [], []
        rows_per_step = np.zeros(n_steps, dtype=np.int64)
        groups_per_step = np.zeros(n_steps, dtype=np.int64)
        max_group = np.zeros(n_steps, dtype=np.int64)
        for s in range(n_steps):
            live = caps > s + 1
            p = prompts[live]
            rows_per_step[s] = p.shape[0]
            rp.append(p); rr.append(rollouts[live]); rk.append(kv0[live]); rt.append(rid[live] * wl.max_new + s)
            rs.append(np.full(p.shape[0], s, dtype=np.int32))
            starts = np.flatnonzero(np.r_[True, p[1:] != p[:-1]])
            bounds = np.r_[starts, p.shape[0]]
            groups_per_step[s] = starts.shape[0]
            max_group[s] = int(np.max(np.diff(bounds)))
            gs.append(bounds.astype(np.int32))
        cat = lambda xs, dt: torch.from_numpy(np.concatenate(xs).astype(dt) if xs else np.zeros(0, dt)).to(dev)
        row_off = np.r_[0, np.cumsum(rows_per_step)[:-1]] if n_steps else np.zeros(0, np.int64)
        group_off = np.r_[0, np.cumsum(groups_per_step + 1)[:-1]] if n_steps else np.zeros(0, np.int64)
        steps = np.zeros(n_steps, dtype=STEP_DESC_DTYPE)
        steps["n_rows"], steps["n_groups"], steps["max_group_rows"] = rows_per_step, groups_per_step, max_group
        steps["row_offset"], steps["group_offset"] = row_off, group_off
        steps_dev = torch.from_numpy(steps.view(np.uint8).reshape(-1).copy()).to(dev) if n_steps else torch.zeros(1, dtype=torch.uint8, device=dev)
        return StageSchedule(n_steps, rows_per_step, row_off, groups_per_step, group_off, max_group,
                             cat(rp, np.int32), cat(rr, np.int32), cat(rs, np.int32), cat(rk, np.int64), cat(rt, np.int64),
                             cat(gs, np.int32), int(rows_per_step.sum()), steps, steps_dev)

    def run_stage(self, prompts: np.ndarray, rollouts: np.ndarray, record_logits: Optional[dict] = None,
                  teacher_forced: bool = False, step_range: Optional[tuple] = None) -> int:
        """First token from the prompt's prefill logits, then the decode steps.  Returns tokens generated.

        record_logits: {step: None} asks for the logits of those decode steps (filled in place with
        (logits tensor, row prompts, row rollouts)).  teacher_forced: nothing is sampled; the token
        buffer must already hold every rollout's tokens and every step's logits must be recorded.
        step_range = (first, last): run only these decode steps (measurement of a step deep into a rollout;
        the token buffer and the KV slots before `first` must already hold finite values)."""
        wl, dev = self.wl, self.device
        n = int(prompts.shape[0])
        if n == 0:
            return 0
        sp = B.SampleParams(wl.temperature, wl.sample_seed)
        d_p = torch.from_numpy(prompts.astype(np.int32)).to(dev)
        d_r = torch.from_numpy(rollouts.astype(np.int32)).to(dev)
        d_key = d_p if self.prompt_key_host is None else torch.from_numpy(self.prompt_key_host[prompts].astype(np.int32)).to(dev)
        d_zero = torch.zeros(n, dtype=torch.int32, device=dev)
        rid = prompts.astype(np.int64) * wl.group_size + rollouts
        d_first = torch.from_numpy(rid * wl.max_new).to(dev)
        if not teacher_forced and step_range is None:
            B.pc_sample(n, self.model.vocab, self.last_logits, d_p, wl.temperature, wl.sample_seed, d_key, d_r, d_zero,
                        self.tokens, out_index=d_first)
            if self.logprobs is not None:
                B.pc_token_logprob(n, self.model.vocab, self.last_logits, d_p, wl.temperature, self.tokens, d_first, self.logprobs,
                                   d_first)
        sch = self.build_schedule(prompts, rollouts)
        pr, rr, rs = sch.row_prompt.data_ptr(), sch.row_rollout.data_ptr(), sch.row_step.data_ptr()
        rk, rt, gs = sch.row_kv_start.data_ptr(), sch.row_tok_index.data_ptr(), sch.group_row_start.data_ptr()
        first, last = (0, sch.n_steps) if step_range is None else (step_range[0], min(step_range[1], sch.n_steps))

        def eager(s):
            nr, o, go = int(sch.rows_per_step[s]), int(sch.row_off[s]), int(sch.group_off[s])
            logits_out = None
            if record_logits is not None and s in record_logits:
                logits_out = torch.empty((nr, self.model.vocab), dtype=torch.float32, device=dev)
                record_logits[s] = (logits_out, sch.row_prompt[o:o + nr].cpu().numpy(), sch.row_rollout[o:o + nr].cpu().numpy())
            if profiled(s):
                evs = [torch.cuda.Event(enable_timing=True) for _ in B.PROFILE_MARKS]
                for e in evs:
                    e.record()                       # creates the underlying CUDA events
                B.pc_profile_step(self.ctx, self.profile_layer, evs)
                self.profile_samples.append((evs, nr, s + 1))
            B.pc_decode_step(self.ctx, nr, pr + 4 * o, rr + 4 * o, rs + 4 * o, rk + 8 * o, self.tokens, rt + 8 * o,
                             int(sch.groups_per_step[s]), gs + 4 * go, int(sch.max_group_rows[s]), self.prompt_len,
                             self.prompt_kv, self.total_prompt_tokens, self.prompt_kv_start, self.suffix_kv,
                             self.suffix_slots, logits_out, None if teacher_forced else sp)
            if logits_out is not None and self.record_rows is not None:
                _, rec_p, rec_r = record_logits[s]
                keep = np.flatnonzero([(int(a), int(b)) in self.record_rows for a, b in zip(rec_p, rec_r)])
                record_logits[s] = (logits_out[torch.from_numpy(keep).to(dev)].clone(), rec_p[keep], rec_r[keep])

        def profiled(s):
            return bool(self.profile_every) and s % self.profile_every == self.profile_every // 2

        def needs_eager(s):
            return teacher_forced or not self.use_graphs or (record_logits is not None and s in record_logits) or profiled(s)

        s = first
        while s < last:
            if needs_eager(s):
                eager(s)
                s += 1
                continue
            e = s
            while e < last and not needs_eager(e):
                e += 1
            # steps s .. e-1 natively: one graph launch per step, issued by the library
            item = STEP_DESC_DTYPE.itemsize
            B.pc_decode_run(self.ctx, e - s, sch.steps_host.ctypes.data + s * item, sch.steps_dev.data_ptr() + s * item,
                            pr, rr, rs, rk, self.tokens, rt, gs, self.prompt_len, self.prompt_kv, self.total_prompt_tokens,
                            self.prompt_kv_start, self.suffix_kv, self.suffix_slots, sp)
            s = e
        self._keep_schedule = sch
        self.stage_rows_per_step.append(sch.rows_per_step.copy())
        return int(self.batch.caps[prompts, rollouts].sum())

    # ------------------------------------------------------------------------------------------
    def pilot_commit_step(self, wl: Workload, batch: Batch, b_t: Optional[int] = None,
                          host_inputs: Optional[Dict[str, torch.Tensor]] = None) -> dict:
        """The whole step.  Returns host copies of every output plus token counts."""
        self.load_batch(wl, batch, host_inputs)
        status, n_tok = self.run_device(b_t)
        out = self.collect(status)
        out["generated_tokens"] = n_tok
        return out

    def run_device(self, b_t: Optional[int] = None):
        """Everything between the uploaded batch and the finished advantages: prefill, pilot stage, statistics,
        allocation, commit stage, union statistics, advantages.  Returns (status on the host, tokens generated)."""
        wl = self.wl
        P, G, k = wl.n_prompts, wl.group_size, wl.n_pilot
        b_t = P if b_t is None else b_t
        self.prefill_events = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
        self.prefill_events[0].record()
        self.prefill()
        self.prefill_events[1].record()
        pp, rr = np.repeat(np.arange(P), k), np.tile(np.arange(k), P)
        n_tok = self.run_stage(pp, rr, record_logits=self.record_pilot_logits)
        pilot_count = torch.full((P,), k, dtype=torch.int32, device=self.device)
        B.pc_reward_last_token(P * G, self.tokens, self.last_index, self.thresholds, self.rewards)
        B.pc_group_stats(P, self.rewards, self.group_start, pilot_count, self.pilot_n, self.pilot_success, self.pilot_mean,
                         self.pilot_var)
        B.pc_allocate(P, self.pilot_success, self.pilot_n, B.AllocParams(wl.p_lower, wl.p_upper, wl.p_solve, G - k, b_t),
                      self.status, self.extra, self.evict, self.n_selected, self.total_rollouts)
        status = self.status.cpu().numpy()            # the commit stage's row set depends on it
        commit = np.flatnonzero(status == B.PC_STATUS_COMMIT)
        if G > k and commit.size:
            n_tok += self.run_stage(np.repeat(commit, G - k), np.tile(np.arange(k, G), commit.size),
                                    record_logits=self.record_commit_logits)
        B.pc_reward_last_token(P * G, self.tokens, self.last_index, self.thresholds, self.rewards)
        union_count = torch.from_numpy(np.where(status == B.PC_STATUS_COMMIT, G, k).astype(np.int32)).to(self.device)
        B.pc_group_stats(P, self.rewards, self.group_start, union_count, self.union_n, self.union_success, self.union_mean,
                         self.union_var)
        B.pc_grpo_advantage(P, self.rewards, self.group_start, union_count, self.status, self.adv)
        return status, n_tok

    def bound_pass(self, wl: Workload, batch_a: Batch, commit_a: np.ndarray, batch_b: Batch) -> dict:
        """Section 3.4, "Binding pilot and commit": ONE inference pass that generates the commit rollouts (k .. G-1) of the
        prompts `commit_a` of batch A together with the pilot rollouts (0 .. k-1) of the new batch B.

        Must follow the pass that ran A's pilot rollouts on this engine: A's prompt KV and last-position logits are taken
        over from it (the prompt is not evaluated again), B is prefilled.  Rollouts keep the sampling keys they would have
        had in separate passes, so their tokens do not depend on the binding.
        Returns {"a": {(p, i): tokens}, "b": {(p, i): tokens}} with the prompts' indices in their own batches."""
        dev, G, k = self.device, wl.group_size, wl.n_pilot
        commit_a = np.asarray(commit_a, dtype=np.int64)
        nA, PB = len(commit_a), len(batch_b.prompt_lens)
        old_kv, old_start, old_last = self.prompt_kv, self.batch.prompt_offsets[:-1].astype(np.int64), self.last_logits
        lens = np.concatenate([batch_a.prompt_lens[commit_a], batch_b.prompt_lens]).astype(np.int32)
        offsets = np.zeros(nA + PB + 1, dtype=np.int32)
        offsets[1:] = np.cumsum(lens)
        toks_a = [batch_a.prompt_tokens[batch_a.prompt_offsets[p]:batch_a.prompt_offsets[p + 1]] for p in commit_a]
        comb = Batch(lens, offsets, np.concatenate(toks_a + [batch_b.prompt_tokens]).astype(np.int32),
                     np.concatenate([batch_a.tau[commit_a], batch_b.tau]),
                     np.concatenate([batch_a.reward_threshold[commit_a], batch_b.reward_threshold]).astype(np.int32),
                     np.concatenate([batch_a.caps[commit_a], batch_b.caps]).astype(np.int32))
        wl_c = dataclasses.replace(wl, n_prompts=nA + PB)
        self._arenas["prompt"] = None                       # keep A's arena alive through old_kv while the new one is filled
        self.load_batch(wl_c, comb)
        for j, p in enumerate(commit_a):                    # A's prompt KV stays what its own pass computed
            L, s_old, s_new = int(batch_a.prompt_lens[p]), int(old_start[p]), int(offsets[j])
            self.prompt_kv[:, :, :, s_new:s_new + L] = old_kv[:, :, :, s_old:s_old + L]
        self.last_logits[:nA] = old_last[torch.from_numpy(commit_a).to(dev)]
        if PB:
            off0 = int(offsets[nA])
            offs_b = torch.from_numpy((offsets[nA:] - off0).astype(np.int32)).to(dev)
            B.pc_prefill_shared(self.ctx, PB, self.prompt_tokens[off0:], offs_b, int(offsets[-1]) - off0,
                                int(batch_b.prompt_lens.max()), self.prompt_kv, self.total_prompt_tokens,
                                self.prompt_kv_start[nA:], self.last_logits[nA:])
        self.prompt_key_host = np.concatenate([commit_a, np.arange(PB)]).astype(np.int32)
        self.prompt_key_dev = torch.from_numpy(self.prompt_key_host).to(dev)
        B.pc_set_prompt_keys(self.ctx, self.prompt_key_dev)
        prompts = np.concatenate([np.repeat(np.arange(nA), G - k), np.repeat(nA + np.arange(PB), k)])
        rollouts = np.concatenate([np.tile(np.arange(k, G), nA), np.tile(np.arange(k), PB)])
        self.run_stage(prompts, rollouts, record_logits=self.record_pilot_logits)
        self.check_error_flag()
        toks = self.tokens.cpu().numpy().reshape(nA + PB, G, wl.max_new)
        out = {"a": {}, "b": {}}
        for j, p in enumerate(commit_a):
            for i in range(k, G):
                out["a"][(int(p), i)] = toks[j, i, :batch_a.caps[p, i]].copy()
        for p in range(PB):
            for i in range(k):
                out["b"][(p, i)] = toks[nA + p, i, :batch_b.caps[p, i]].copy()
        return out

    def collect(self, status: np.ndarray) -> dict:
        wl, P, G, k = self.wl, self.wl.n_prompts, self.wl.group_size, self.wl.n_pilot
        self.check_error_flag()
        toks = self.tokens.cpu().numpy().reshape(P, G, wl.max_new)
        generated = np.zeros((P, G), dtype=bool)
        generated[:, :k] = True
        generated[status == B.PC_STATUS_COMMIT, :] = True
        tokens = [[toks[p, i, :self.batch.caps[p, i]].copy() if generated[p, i] else None for i in range(G)] for p in range(P)]
        rewards = self.rewards.cpu().numpy().reshape(P, G).copy()
        rewards[~generated] = 0.0          # cells of rollouts that were never generated hold no reward
        h = lambda t: t.cpu().numpy()
        return dict(tokens=tokens, rewards=rewards, generated=generated,
                    pilot_n=h(self.pilot_n), pilot_success=h(self.pilot_success), pilot_mean=h(self.pilot_mean),
                    pilot_var=h(self.pilot_var), status=status, extra=h(self.extra), evict=h(self.evict),
                    n_selected=int(self.n_selected.item()), total_rollouts=int(self.total_rollouts.item()),
                    union_n=h(self.union_n), union_success=h(self.union_success), union_mean=h(self.union_mean),
                    union_var=h(self.union_var), advantages=h(self.adv).reshape(P, G),
                    logprobs=None if self.logprobs is None else h(self.logprobs).reshape(P, G, wl.max_new))
