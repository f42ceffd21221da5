"""Benchmark of the Pilot-Commit rollout hot path on B200.

    python bench.py --gpus N --steps K --warmup W                 (N > 1: launched through torch.distributed.run)
    python bench.py --impl reference --gpus N --steps K --warmup W  (the CPU oracle on the host cores)

One step = one pass of the whole hot path over one sampling batch: shared prefill of every prompt, the pilot
stage (k rollouts per prompt), rewards, group statistics, pilot filter / eviction / commit allocation, the
commit stage (G - k more rollouts for the selected prompts, on the same resident prompt KV), union statistics
and GRPO advantages.  Metric: generated tokens per second.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_26606_b200 import dist_util  # noqa: E402
from paper_2605_26606_b200 import workloads as wl  # noqa: E402

# DRAM traffic of the suffix attention kernel per algorithmic byte, from the ncu capture summarised in
# profiles/attn_suffix_kernel_ncu.md (304 rollouts x 513 slots: 168.98 MB moved for 161.6 MB algorithmic).  The kernel
# streams every (rollout, KV head) suffix once, so traffic grows in proportion to the algorithmic bytes of a launch.
SUFFIX_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.046
METRIC = "generated tokens/s"
UNIT = "tokens/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        super().__init__(daemon=True)
        self.gpu_index, self.lines, self.proc = gpu_index, [], None

    def run(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "500"], stdout=subprocess.PIPE, text=True)
            for line in self.proc.stdout:
                self.lines.append(line.strip())
        except Exception:
            pass

    def stop(self) -> dict:
        if self.proc is not None:
            self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": float(np.max(mx)) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(w, weights, batch, n_rollouts=2, n_tokens=3):
    """The CPU oracle, as it stands, on a bounded sample of the workload: the shortest prompt of the batch is
    prefilled and n_rollouts rollouts of n_tokens tokens each are generated with the cached decoder.
    Returns (tokens generated, seconds, threads used)."""
    from oracle import rollout as orollout
    from oracle.decoder import Decoder
    try:
        import threadpoolctl
        threads = max([p["num_threads"] for p in threadpoolctl.threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        threads = os.cpu_count() or 1
    dec = Decoder(w.model, weights, cache_weights=False)
    p = int(np.argmin(batch.prompt_lens))
    pt = batch.prompt_tokens[batch.prompt_offsets[p]:batch.prompt_offsets[p + 1]]
    t0 = time.perf_counter()
    out = orollout.generate_group(dec, pt, p, list(range(n_rollouts)), [n_tokens] * n_rollouts, w.sample_seed, w.temperature)
    dt = time.perf_counter() - t0
    n = sum(len(v) for v in out.values())
    desc = (f"prompt {p} ({len(pt)} tokens) prefilled once, {n_rollouts} rollouts x {n_tokens} tokens, KV-cached decode, "
            f"float64 numpy")
    return n, dt, threads, desc


def run_reference(args):
    rank, _, world = dist_util.env_world()
    if rank != 0:
        return
    w = wl.WORKLOADS[args.config]
    weights = wl.gen_weights(w.model, seed=0)
    batch = wl.gen_batch(w)
    times, toks, threads, desc = [], 0, 1, ""
    for i in range(args.warmup + args.steps):
        n, dt, threads, desc = oracle_sample(w, weights, batch)
        if i >= args.warmup:
            times.append(dt); toks += n
    total = sum(times)
    value = toks / total
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * total / max(args.steps, 1), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "model": w.model.name, "sample": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_probe(args):
    """Decode-step microbenchmark: R rollouts in 16 groups, every rollout S tokens deep, N steps timed."""
    import torch
    from paper_2605_26606_b200 import binding as B
    from paper_2605_26606_b200 import build as _build
    from paper_2605_26606_b200.engine import RolloutEngine
    _build.build()
    kv = dict(x.split("=") for x in args.probe.split(","))
    rows, suffix, steps, plen = int(kv.get("rows", 256)), int(kv.get("suffix", 512)), int(kv.get("steps", 4)), int(kv.get("prompt", 640))
    base = wl.WORKLOADS[args.config]
    P = min(16, rows)
    G = rows // P
    cap = suffix + steps + 1
    w = dataclasses.replace(base, n_prompts=P, group_size=G, n_pilot=G, prompt_len_lo=plen, prompt_len_hi=plen, max_new=cap,
                            cap_lo=cap, cap_hi=cap, forced_frac=0.0, forced_explicit=None)
    weights = wl.gen_weights(w.model, seed=0)
    batch = wl.gen_batch(w)
    eng = RolloutEngine(w.model, weights, max_rows=P * G, max_prefill_tokens=int(batch.prompt_offsets[-1]))
    eng.use_graphs = kv.get("graphs", "1") != "0"
    B.pc_set_decode_mode(eng.ctx, int(kv.get("mode", 1)))
    eng.load_batch(w, batch)
    eng.suffix_kv.zero_()
    eng.tokens.random_(0, w.model.vocab)
    eng.prefill()
    pp, rr = np.repeat(np.arange(P), G), np.tile(np.arange(G), P)
    eng.run_stage(pp, rr, step_range=(suffix, suffix + 2))            # warm-up
    torch.cuda.synchronize()
    l0 = B.pc_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    t0 = time.perf_counter()
    eng.run_stage(pp, rr, step_range=(suffix, suffix + steps))
    host_ms = (time.perf_counter() - t0) * 1e3 / steps          # time the host needs to issue one step
    e1.record()
    torch.cuda.synchronize()
    eng.check_error_flag()
    ms = e0.elapsed_time(e1) / steps
    m = w.model
    bytes_step = m.weight_bytes_per_decode_step() + (P * G * (suffix + 1) + P * plen) * m.kv_bytes_per_token
    peak, kind = load_peaks()
    print(json.dumps({"probe": {"rows": P * G, "suffix": suffix, "steps": steps, "prompt_len": plen}, "ms_per_decode_step": ms, "host_issue_ms_per_step": host_ms,
                      "tokens_per_s": P * G / (ms * 1e-3), "launches_per_step": (B.pc_launch_count() - l0) / steps,
                      "hbm_bytes_per_step": bytes_step, "hbm_frac": bytes_step / (ms * 1e-3) / 1e9 / peak, "peak_kind": kind}),
          flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="config2", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--also-bound", action="store_true",
                    help="additionally time one bound pass (Section 3.4): the commit rollouts of the timed batch's survivors and the "
                         "pilot rollouts of a second batch in one decode batch; reported as bound_pass")
    ap.add_argument("--also-logprobs", action="store_true",
                    help="additionally time one step that also keeps the behaviour log-probability of every sampled token (Eq. 2's "
                         "denominator); reported as with_logprobs")
    ap.add_argument("--also-grpo", action="store_true",
                    help="additionally time one step with k = G (all P*G rollouts concurrent, no filter) and report it as grpo_mode")
    ap.add_argument("--probe", default=None, metavar="rows=R,suffix=S,steps=N,prompt=L",
                    help="time N decode steps of R rollouts (16 groups) that already hold S suffix tokens, then exit")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    from paper_2605_26606_b200 import binding as B
    from paper_2605_26606_b200 import build as _build
    from paper_2605_26606_b200.engine import RolloutEngine

    if args.probe is not None:
        run_probe(args)
        return

    rank, local_rank, world = dist_util.init("nccl")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    _build.build()
    base = wl.WORKLOADS[args.config]
    w = dataclasses.replace(base, data_seed=dist_util.rank_data_seed(base.data_seed, rank))
    P, G, k = w.n_prompts, w.group_size, w.n_pilot
    weights = wl.gen_weights(w.model, seed=0)
    batch = wl.gen_batch(w)

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:       # before the first GPU call
        n, dt, threads, desc = oracle_sample(w, weights, batch)
        cpu_baseline = {"value": n / dt, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    total_prompt = int(batch.prompt_offsets[-1])
    eng = RolloutEngine(w.model, weights, max_rows=max(P * k, P * (G - k), 1), max_prefill_tokens=total_prompt, device=dev)
    host_inputs = {"prompt_tokens": torch.from_numpy(batch.prompt_tokens).pin_memory(),
                   "prompt_offsets": torch.from_numpy(batch.prompt_offsets).pin_memory()}
    h2d_bytes = sum(t.numel() * t.element_size() for t in host_inputs.values())
    host_out = {"tokens": torch.empty(P * G * w.max_new, dtype=torch.int32).pin_memory(),
                "rewards": torch.empty(P * G, dtype=torch.float32).pin_memory(),
                "adv": torch.empty(P * G, dtype=torch.float32).pin_memory(),
                "status": torch.empty(P, dtype=torch.int32).pin_memory()}
    d2h_bytes = sum(t.numel() * t.element_size() for t in host_out.values())

    def one_step(timed: bool):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        ev[0].record()
        eng.load_batch(w, batch, host_inputs)          # host -> device copies of this step's inputs
        ev[1].record()
        status, n_tok = eng.run_device()
        ev[2].record()
        host_out["tokens"].copy_(eng.tokens, non_blocking=True)
        host_out["rewards"].copy_(eng.rewards, non_blocking=True)
        host_out["adv"].copy_(eng.adv, non_blocking=True)
        host_out["status"].copy_(eng.status, non_blocking=True)
        ev[3].record()
        torch.cuda.synchronize()
        eng.check_error_flag()
        return n_tok, ev[1].elapsed_time(ev[2]), ev[0].elapsed_time(ev[3]), status

    for _ in range(args.warmup):
        one_step(False)
    eng.profile_every = 32
    eng.profile_samples = []
    sampler = ClockSampler(local_rank)
    sampler.start()
    dist_util.barrier()
    torch.cuda.synchronize()
    launches0 = B.pc_launch_count()
    dev_ms, e2e_ms, tokens, status = 0.0, 0.0, 0, None
    for _ in range(args.steps):
        n_tok, d, e, status = one_step(True)
        dev_ms += d; e2e_ms += e; tokens += n_tok
    torch.cuda.synchronize()
    dist_util.barrier()
    launches = B.pc_launch_count() - launches0
    clocks = sampler.stop()

    # roofline of the dominant kernel (suffix attention): algorithmic bytes of the sampled launches / their duration
    m = w.model
    per_pos = 2 * m.n_kv_heads * m.head_dim * m.elem_bytes                 # K and V of one position, one layer
    per_row = 2 * m.n_q_heads * m.head_dim * m.elem_bytes                  # q read + output written
    s_bytes = sum(nr * (npos * per_pos + per_row) for (_, _, nr, npos) in eng.profile_samples)
    s_ms = sum(e0.elapsed_time(e1) for (e0, e1, _, _) in eng.profile_samples)
    peak, peak_kind = load_peaks()
    achieved = s_bytes / (s_ms * 1e-3) / 1e9 if s_ms > 0 else 0.0
    n_samp = max(len(eng.profile_samples), 1)
    roofline = {"bound": "hbm", "kernel": "attn_suffix_kernel", "achieved": achieved, "peak": peak, "peak_kind": peak_kind,
                "unit": "GB/s", "frac": achieved / peak,
                "traffic": SUFFIX_TRAFFIC_PER_ALGORITHMIC_BYTE * s_bytes / n_samp, "traffic_note": "ncu capture of a smaller case scaled by algorithmic bytes", "launches_sampled": len(eng.profile_samples),
                "avg_launch_ms": s_ms / n_samp, "avg_algorithmic_bytes": s_bytes / n_samp}

    # whole-step HBM roofline named by the metric: (weight bytes + KV bytes) each decode step must move / peak
    caps = batch.caps.astype(np.int64)
    gen = np.zeros((P, G), dtype=bool); gen[:, :k] = True; gen[status == B.PC_STATUS_COMMIT, :] = True
    kv_tok = m.kv_bytes_per_token
    steps_pilot = int(caps[:, :k].max() - 1)
    commit_rows = gen.copy(); commit_rows[:, :k] = False
    steps_commit = int(caps[commit_rows].max() - 1) if commit_rows.any() else 0
    suffix_reads = float(np.sum((caps[gen] - 1) * caps[gen] / 2.0)) * kv_tok           # sum over steps of (s + 1) per rollout
    prompt_reads = 0.0
    for stage_rows, n_st in ((np.pad(gen[:, :k], ((0, 0), (0, G - k))), steps_pilot), (commit_rows, steps_commit)):
        for p in range(P):
            c = caps[p][stage_rows[p]]
            if c.size:
                prompt_reads += float(c.max() - 1) * float(batch.prompt_lens[p]) * kv_tok   # once per group per step
    weight_reads = float(steps_pilot + steps_commit) * m.weight_bytes_per_decode_step()
    kv_writes = float(np.sum(caps[gen] - 1)) * kv_tok
    step_bytes = suffix_reads + prompt_reads + weight_reads + kv_writes

    t_ms, n_tokens = dist_util.aggregate(dev_ms, tokens, device=dev)
    t_e2e, _ = dist_util.aggregate(e2e_ms, tokens, device=dev)
    if rank != 0:
        return
    value = n_tokens / (t_ms * 1e-3)
    n_roll = int(gen.sum())
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": t_ms / max(args.steps, 1), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": ("f16" if eng.half_gemm else "bf16") if m.dtype == wl.DTYPE_BF16 else "f32", "data": "synthetic",
        "config": {"workload": w.name, "model": m.name, "prompts": P, "group_size": G, "n_pilot": k, "max_new": w.max_new,
                   "mode": "pilot-commit",
                   "arithmetic": "16-bit storage (bf16 model); GEMM operands IEEE half, K / q / embedding bfloat16, float32 accumulation"
                                 if m.dtype == wl.DTYPE_BF16 and eng.half_gemm else "model storage type, float32 accumulation", "committed_prompts": int((status == B.PC_STATUS_COMMIT).sum()),
                   "rollouts_generated": n_roll, "rollouts_per_s": n_roll * world / (t_ms * 1e-3 / max(args.steps, 1)),
                   "l2": "inputs larger than L2 (3.1 GB of weights and tens of GB of KV per step); no flush",
                   "parallelism": f"replicas x{world}, one sampling batch per GPU"},
        "clocks": clocks,
        "e2e": {"value": n_tokens / (t_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d_bytes, "d2h_bytes_per_step": d2h_bytes},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "hbm_step": {"bytes_per_step": step_bytes, "achieved_gbs": step_bytes * args.steps / (dev_ms * 1e-3) / 1e9,
                     "frac_of_measured": step_bytes * args.steps / (dev_ms * 1e-3) / 1e9 / peak,
                     "frac_of_8tbs": step_bytes * args.steps / (dev_ms * 1e-3) / 1e9 / 8000.0,
                     "parts": {"suffix_kv_read": suffix_reads, "prompt_kv_read": prompt_reads, "weights": weight_reads,
                               "kv_write": kv_writes}},
    }
    if cpu_baseline is not None:
        line["cpu_baseline"] = cpu_baseline
    if args.also_logprobs and world == 1:
        eng.profile_every = 0
        eng.collect_logprobs = True
        one_step(False)                                       # buffers and graphs of this mode
        n_tok, d_ms, _, _ = one_step(True)
        eng.collect_logprobs = False
        line["with_logprobs"] = {"tokens": n_tok, "ms_per_step": d_ms, "tokens_per_s": n_tok / (d_ms * 1e-3),
                                 "step_time_ratio": d_ms / (t_ms / max(args.steps, 1))}
    if args.also_bound and world == 1:
        # steady state of Section 3.4: batch A's pilot pass has just run on this engine (the timed step leaves A's prompt KV,
        # last-position logits and statuses in place); one pass then generates A's commit rollouts and B's pilot rollouts
        eng.profile_every = 0
        wb = dataclasses.replace(w, data_seed=w.data_seed + 1000)
        batch_b = wl.gen_batch(wb)
        commit_a = np.flatnonzero(status == B.PC_STATUS_COMMIT)
        times = []
        for rep in range(2):                                   # first repetition: graphs and allocator
            eng.load_batch(w, batch)
            eng.run_device()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            out_b = eng.bound_pass(w, batch, commit_a, batch_b)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        n_tok_b = int(sum(len(t) for t in out_b["a"].values()) + sum(len(t) for t in out_b["b"].values()))
        rows_b = len(commit_a) * (G - k) + P * k
        line["bound_pass"] = {"rows": rows_b, "commit_prompts_of_previous_batch": int(len(commit_a)), "pilot_prompts": P, "tokens": n_tok_b,
                              "ms_per_pass": times[-1], "tokens_per_s": n_tok_b / (times[-1] * 1e-3),
                              "note": "prefill of the new batch, decode of both row sets and the read-back of the tokens included"}
    if args.also_grpo and world == 1:
        # every rollout of every group at once (what plain GRPO generates for the same prompts): same kernels, k = G
        wg = dataclasses.replace(w, n_pilot=G)
        del eng
        torch.cuda.empty_cache()
        eng2 = RolloutEngine(wg.model, weights, max_rows=P * G, max_prefill_tokens=total_prompt, device=dev)
        eng2.load_batch(wg, batch)
        eng2.run_device()                       # warm-up (graph capture, allocator)
        torch.cuda.synchronize()
        eng2.load_batch(wg, batch)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        _, n_tok = eng2.run_device()
        e1.record()
        torch.cuda.synchronize()
        eng2.check_error_flag()
        ms = e0.elapsed_time(e1)
        cg = batch.caps.astype(np.float64)
        b = (float(np.sum((cg - 1) * cg / 2.0)) + float(np.sum(cg - 1))) * kv_tok \
            + float(sum((batch.caps[p].max() - 1) * batch.prompt_lens[p] for p in range(P))) * kv_tok \
            + float(batch.caps.max() - 1) * m.weight_bytes_per_decode_step()
        line["grpo_mode"] = {"rows": P * G, "tokens": n_tok, "ms_per_step": ms, "tokens_per_s": n_tok / (ms * 1e-3),
                             "hbm_bytes_per_step": b, "hbm_frac_of_measured": b / (ms * 1e-3) / 1e9 / peak}
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
