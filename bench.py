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

# DRAM traffic of the suffix attention kernel per algorithmic byte, from the ncu captures summarised in
# profiles/attn_suffix_kernel_ncu.md (current build: 143.5 MB moved for 136.0 MB algorithmic at 256 rollouts x 513 slots, 1,157 MB
# for 1,088 MB at 2048 x 513).  The kernel streams every (rollout, KV head) suffix once, so traffic grows in proportion to the
# algorithmic bytes of a launch.
SUFFIX_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.06
METRIC = "generated tokens/s"
UNIT = "tokens/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def load_tensor_peaks():
    """(burst, sustained) dense bf16 TFLOP/s: measured on this machine when the driver's file is there, else the earlier pool figures."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p.get("bf16_tflops", 1590.0)), float(p.get("bf16_tflops_sustained", 1400.0))
    return 1590.0, 1400.0


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
    B.pc_set_decode_mode(eng.ctx, int(kv.get("mode", 0)))
    B.pc_set_attention_overlap(eng.ctx, int(kv.get("overlap", 0)))
    B.pc_set_fused_sampler(eng.ctx, int(kv.get("fused", 0)))
    B.pc_set_fused_epilogues(eng.ctx, int(kv.get("epi", 1)))
    B.pc_set_dependent_launch(eng.ctx, int(kv.get("dep", 1)))
    if "plan" in kv:            # forced GEMM plans, e.g. plan=qkv:128x1+o:64x1
        B.pc_set_gemm_plan(eng.ctx, kv["plan"].replace(":", "=").replace("+", ","))
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
    line = {"probe": {"rows": P * G, "suffix": suffix, "steps": steps, "prompt_len": plen}, "ms_per_decode_step": ms, "host_issue_ms_per_step": host_ms,
            "tokens_per_s": P * G / (ms * 1e-3), "launches_per_step": (B.pc_launch_count() - l0) / steps,
            "hbm_bytes_per_step": bytes_step, "hbm_frac": bytes_step / (ms * 1e-3) / 1e9 / peak, "peak_kind": kind}
    if kv.get("trace") == "1" and int(kv.get("mode", 0)) == 1:
        line["chain_trace_us"] = chain_trace(eng, B, torch, pp, rr, suffix + steps - 1)        # the last timed step once more
    print(json.dumps(line), flush=True)


def chain_trace(eng, B, torch, pp, rr, step):
    """SM-clock stamps of the persistent decode kernel (pc_set_decode_mode 1) for one more decode step, as microseconds from the
    start of the launch that holds the middle layers: per phase of one layer, when the row-wise warps (W), the GEMM producer
    (P), the MMA issuer (M) and the epilogue (E) began, passed their grid barrier and finished."""
    eng.use_graphs = False
    n = B.pc_chain_trace_words(eng.ctx)
    tr = torch.zeros(n, dtype=torch.int64, device="cuda")
    B.pc_set_chain_trace(eng.ctx, tr)
    eng.run_stage(pp, rr, step_range=(step, step + 1))
    torch.cuda.synchronize()
    eng.check_error_flag()
    B.pc_set_chain_trace(eng.ctx, None)
    t = tr.cpu().numpy().reshape(-1, 10, 4, 16)             # [launch segment][phase][traced CTA][stamp]
    names = ["W_BEGIN", "W_WAITED", "W_DONE", "P_BEGIN", "P_BARRIER", "P_DONE", "M_FIRST", "M_DONE", "E_FIRST", "E_DONE"]
    ghz = 1.965
    seg = t.shape[0] // 2
    out = {}
    for cta in (0, 3):
        t0 = t[seg, 0, cta, 10]
        d = {"kernel_us": round(float(t[seg, 0, cta, 11] - t0) / ghz / 1e3, 1)}
        for j in range(9):
            ev = t[seg, j, cta]
            if ev[:10].any():
                d[f"phase{j}"] = {names[e]: round(float(ev[e] - t0) / ghz / 1e3, 1) for e in range(10) if ev[e]}
        out[f"cta{cta}"] = d
    return out


def phase_table(eng, B, n_layers):
    """Per-operation device time from the sampled decode steps: every sample holds the CUDA events pc_profile_step
    recorded around the operations of one decoder layer and of the step's tail (LM head, sampler)."""
    names = B.PROFILE_MARKS
    ix = {n: i for i, n in enumerate(names)}
    layer_ops = [("norm_attn", "layer_begin", "norm_attn"), ("qkv_gemm", "norm_attn", "qkv"), ("qkv_post", "qkv", "post"),
                 ("attn_prefix", "post", "group"), ("attn_suffix", "group", "suffix"), ("attn_merge", "suffix", "merge"),
                 ("o_gemm", "merge", "o"), ("norm_mlp", "o", "norm_mlp"), ("gate_up_gemm", "norm_mlp", "gate_up"),
                 ("down_gemm", "gate_up", "down")]
    tail_ops = [("lm_head", "lm_begin", "lm_head"), ("sampler", "lm_head", "sample")]
    tot = {k: 0.0 for k, _, _ in layer_ops + tail_ops}
    per_sample = []
    for evs, nr, npos in eng.profile_samples:
        d = {}
        for k, a, b in layer_ops + tail_ops:
            d[k] = evs[ix[a]].elapsed_time(evs[ix[b]])
            tot[k] += d[k]
        per_sample.append((d, nr, npos))
    n = max(len(per_sample), 1)
    # one sampled step stands for its neighbours: a layer operation runs n_layers times per step, a tail operation once
    est = {k: tot[k] / n * (1 if k in ("lm_head", "sampler") else n_layers) for k in tot}
    return per_sample, {k: tot[k] / n for k in tot}, est


def composite_bound_seconds(m, rows_per_step_list, caps_by_stage, prompt_lens_by_stage, peak_gbs, peak_tflops):
    """Lower bound of a run's decode time when every phase of every step runs at its own roofline:
    GEMMs max(weight bytes / BW, flops / tensor peak), attention KV bytes / BW."""
    bw, tf = peak_gbs * 1e9, peak_tflops * 1e12
    w_bytes = m.weight_bytes_per_decode_step()
    params = w_bytes / m.elem_bytes
    t_gemm = t_attn = 0.0
    for rows_per_step, caps, plens in zip(rows_per_step_list, caps_by_stage, prompt_lens_by_stage):
        rows = rows_per_step.astype(np.float64)
        t_gemm += float(np.sum(np.maximum(w_bytes / bw, 2.0 * rows * params / tf)))
        caps = caps.astype(np.float64)
        suffix_tok = float(np.sum((caps - 1) * caps / 2.0))
        prompt_tok = float(np.sum(plens))                       # prompt KV read once per group per step: sum over (group, step)
        t_attn += (suffix_tok + prompt_tok) * m.kv_bytes_per_token / bw
    return t_gemm, t_attn


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="config2", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the additional single-step measurements reported beside the main one: grpo_mode (all P*G rollouts "
                         "concurrent), loop_bound (Algorithm 1 as a running loop with bound passes, Section 3.4), bf16_operands")
    ap.add_argument("--also-logprobs", action="store_true",
                    help="additionally time one step that also keeps the behaviour log-probability of every sampled token (Eq. 2's "
                         "denominator); reported as with_logprobs")
    ap.add_argument("--probe", default=None, metavar="rows=R,suffix=S,steps=N,prompt=L,mode=M,plan=qkv:128x1+o:64x1",
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
    m = w.model

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

    def one_step(engine):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        ev[0].record()
        engine.load_batch(engine_wl[engine], batch, host_inputs)          # host -> device copies of this step's inputs
        ev[1].record()
        status, n_tok = engine.run_device()
        ev[2].record()
        host_out["tokens"].copy_(engine.tokens, non_blocking=True)
        host_out["rewards"].copy_(engine.rewards, non_blocking=True)
        host_out["adv"].copy_(engine.adv, non_blocking=True)
        host_out["status"].copy_(engine.status, non_blocking=True)
        ev[3].record()
        torch.cuda.synchronize()
        engine.check_error_flag()
        return n_tok, ev[1].elapsed_time(ev[2]), ev[0].elapsed_time(ev[3]), status

    engine_wl = {eng: w}
    eng.profile_every = 32                           # warm-up and timed steps take the same path
    for _ in range(args.warmup):
        one_step(eng)
    eng.profile_samples = []
    eng.stage_rows_per_step = []
    sampler = ClockSampler(local_rank)
    sampler.start()
    dist_util.barrier()
    torch.cuda.synchronize()
    launches0, captures0 = B.pc_launch_count(), B.pc_capture_count(eng.ctx)
    dev_ms, e2e_ms, tokens, status, prefill_ms = 0.0, 0.0, 0, None, 0.0
    for _ in range(args.steps):
        n_tok, d, e, status = one_step(eng)
        dev_ms += d; e2e_ms += e; tokens += n_tok
        prefill_ms += eng.prefill_events[0].elapsed_time(eng.prefill_events[1])
    torch.cuda.synchronize()
    dist_util.barrier()
    launches = B.pc_launch_count() - launches0
    captures = B.pc_capture_count(eng.ctx) - captures0
    clocks = sampler.stop()
    peak, peak_kind = load_peaks()
    tf_burst, tf_sustained = load_tensor_peaks()

    # ---- what the decode steps of this Pilot-Commit step must move (the HBM roofline the metric names)
    caps = batch.caps.astype(np.int64)
    gen = np.zeros((P, G), dtype=bool); gen[:, :k] = True; gen[status == B.PC_STATUS_COMMIT, :] = True
    kv_tok = m.kv_bytes_per_token
    steps_pilot = int(caps[:, :k].max() - 1)
    commit_rows = gen.copy(); commit_rows[:, :k] = False
    steps_commit = int(caps[commit_rows].max() - 1) if commit_rows.any() else 0
    suffix_reads = float(np.sum((caps[gen] - 1) * caps[gen] / 2.0)) * kv_tok           # sum over steps of (s + 1) per rollout
    prompt_reads = 0.0
    prompt_tok_by_stage = []
    for stage_rows, n_st in ((np.pad(gen[:, :k], ((0, 0), (0, G - k))), steps_pilot), (commit_rows, steps_commit)):
        tok = 0.0
        for p in range(P):
            c = caps[p][stage_rows[p]]
            if c.size:
                tok += float(c.max() - 1) * float(batch.prompt_lens[p])             # once per group per step
        prompt_tok_by_stage.append(np.array([tok]))
        prompt_reads += tok * kv_tok
    weight_reads = float(steps_pilot + steps_commit) * m.weight_bytes_per_decode_step()
    kv_writes = float(np.sum(caps[gen] - 1)) * kv_tok
    step_bytes = suffix_reads + prompt_reads + weight_reads + kv_writes
    decode_ms = dev_ms - prefill_ms
    achieved_step = step_bytes * args.steps / (decode_ms * 1e-3) / 1e9

    # ---- per-operation time from the sampled steps; roofline figures of the two heaviest kernel families
    per_sample, per_op_ms, est_ms = phase_table(eng, B, m.n_layers)
    per_pos = 2 * m.n_kv_heads * m.head_dim * m.elem_bytes                 # K and V of one position, one layer
    per_row = 2 * m.n_q_heads * m.head_dim * m.elem_bytes                  # q read + output written
    s_bytes = sum(nr * (npos * per_pos + per_row) for (_, nr, npos) in per_sample)
    s_ms = sum(d["attn_suffix"] for (d, _, _) in per_sample)
    n_samp = max(len(per_sample), 1)
    layer_w_bytes = m.layer_params() * m.elem_bytes
    g_ms = sum(d["qkv_gemm"] + d["o_gemm"] + d["gate_up_gemm"] + d["down_gemm"] for (d, _, _) in per_sample)
    g_flops = sum(2.0 * nr * m.layer_params() for (_, nr, _) in per_sample)
    g_bound_s = sum(max(layer_w_bytes / (peak * 1e9), 2.0 * nr * m.layer_params() / (tf_burst * 1e12)) for (_, nr, _) in per_sample)
    kernels = {
        "attn_suffix_kernel": {"bound": "hbm", "achieved": s_bytes / (s_ms * 1e-3) / 1e9 if s_ms > 0 else 0.0, "peak": peak, "unit": "GB/s",
                               "frac": (s_bytes / (s_ms * 1e-3) / 1e9 / peak) if s_ms > 0 else 0.0,
                               "traffic": SUFFIX_TRAFFIC_PER_ALGORITHMIC_BYTE * s_bytes / n_samp,
                               "traffic_note": "ncu capture of a smaller case scaled by algorithmic bytes (profiles/attn_suffix_kernel_ncu.md)",
                               "avg_launch_ms": s_ms / n_samp, "avg_algorithmic_bytes": s_bytes / n_samp},
        "gemm_tc_kernel (QKV, O, gate/up, down of one layer)": {
            "bound": "hbm below about %d rows, tensor above" % int(tf_burst * 1e12 / (peak * 1e9) / 2 * m.elem_bytes),
            "avg_ms_per_layer": g_ms / n_samp, "weight_gbs": layer_w_bytes * n_samp / (g_ms * 1e-3) / 1e9 if g_ms > 0 else 0.0,
            "weight_frac_of_hbm_peak": (layer_w_bytes * n_samp / (g_ms * 1e-3) / 1e9 / peak) if g_ms > 0 else 0.0,
            "tflops": g_flops / (g_ms * 1e-3) / 1e12 if g_ms > 0 else 0.0,
            "tensor_frac_of_bf16_burst": (g_flops / (g_ms * 1e-3) / 1e12 / tf_burst) if g_ms > 0 else 0.0,
            "frac_of_own_bound": g_bound_s / (g_ms * 1e-3) if g_ms > 0 else 0.0, "traffic": None},
    }
    stage_rows = eng.stage_rows_per_step[-2:] if len(eng.stage_rows_per_step) >= 2 else eng.stage_rows_per_step
    stage_caps = [caps[:, :k].reshape(-1), caps[commit_rows]][:len(stage_rows)]
    t_gemm_b, t_attn_b = composite_bound_seconds(m, stage_rows, stage_caps, prompt_tok_by_stage, peak, tf_burst)
    all_rows = np.concatenate(stage_rows) if stage_rows else np.zeros(0)
    hist_edges = [0, 16, 32, 64, 128, 192, 256, 384, 512, 1024, 2048, 4096]
    live_hist = {f"{a + 1}-{b}": int(np.sum((all_rows > a) & (all_rows <= b))) for a, b in zip(hist_edges[:-1], hist_edges[1:])}

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
                   "arithmetic": "16-bit storage (bf16 model); GEMM operands, q, K and V IEEE half, embedding bfloat16, float32 accumulation and residual stream"
                                 if m.dtype == wl.DTYPE_BF16 and eng.half_gemm else "model storage type, float32 accumulation", "committed_prompts": int((status == B.PC_STATUS_COMMIT).sum()),
                   "rollouts_generated": n_roll, "rollouts_per_s": n_roll * world / (t_ms * 1e-3 / max(args.steps, 1)),
                   "l2": "inputs larger than L2 (3.1 GB of weights and tens of GB of KV per step); no flush",
                   "parallelism": f"replicas x{world}, one sampling batch per GPU"},
        "clocks": clocks,
        "e2e": {"value": n_tokens / (t_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d_bytes, "d2h_bytes_per_step": d2h_bytes},
        "gpu_launches": int(launches),
        "graph_captures_in_timed_region": int(captures),
        # the quantity the metric names: bytes every decode step of the job must move (weights + KV) over the decode time
        "roofline": {"bound": "hbm", "kernel": "decode steps of the Pilot-Commit step, all kernels (prefill excluded)",
                     "achieved": achieved_step, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved_step / peak,
                     "frac_of_8tbs": achieved_step / 8000.0, "traffic": None,
                     "traffic_note": "not captured for the 4,100-step job; ncu captures of single decode steps moved 1.22 x (256 rows x 512) "
                                     "and 1.26 x (2048 rows x 512) their algorithmic bytes (profiles/decode_step_launch_list_config2.md)",
                     "bytes_per_step": step_bytes, "decode_ms_per_step": decode_ms / max(args.steps, 1),
                     "parts": {"suffix_kv_read": suffix_reads, "prompt_kv_read": prompt_reads, "weights": weight_reads, "kv_write": kv_writes},
                     "target": 0.60},
        "composite_bound": {"note": "sum over decode steps of max(weight bytes / HBM peak, flops / bf16 burst peak) for the GEMMs plus KV bytes / HBM peak",
                            "gemm_bound_s": t_gemm_b, "attention_bound_s": t_attn_b,
                            "frac": (t_gemm_b + t_attn_b) / (decode_ms * 1e-3 / max(args.steps, 1)) if decode_ms > 0 else 0.0},
        "kernels": kernels,
        "phase_ms": {"prefill_per_step": prefill_ms / max(args.steps, 1),
                     "sampled_decode_steps": len(per_sample), "per_launch_avg": per_op_ms,
                     "estimated_per_decode_step": est_ms,
                     "note": "CUDA events around the operations of layer %d and the LM head / sampler in every 32nd decode step; "
                             "a layer operation is counted n_layers times; the sampled steps run in plain stream order (an event between "
                             "two kernels rules out the dependent launches the other steps use)" % eng.profile_layer},
        "live_rows_histogram": live_hist,
        "hbm_step": {"bytes_per_step": step_bytes, "achieved_gbs": step_bytes * args.steps / (dev_ms * 1e-3) / 1e9,
                     "frac_of_measured": step_bytes * args.steps / (dev_ms * 1e-3) / 1e9 / peak,
                     "frac_of_8tbs": step_bytes * args.steps / (dev_ms * 1e-3) / 1e9 / 8000.0,
                     "note": "as above with the prefill inside the time"},
    }
    if cpu_baseline is not None:
        line["cpu_baseline"] = cpu_baseline
    kv_tok_f = float(kv_tok)
    if args.also_logprobs and world == 1:
        eng.profile_every = 0
        eng.collect_logprobs = True
        one_step(eng)                                         # buffers and graphs of this mode
        n_tok, d_ms, _, _ = one_step(eng)
        eng.collect_logprobs = False
        line["with_logprobs"] = {"tokens": n_tok, "ms_per_step": d_ms, "tokens_per_s": n_tok / (d_ms * 1e-3),
                                 "step_time_ratio": d_ms / (t_ms / max(args.steps, 1))}
    if not args.no_extras and world == 1:
        eng._arenas.clear()
        eng.prompt_kv = eng.suffix_kv = None
        del eng
        torch.cuda.empty_cache()
        # (1) every rollout of every group at once (what plain GRPO generates for the same prompts): same kernels, k = G
        wg = dataclasses.replace(w, n_pilot=G)
        eng2 = RolloutEngine(wg.model, weights, max_rows=P * G, max_prefill_tokens=total_prompt, device=dev)
        engine_wl[eng2] = wg
        one_step(eng2)                           # warm-up (graph capture, allocator)
        n_tok, ms, _, _ = one_step(eng2)
        cg = batch.caps.astype(np.float64)
        b = (float(np.sum((cg - 1) * cg / 2.0)) + float(np.sum(cg - 1))) * kv_tok_f \
            + float(sum((batch.caps[p].max() - 1) * batch.prompt_lens[p] for p in range(P))) * kv_tok_f \
            + float(batch.caps.max() - 1) * m.weight_bytes_per_decode_step()
        tg, ta = composite_bound_seconds(m, eng2.stage_rows_per_step[-1:], [batch.caps.reshape(-1)],
                                         [np.array([float(sum((batch.caps[p].max() - 1) * batch.prompt_lens[p] for p in range(P)))])],
                                         peak, tf_burst)
        line["grpo_mode"] = {"rows": P * G, "tokens": n_tok, "ms_per_step": ms, "tokens_per_s": n_tok / (ms * 1e-3),
                             "hbm_bytes_per_step": b, "hbm_frac_of_measured": b / (ms * 1e-3) / 1e9 / peak,
                             "composite_bound_frac": (tg + ta) / (ms * 1e-3)}
        eng2._arenas.clear()
        eng2.prompt_kv = eng2.suffix_kv = None
        del eng2
        torch.cuda.empty_cache()
        # (2) Algorithm 1 as a running loop with bound passes (Section 3.4): three sampling batches, each pass holding the pilot
        #     rollouts of a new batch and the commit rollouts of the previous batch's survivors on their resident prompt KV
        from paper_2605_26606_b200.loop import RolloutLoop
        n_b = 3
        wd = dataclasses.replace(w, n_prompts=n_b * P)
        data = wl.gen_batch(wd)
        eng3 = RolloutEngine(w.model, weights, max_rows=P * k + P * (G - k), max_prefill_tokens=int(data.prompt_lens.max()) * P, device=dev)
        loop = RolloutLoop(eng3, w, data, b_g=P, b_t=P, max_delay=1, bind=True, max_resident_prompts=3 * P)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        recs = loop.run(list(range(n_b * P)), 1)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        n_tok = int(sum(len(t) for r in recs for t in r.tokens.values()))
        line["loop_bound"] = {"training_steps": len(recs), "passes": int(sum(r.passes for r in recs)), "sampling_batch": P, "b_t": P,
                              "committed_per_step": [len(r.plan.committed) for r in recs],
                              "rollouts_sampled_per_step": [r.plan.rollouts_sampled for r in recs],
                              "second_round_share": float(np.mean([r.plan.rounds > 1 for r in recs])),
                              "tokens": n_tok, "ms_total": ms, "tokens_per_s": n_tok / (ms * 1e-3),
                              "note": "prefills, decode passes, statistics, allocation, advantages and the read-back of every rollout included; "
                                      "the first pass has no commit rows and the last no pilot rows"}
        eng3._arenas.clear()
        eng3.prompt_kv = eng3.suffix_kv = None
        del eng3, loop
        torch.cuda.empty_cache()
        # (3) the main step with bfloat16 GEMM operands (value + rounding remainder for QKV / O / LM head) instead of IEEE half
        if m.dtype == wl.DTYPE_BF16:
            eng4 = RolloutEngine(w.model, weights, max_rows=max(P * k, P * (G - k), 1), max_prefill_tokens=total_prompt, device=dev,
                                 half_gemm=False)
            engine_wl[eng4] = w
            one_step(eng4)
            n_tok, ms, _, st4 = one_step(eng4)
            line["bf16_operands"] = {"tokens": n_tok, "ms_per_step": ms, "tokens_per_s": n_tok / (ms * 1e-3),
                                     "committed_prompts": int((st4 == B.PC_STATUS_COMMIT).sum())}
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
