"""ctypes binding of libpc.so: one Python function per C entry point of include/pc.h, same names.

Argument marshalling only -- every computation happens in the CUDA library.  Device
arguments are torch CUDA tensors (or None where the C side accepts NULL); the current
torch stream is passed as the CUDA stream.  The library is required: importing works
anywhere, but the first call raises if libpc.so has not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpc.so")

PC_OK = 0
PC_ERR_INVALID_ARG, PC_ERR_SHAPE, PC_ERR_ALIGNMENT, PC_ERR_CAPACITY = 1, 2, 3, 4
PC_ERR_UNSUPPORTED, PC_ERR_CUDA, PC_ERR_NO_WORKSPACE = 5, 6, 7
PC_DTYPE_F32, PC_DTYPE_BF16 = 0, 1
PC_STATUS_COMMIT, PC_STATUS_BUFFERED, PC_STATUS_DEFER_HARD, PC_STATUS_SKIP_EASY, PC_STATUS_LOW_VARIANCE = 0, 1, 2, 3, 4

EXPORTS = ["pc_status_string", "pc_last_cuda_error", "pc_launch_count", "pc_profile_step", "pc_set_gemm_plan", "pc_set_decode_mode", "pc_set_attention_overlap", "pc_set_fused_sampler", "pc_set_fused_epilogues", "pc_set_dependent_launch", "pc_set_chain_trace", "pc_chain_trace_words", "pc_capture_count", "pc_set_index_bounds", "pc_selftest_wait_timeout", "pc_create", "pc_destroy", "pc_workspace_bytes",
           "pc_set_workspace", "pc_prefill_shared", "pc_decode_step", "pc_decode_run", "pc_sample", "pc_sample_static", "pc_token_logprob", "pc_set_logprob_buffer", "pc_set_prompt_keys", "pc_reward_last_token",
           "pc_group_stats", "pc_allocate", "pc_allocate_variance", "pc_grpo_advantage"]


class ModelDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ff", "vocab")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_int32) for n in ("dtype", "tied_embed", "qk_norm", "qkv_bias", "half_gemm")]


class WeightsDesc(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "wqkv", "bqkv", "q_norm", "k_norm", "wo", "mlp_norm",
                                                      "w_gate_up", "w_down")]


class StepDesc(C.Structure):
    _fields_ = [("n_rows", C.c_int32), ("n_groups", C.c_int32), ("max_group_rows", C.c_int32), ("reserved", C.c_int32),
                ("row_offset", C.c_int64), ("group_offset", C.c_int64)]


class SampleParams(C.Structure):
    _fields_ = [("temperature", C.c_float), ("seed", C.c_uint64)]


class AllocParams(C.Structure):
    _fields_ = [("p_lower", C.c_double), ("p_upper", C.c_double), ("p_solve", C.c_double),
                ("n_commit", C.c_int32), ("b_t", C.c_int32)]


class PcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        lib = _lib()
        msg = lib.pc_status_string(status).decode()
        if status == PC_ERR_CUDA:
            msg += ": " + lib.pc_last_cuda_error().decode()
        super().__init__(f"{where} failed with status {status} ({msg})")


_LIB = None


def _lib():
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_26606_b200.build` "
                               "(there is no fallback path)")
        lib = C.CDLL(LIB_PATH)
        lib.pc_status_string.restype = C.c_char_p
        lib.pc_status_string.argtypes = [C.c_int]
        lib.pc_last_cuda_error.restype = C.c_char_p
        lib.pc_launch_count.restype = C.c_uint64
        lib.pc_launch_count.argtypes = []
        lib.pc_profile_step.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_void_p), C.c_int]
        lib.pc_set_gemm_plan.argtypes = [C.c_void_p, C.c_char_p]
        lib.pc_set_decode_mode.argtypes = [C.c_void_p, C.c_int]
        lib.pc_set_attention_overlap.argtypes = [C.c_void_p, C.c_int]
        lib.pc_set_fused_sampler.argtypes = [C.c_void_p, C.c_int]
        lib.pc_set_fused_epilogues.argtypes = [C.c_void_p, C.c_int]
        lib.pc_set_dependent_launch.argtypes = [C.c_void_p, C.c_int]
        lib.pc_capture_count.argtypes = [C.c_void_p]
        lib.pc_capture_count.restype = C.c_uint64
        lib.pc_set_index_bounds.argtypes = [C.c_void_p, C.c_int, C.c_int64]
        lib.pc_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
        lib.pc_set_chain_trace.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
        lib.pc_chain_trace_words.argtypes = [C.c_void_p]
        lib.pc_chain_trace_words.restype = C.c_size_t
        lib.pc_destroy.restype = None
        lib.pc_destroy.argtypes = [C.c_void_p]
        p, i, i64, f, u64 = C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_uint64
        lib.pc_create.argtypes = [C.POINTER(ModelDesc), C.POINTER(WeightsDesc), C.POINTER(C.c_void_p)]
        lib.pc_workspace_bytes.argtypes = [p, i, i, C.POINTER(C.c_size_t)]
        lib.pc_set_workspace.argtypes = [p, p, C.c_size_t, i, i, p]
        lib.pc_prefill_shared.argtypes = [p, p, i, p, p, i, i, p, i64, p, p]
        lib.pc_decode_step.argtypes = [p, p, i, p, p, p, p, p, p, i, p, i, p, p, i64, p, p, i64, p, C.POINTER(SampleParams)]
        lib.pc_decode_run.argtypes = [p, p, i, p, p, p, p, p, p, p, p, p, p, p, i64, p, p, i64, C.POINTER(SampleParams)]
        lib.pc_sample.argtypes = [p, i, i, p, p, f, u64, p, p, p, p, p, p, p, C.c_size_t]
        lib.pc_sample_static.argtypes = [p, i, i, p, p, f, u64, p, p, p, p, p, p]
        lib.pc_token_logprob.argtypes = [p, i, i, p, p, f, p, p, p, p]
        lib.pc_set_logprob_buffer.argtypes = [p, p]
        lib.pc_set_prompt_keys.argtypes = [p, p]
        lib.pc_reward_last_token.argtypes = [p, i, p, p, p, p]
        lib.pc_group_stats.argtypes = [p, i, p, p, p, p, p, p, p]
        lib.pc_allocate.argtypes = [p, i, p, p, C.POINTER(AllocParams), p, p, p, p, p]
        lib.pc_grpo_advantage.argtypes = [p, i, p, p, p, p, p]
        lib.pc_allocate_variance.argtypes = [p, i, p, p, C.c_double, i, i, p, p, p, p]
        for name in EXPORTS[3:]:
            if name not in ("pc_destroy", "pc_chain_trace_words", "pc_capture_count"):
                getattr(lib, name).restype = C.c_int
        _LIB = lib
    return _LIB


def _check(status: int, where: str) -> None:
    if status != PC_OK:
        raise PcError(status, where)


def _ptr(t: Optional[torch.Tensor], dtype: Optional[torch.dtype] = None) -> Optional[int]:
    """Device address of a contiguous CUDA tensor (None -> NULL)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not t.is_cuda:
        raise TypeError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise TypeError("expected a contiguous tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"expected dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def pc_status_string(status: int) -> str:
    return _lib().pc_status_string(status).decode()


def pc_last_cuda_error() -> str:
    return _lib().pc_last_cuda_error().decode()


def pc_launch_count() -> int:
    return int(_lib().pc_launch_count())


def pc_set_gemm_plan(ctx: "Context", spec: Optional[str]) -> None:
    _check(_lib().pc_set_gemm_plan(ctx.handle, None if spec is None else spec.encode()), "pc_set_gemm_plan")


def pc_set_decode_mode(ctx: "Context", mode: int) -> None:
    _check(_lib().pc_set_decode_mode(ctx.handle, mode), "pc_set_decode_mode")


def pc_set_fused_epilogues(ctx: "Context", on: int) -> None:
    _check(_lib().pc_set_fused_epilogues(ctx.handle, on), "pc_set_fused_epilogues")


def pc_set_dependent_launch(ctx: "Context", mask: int) -> None:
    _check(_lib().pc_set_dependent_launch(ctx.handle, mask), "pc_set_dependent_launch")


def pc_set_fused_sampler(ctx: "Context", on: int) -> None:
    _check(_lib().pc_set_fused_sampler(ctx.handle, on), "pc_set_fused_sampler")


def pc_set_attention_overlap(ctx: "Context", on: int) -> None:
    _check(_lib().pc_set_attention_overlap(ctx.handle, on), "pc_set_attention_overlap")


def pc_capture_count(ctx: "Context") -> int:
    return int(_lib().pc_capture_count(ctx.handle))


def pc_set_index_bounds(ctx: "Context", n_prompts: int, n_tokens: int) -> None:
    _check(_lib().pc_set_index_bounds(ctx.handle, n_prompts, n_tokens), "pc_set_index_bounds")


def pc_selftest_wait_timeout(spin_limit: int, err_flag: torch.Tensor) -> None:
    _check(_lib().pc_selftest_wait_timeout(_stream(), spin_limit, _ptr(err_flag, torch.int32)), "pc_selftest_wait_timeout")


def pc_chain_trace_words(ctx: "Context") -> int:
    return int(_lib().pc_chain_trace_words(ctx.handle))


def pc_set_chain_trace(ctx: "Context", trace: Optional[torch.Tensor]) -> None:
    _check(_lib().pc_set_chain_trace(ctx.handle, _ptr(trace, torch.int64) if trace is not None else None,
                                     trace.numel() if trace is not None else 0), "pc_set_chain_trace")
    ctx._keep.append(trace)


PROFILE_MARKS = ["layer_begin", "norm_attn", "qkv", "post", "group", "suffix", "merge", "o", "norm_mlp", "gate_up", "down", "lm_begin",
                 "lm_head", "sample"]


def pc_profile_step(ctx: "Context", layer: int, events: Sequence[torch.cuda.Event]) -> None:
    """events: len(PROFILE_MARKS) events created with enable_timing=True and recorded once (so that they exist)."""
    arr = (C.c_void_p * len(events))(*[e.cuda_event for e in events])
    _check(_lib().pc_profile_step(ctx.handle, layer, arr, len(events)), "pc_profile_step")


class Context:
    """Owns a pc_ctx* and keeps the tensors it points at alive."""

    def __init__(self, handle: int, keep):
        self.handle = handle
        self._keep = keep

    def close(self) -> None:
        if self.handle:
            _lib().pc_destroy(self.handle)
            self.handle = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def pc_create(desc: ModelDesc, embed, lm_head, final_norm, attn_norm: Sequence, wqkv: Sequence, bqkv, q_norm, k_norm,
              wo: Sequence, mlp_norm: Sequence, w_gate_up: Sequence, w_down: Sequence) -> Context:
    n = desc.n_layers

    def table(ts):
        if ts is None:
            return None
        arr = (C.c_void_p * n)(*[_ptr(t) for t in ts])
        return arr

    tabs = {k: table(v) for k, v in dict(attn_norm=attn_norm, wqkv=wqkv, bqkv=bqkv, q_norm=q_norm, k_norm=k_norm, wo=wo,
                                           mlp_norm=mlp_norm, w_gate_up=w_gate_up, w_down=w_down).items()}
    w = WeightsDesc()
    w.embed, w.lm_head, w.final_norm = _ptr(embed), _ptr(lm_head), _ptr(final_norm, torch.float32)
    for k, v in tabs.items():
        setattr(w, k, C.cast(v, C.POINTER(C.c_void_p)) if v is not None else None)
    out = C.c_void_p()
    _check(_lib().pc_create(C.byref(desc), C.byref(w), C.byref(out)), "pc_create")
    keep = [embed, lm_head, final_norm, attn_norm, wqkv, bqkv, q_norm, k_norm, wo, mlp_norm, w_gate_up, w_down]
    return Context(out.value, keep)


def pc_workspace_bytes(ctx: Context, max_rows: int, max_prefill_tokens: int) -> int:
    out = C.c_size_t()
    _check(_lib().pc_workspace_bytes(ctx.handle, max_rows, max_prefill_tokens, C.byref(out)), "pc_workspace_bytes")
    return out.value


def pc_set_workspace(ctx: Context, ws: torch.Tensor, max_rows: int, max_prefill_tokens: int, err_flag: torch.Tensor) -> None:
    _check(_lib().pc_set_workspace(ctx.handle, _ptr(ws), ws.numel() * ws.element_size(), max_rows, max_prefill_tokens,
                                   _ptr(err_flag, torch.int32)), "pc_set_workspace")
    ctx._keep += [ws, err_flag]


def pc_prefill_shared(ctx: Context, n_prompts, prompt_tokens, prompt_offsets, total_tokens, max_prompt_len, prompt_kv,
                      prompt_slots, prompt_kv_start, last_logits) -> None:
    _check(_lib().pc_prefill_shared(ctx.handle, _stream(), n_prompts, _ptr(prompt_tokens, torch.int32),
                                    _ptr(prompt_offsets, torch.int32), total_tokens, max_prompt_len, _ptr(prompt_kv),
                                    prompt_slots, _ptr(prompt_kv_start, torch.int64), _ptr(last_logits, torch.float32)),
           "pc_prefill_shared")


def pc_decode_step(ctx: Context, n_rows, row_prompt, row_rollout, row_step, row_kv_start, tokens, row_tok_index, n_groups,
                   group_row_start, max_group_rows, prompt_len, prompt_kv, prompt_slots, prompt_kv_start, suffix_kv,
                   suffix_slots, logits_out=None, sample: Optional[SampleParams] = None) -> None:
    """Pointer arguments may be CUDA tensors or raw device addresses (int), so that a driver can
    step through slices of pre-uploaded schedules without creating tensor views."""
    _check(_lib().pc_decode_step(ctx.handle, _stream(), n_rows, _ptr(row_prompt), _ptr(row_rollout), _ptr(row_step),
                                 _ptr(row_kv_start), _ptr(tokens), _ptr(row_tok_index), n_groups, _ptr(group_row_start),
                                 max_group_rows, _ptr(prompt_len), _ptr(prompt_kv), prompt_slots, _ptr(prompt_kv_start),
                                 _ptr(suffix_kv), suffix_slots, _ptr(logits_out),
                                 C.byref(sample) if sample is not None else None), "pc_decode_step")


def pc_decode_run(ctx: Context, n_steps, steps_host, steps_dev, row_prompt, row_rollout, row_step, row_kv_start, tokens,
                  row_tok_index, group_row_start, prompt_len, prompt_kv, prompt_slots, prompt_kv_start, suffix_kv, suffix_slots,
                  sample: SampleParams) -> None:
    """steps_host: address (int) of n_steps StepDesc records in host memory; steps_dev: the same records on the device."""
    _check(_lib().pc_decode_run(ctx.handle, _stream(), n_steps, steps_host, _ptr(steps_dev), _ptr(row_prompt), _ptr(row_rollout),
                                _ptr(row_step), _ptr(row_kv_start), _ptr(tokens), _ptr(row_tok_index), _ptr(group_row_start),
                                _ptr(prompt_len), _ptr(prompt_kv), prompt_slots, _ptr(prompt_kv_start), _ptr(suffix_kv),
                                suffix_slots, C.byref(sample)), "pc_decode_run")


def pc_sample(n_rows, vocab, logits, logits_row, temperature, seed, row_prompt, row_rollout, row_step, out_tokens,
              out_index=None, out_top2_gap=None, scratch: Optional[torch.Tensor] = None) -> None:
    _check(_lib().pc_sample(_stream(), n_rows, vocab, _ptr(logits, torch.float32), _ptr(logits_row), temperature, seed,
                            _ptr(row_prompt), _ptr(row_rollout), _ptr(row_step), _ptr(out_tokens), _ptr(out_index),
                            _ptr(out_top2_gap), _ptr(scratch), scratch.numel() * scratch.element_size() if scratch is not None else 0),
           "pc_sample")


def pc_sample_static(n_rows, vocab, logits, logits_row, temperature, seed, row_prompt, row_rollout, row_step, out_tokens,
                     out_index=None, out_top2_gap=None) -> None:
    """pc_sample without caller scratch: the sampler's intermediate records live in an array inside libpc.so (at most
    4096 rows per call).  For callers that may not allocate device memory when they sample; calls that overlap on the
    GPU must be ordered by the caller because they share that array."""
    _check(_lib().pc_sample_static(_stream(), n_rows, vocab, _ptr(logits, torch.float32), _ptr(logits_row), temperature, seed,
                                   _ptr(row_prompt), _ptr(row_rollout), _ptr(row_step), _ptr(out_tokens), _ptr(out_index),
                                   _ptr(out_top2_gap)), "pc_sample_static")


def pc_token_logprob(n_rows, vocab, logits, logits_row, temperature, tokens, tok_index, out_logprob, out_index=None) -> None:
    _check(_lib().pc_token_logprob(_stream(), n_rows, vocab, _ptr(logits, torch.float32), _ptr(logits_row), temperature,
                                   _ptr(tokens, torch.int32), _ptr(tok_index), _ptr(out_logprob, torch.float32), _ptr(out_index)),
           "pc_token_logprob")


def pc_set_logprob_buffer(ctx: Context, logprobs: Optional[torch.Tensor]) -> None:
    _check(_lib().pc_set_logprob_buffer(ctx.handle, _ptr(logprobs)), "pc_set_logprob_buffer")
    ctx._keep.append(logprobs)


def pc_set_prompt_keys(ctx: Context, prompt_key: Optional[torch.Tensor]) -> None:
    _check(_lib().pc_set_prompt_keys(ctx.handle, _ptr(prompt_key)), "pc_set_prompt_keys")
    ctx._keep.append(prompt_key)


def pc_reward_last_token(n, tokens, last_index, threshold, reward) -> None:
    _check(_lib().pc_reward_last_token(_stream(), n, _ptr(tokens, torch.int32), _ptr(last_index, torch.int64),
                                       _ptr(threshold, torch.int32), _ptr(reward, torch.float32)), "pc_reward_last_token")


def pc_group_stats(n_groups, rewards, group_start, group_count, n, n_success, mean, var) -> None:
    _check(_lib().pc_group_stats(_stream(), n_groups, _ptr(rewards, torch.float32), _ptr(group_start, torch.int32),
                                 _ptr(group_count, torch.int32), _ptr(n, torch.int32), _ptr(n_success, torch.int32),
                                 _ptr(mean, torch.float32), _ptr(var, torch.float32)), "pc_group_stats")


def pc_allocate(n_prompts, pilot_success, pilot_n, params: AllocParams, status, extra_rollouts, evict, n_selected,
                total_rollouts) -> None:
    _check(_lib().pc_allocate(_stream(), n_prompts, _ptr(pilot_success, torch.int32), _ptr(pilot_n, torch.int32),
                              C.byref(params), _ptr(status, torch.int32), _ptr(extra_rollouts, torch.int32),
                              _ptr(evict, torch.int32), _ptr(n_selected, torch.int32), _ptr(total_rollouts, torch.int64)),
           "pc_allocate")


def pc_allocate_variance(n_prompts, pilot_var, pilot_n, var_min: float, n_commit: int, b_t: int, status, extra_rollouts, n_selected,
                         total_rollouts) -> None:
    _check(_lib().pc_allocate_variance(_stream(), n_prompts, _ptr(pilot_var, torch.float32), _ptr(pilot_n, torch.int32), var_min,
                                       n_commit, b_t, _ptr(status, torch.int32), _ptr(extra_rollouts, torch.int32),
                                       _ptr(n_selected, torch.int32), _ptr(total_rollouts, torch.int64)), "pc_allocate_variance")


def pc_grpo_advantage(n_groups, rewards, group_start, group_count, status, adv) -> None:
    _check(_lib().pc_grpo_advantage(_stream(), n_groups, _ptr(rewards, torch.float32), _ptr(group_start, torch.int32),
                                    _ptr(group_count, torch.int32), _ptr(status), _ptr(adv, torch.float32)),
           "pc_grpo_advantage")
