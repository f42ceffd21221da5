"""Seeded synthetic inputs: model shapes, weights, prompts, reward thresholds, length caps.

This module only *draws inputs*.  It holds none of the method's arithmetic (no
decoder math, no sampler, no statistics), so both the CUDA binding and the CPU
oracle may import it without sharing any computation.

The paper trains Qwen2.5-Math-1.5B and Qwen3-4B/8B/14B-Base on math prompts with
a binary verifier reward (Section 4.1, Section 4.2).  Neither the checkpoints,
the prompt sets nor the verifier are available offline, so every input here is a
stand-in with the same *shape*: decoder dimensions of those model families,
group sizes G in {8, 16, 64, 128} split into pilot/commit counts, ragged
response lengths, and a fraction of prompts whose groups collapse to all-wrong
or all-right (the paper reports 22-35 % of prompts being evicted as solved).

Random streams come from numpy's Philox bit generator keyed by
(seed, stream tag); each tensor has its own stream so that a layer can be
regenerated on its own.
"""
from __future__ import annotations

import dataclasses
import math
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, List, Optional

import numpy as np

DTYPE_F32 = 0
DTYPE_BF16 = 1


@dataclasses.dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    rms_eps: float = 1e-6
    rope_theta: float = 1e4
    dtype: int = DTYPE_BF16
    tied_embed: bool = False
    qk_norm: bool = False
    qkv_bias: bool = False

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == DTYPE_F32 else 2

    @property
    def kv_bytes_per_token(self) -> int:
        return self.n_layers * 2 * self.kv_dim * self.elem_bytes

    def layer_params(self) -> int:
        d, f = self.d_model, self.d_ff
        n = (self.q_dim + 2 * self.kv_dim) * d + d * self.q_dim + 3 * d * f
        return n

    def weight_bytes_per_decode_step(self) -> int:
        """Matrix bytes every decode step must stream: all layers + the LM head."""
        n = self.n_layers * self.layer_params() + self.vocab * self.d_model
        return n * self.elem_bytes


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    model: ModelShape
    n_prompts: int
    prompt_len_lo: int
    prompt_len_hi: int
    group_size: int          # G = n_pilot + n_commit
    n_pilot: int             # k
    max_new: int
    cap_lo: int
    cap_hi: int
    forced_frac: float       # share of prompts forced to tau in {0, 1}
    forced_explicit: Optional[tuple] = None   # ((prompt, tau), ...) overrides forced_frac
    temperature: float = 1.0
    sample_seed: int = 1234
    data_seed: int = 0
    p_lower: float = 0.125   # Section 4.2, "Pilot-Commit hyperparameters"
    p_upper: float = 0.75
    p_solve: float = 1.0

    @property
    def n_commit(self) -> int:
        return self.group_size - self.n_pilot


TINY = ModelShape("tiny-fp32", 2, 256, 4, 2, 64, 688, 2048, dtype=DTYPE_F32)
TINY_BF16 = dataclasses.replace(TINY, name="tiny-bf16", dtype=DTYPE_BF16, qkv_bias=True, d_ff=704)
SMALL_BF16 = ModelShape("small-bf16", 2, 512, 4, 2, 128, 1024, 4096, dtype=DTYPE_BF16,
                        tied_embed=True, qkv_bias=True)
SMALL_QKNORM_BF16 = ModelShape("small-qknorm-bf16", 2, 512, 4, 2, 128, 1024, 4096, dtype=DTYPE_BF16,
                               qk_norm=True, rope_theta=1e6)
QWEN25_1P5B = ModelShape("qwen2.5-1.5b-shape", 28, 1536, 12, 2, 128, 8960, 151936,
                         tied_embed=True, qkv_bias=True)
QWEN3_8B = ModelShape("qwen3-8b-shape", 36, 4096, 32, 8, 128, 12288, 151936,
                      rope_theta=1e6, qk_norm=True)
QWEN3_14B = ModelShape("qwen3-14b-shape", 40, 5120, 40, 8, 128, 17408, 151936,
                       rope_theta=1e6, qk_norm=True)

WORKLOADS: Dict[str, Workload] = {
    "config0": Workload("config0", TINY, 4, 32, 32, 8, 2, 16, 16, 16, 0.0,
                        forced_explicit=((0, 0.0), (3, 1.0)), data_seed=6),
    "config1": Workload("config1", QWEN25_1P5B, 32, 256, 256, 16, 4, 512, 128, 512, 0.0),
    "config2": Workload("config2", QWEN25_1P5B, 16, 256, 1024, 128, 16, 2048, 512, 2048, 0.3),
    "config3": Workload("config3", QWEN3_8B, 8, 512, 512, 64, 8, 1024, 256, 1024, 0.3),
    "config4": Workload("config4", QWEN3_14B, 4, 512, 512, 64, 8, 2048, 512, 2048, 0.3),
}

_TAG_PROMPT_LEN, _TAG_PROMPT_TOK, _TAG_TAU, _TAG_FORCED, _TAG_CAP = 101, 102, 103, 104, 105


def _rng(seed: int, tag: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(tag)]))


# ----------------------------------------------------------------------------------------
# bf16 helpers (storage format only)
# ----------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bfloat16 (ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


class Weights:
    """Mapping tensor name -> float32 array.

    Matrices of a bf16 model are stored as uint16 bit patterns (half the host
    memory) and expanded to float32 on access; every value handed out is exactly
    representable in the model's storage type.
    """

    def __init__(self, model: ModelShape):
        self.model = model
        self._f32: Dict[str, np.ndarray] = {}
        self._bits: Dict[str, np.ndarray] = {}

    def put(self, name: str, arr: np.ndarray, as_bits: bool) -> None:
        if as_bits:
            self._bits[name] = f32_to_bf16_bits(arr)
        else:
            self._f32[name] = np.ascontiguousarray(arr, dtype=np.float32)

    def __contains__(self, name: str) -> bool:
        return name in self._f32 or name in self._bits

    def __getitem__(self, name: str) -> np.ndarray:
        if name in self._f32:
            return self._f32[name]
        return bf16_bits_to_f32(self._bits[name])

    def bits(self, name: str) -> np.ndarray:
        """uint16 bf16 bit patterns of a matrix of a bf16 model."""
        return self._bits[name]

    def names(self) -> List[str]:
        return sorted(list(self._f32) + list(self._bits))


def tensor_specs(model: ModelShape):
    """(name, shape, kind) for every tensor; kind: 'matrix' ~ N(0, 0.02), 'gain' = 1, 'bias' ~ N(0, 0.02)."""
    d, f, hd = model.d_model, model.d_ff, model.head_dim
    specs = [("embed", (model.vocab, d), "matrix")]
    if not model.tied_embed:
        specs.append(("lm_head", (model.vocab, d), "matrix"))
    specs.append(("final_norm", (d,), "gain"))
    for l in range(model.n_layers):
        p = f"layers.{l}."
        specs += [(p + "attn_norm", (d,), "gain"),
                  (p + "wq", (model.q_dim, d), "matrix"),
                  (p + "wk", (model.kv_dim, d), "matrix"),
                  (p + "wv", (model.kv_dim, d), "matrix")]
        if model.qkv_bias:
            specs += [(p + "bq", (model.q_dim,), "bias"),
                      (p + "bk", (model.kv_dim,), "bias"),
                      (p + "bv", (model.kv_dim,), "bias")]
        if model.qk_norm:
            specs += [(p + "q_norm", (hd,), "gain"), (p + "k_norm", (hd,), "gain")]
        specs += [(p + "wo", (d, model.q_dim), "matrix"),
                  (p + "mlp_norm", (d,), "gain"),
                  (p + "w_gate", (f, d), "matrix"),
                  (p + "w_up", (f, d), "matrix"),
                  (p + "w_down", (d, f), "matrix")]
    return specs


def gen_weights(model: ModelShape, seed: int = 0, threads: int = 8, gain_jitter: float = 0.0) -> Weights:
    """Random-init weights: matrices, embedding and biases N(0, 0.02); norm gains 1.

    `gain_jitter` > 0 draws gains as 1 + jitter * N(0, 1) instead (used by tests so
    that a dropped gain is visible).  Matrices of bf16 models are rounded to bf16;
    gains and biases are float32 arrays whose values are bf16-representable for
    bf16 models.
    """
    w = Weights(model)
    specs = tensor_specs(model)
    is_bf16 = model.dtype == DTYPE_BF16

    def make(idx_spec):
        idx, (name, shape, kind) = idx_spec
        g = _rng(seed, 1000 + idx)
        n = int(np.prod(shape))
        if kind == "gain":
            a = np.ones(n, dtype=np.float32)
            if gain_jitter > 0.0:
                a = a + np.float32(gain_jitter) * g.standard_normal(n, dtype=np.float32)
        else:
            a = g.standard_normal(n, dtype=np.float32)
            a *= np.float32(0.02)
        a = a.reshape(shape)
        if kind == "matrix":
            return name, a, is_bf16
        if is_bf16:
            a = round_to_bf16(a)
        return name, a, False

    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        for name, a, as_bits in ex.map(make, enumerate(specs)):
            w.put(name, a, as_bits)
    return w


@dataclasses.dataclass
class Batch:
    """One sampling batch of a workload (everything except the weights)."""
    prompt_lens: np.ndarray        # [P] int32
    prompt_offsets: np.ndarray     # [P+1] int32
    prompt_tokens: np.ndarray      # [sum Lp] int32, packed
    tau: np.ndarray                # [P] float64
    reward_threshold: np.ndarray   # [P] int32 = floor(tau * V): reward 1 iff last token id < threshold
    caps: np.ndarray               # [P, G] int32: number of generated tokens of each rollout


def gen_batch(wl: Workload) -> Batch:
    P, V = wl.n_prompts, wl.model.vocab
    g = _rng(wl.data_seed, _TAG_PROMPT_LEN)
    lens = wl.prompt_len_lo + np.floor(g.random(P) * (wl.prompt_len_hi - wl.prompt_len_lo + 1)).astype(np.int64)
    lens = np.minimum(lens, wl.prompt_len_hi).astype(np.int32)
    offsets = np.zeros(P + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(lens)
    g = _rng(wl.data_seed, _TAG_PROMPT_TOK)
    toks = np.minimum(np.floor(g.random(int(offsets[-1])) * V), V - 1).astype(np.int32)
    # tau ~ Beta(1/2, 1/2) through its inverse CDF sin^2(pi U / 2)
    g = _rng(wl.data_seed, _TAG_TAU)
    tau = np.sin(0.5 * math.pi * g.random(P)) ** 2
    if wl.forced_explicit is not None:
        for p, t in wl.forced_explicit:
            tau[p] = t
    elif wl.forced_frac > 0.0:
        n_forced = int(math.ceil(wl.forced_frac * P))
        perm = _rng(wl.data_seed, _TAG_FORCED).permutation(P)
        for j in range(n_forced):
            tau[perm[j]] = float(j % 2)
    thr = np.floor(tau * V).astype(np.int32)
    g = _rng(wl.data_seed, _TAG_CAP)
    caps = wl.cap_lo + np.floor(g.random((P, wl.group_size)) * (wl.cap_hi - wl.cap_lo + 1)).astype(np.int64)
    caps = np.minimum(caps, min(wl.cap_hi, wl.max_new)).astype(np.int32)
    return Batch(lens, offsets, toks, tau, thr, caps)
