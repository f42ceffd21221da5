"""Decoder forward of the rollout policy pi_theta(o_t | q, o_<t)  (Section 3.1).

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

The paper names the policy only through the model families it trains (Section 4.1:
Qwen2.5-Math-1.5B, Qwen3-4B/8B/14B-Base).  The forward pass written here is the
standard pre-norm decoder of those families:

    h_0      = E[x_t]
    a        = RMSNorm(h; g_attn)
    q, k, v  = a Wq^T (+bq), a Wk^T (+bk), a Wv^T (+bv)
    q, k     = per-head RMSNorm over head_dim with gains g_q, g_k   (Qwen3 only, before RoPE)
    q, k     = RoPE(q, t), RoPE(k, t)       half-split pairing (x_i, x_{i+hd/2}), angle t * theta^(-2i/hd)
    o_j      = softmax_u<=t( q_j . k_u / sqrt(hd) ) v_u,  query head j uses KV head j // (Hq / Hkv)
    h       += o Wo^T
    b        = RMSNorm(h; g_mlp)
    h       += (silu(b Wg^T) * (b Wu^T)) Wd^T
    logits   = RMSNorm(h_L; g_final) W_lm^T      (W_lm = E when embeddings are tied)

    RMSNorm(x; g) = x / sqrt(mean(x^2) + eps) * g,    silu(x) = x / (1 + exp(-x))

Three evaluation modes are kept side by side so that each can be checked against
the others: `forward_full` (whole sequence, causal mask: the definition),
`decode` with per-rollout attention over [prompt KV ; suffix KV] concatenated, and
`decode` with the prompt part and the suffix part attended separately and merged
by their log-sum-exp (what a shared-prefix kernel does).
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Tuple

import numpy as np


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotate x[..., T, H, hd] (T positions given by pos[T]) by the half-split rotary embedding."""
    hd = x.shape[-1]
    half = hd // 2
    i = np.arange(half, dtype=np.float64)
    inv_freq = theta ** (-2.0 * i / hd)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv_freq[None, :]        # [T, half]
    c = np.cos(ang)[:, None, :].astype(x.dtype)
    s = np.sin(ang)[:, None, :].astype(x.dtype)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def softmax_lastdim(s: np.ndarray) -> np.ndarray:
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


class Decoder:
    """Holds the weights in the compute type (float64 by default) and evaluates the policy."""

    def __init__(self, model, weights, dtype=np.float64, cache_weights: bool = True):
        self.m = model
        self.w = weights
        self.dtype = dtype
        self.cache_weights = cache_weights
        self._cache: Dict[str, np.ndarray] = {}
        self.n_rep = model.n_q_heads // model.n_kv_heads

    # -- weights -------------------------------------------------------------------------
    def W(self, name: str) -> np.ndarray:
        if name in self._cache:
            return self._cache[name]
        a = np.asarray(self.w[name], dtype=self.dtype)
        if self.cache_weights:
            self._cache[name] = a
        return a

    def lm_head(self) -> np.ndarray:
        return self.W("embed") if self.m.tied_embed else self.W("lm_head")

    # -- pieces --------------------------------------------------------------------------
    def qkv(self, l: int, a: np.ndarray, pos: np.ndarray):
        """a [T, d] at positions pos [T] -> q [T, Hq, hd], k [T, Hkv, hd], v [T, Hkv, hd] (q, k rotated)."""
        m, p = self.m, f"layers.{l}."
        T = a.shape[0]
        q = a @ self.W(p + "wq").T
        k = a @ self.W(p + "wk").T
        v = a @ self.W(p + "wv").T
        if m.qkv_bias:
            q = q + self.W(p + "bq")
            k = k + self.W(p + "bk")
            v = v + self.W(p + "bv")
        q = q.reshape(T, m.n_q_heads, m.head_dim)
        k = k.reshape(T, m.n_kv_heads, m.head_dim)
        v = v.reshape(T, m.n_kv_heads, m.head_dim)
        if m.qk_norm:
            q = rmsnorm(q, self.W(p + "q_norm"), m.rms_eps)
            k = rmsnorm(k, self.W(p + "k_norm"), m.rms_eps)
        q = rope(q, pos, m.rope_theta)
        k = rope(k, pos, m.rope_theta)
        return q, k, v

    def mlp(self, l: int, h: np.ndarray) -> np.ndarray:
        m, p = self.m, f"layers.{l}."
        b = rmsnorm(h, self.W(p + "mlp_norm"), m.rms_eps)
        return (silu(b @ self.W(p + "w_gate").T) * (b @ self.W(p + "w_up").T)) @ self.W(p + "w_down").T

    def logits_from_hidden(self, h: np.ndarray) -> np.ndarray:
        return rmsnorm(h, self.W("final_norm"), self.m.rms_eps) @ self.lm_head().T

    # -- mode 1: the definition ----------------------------------------------------------
    def forward_full(self, tokens: np.ndarray, return_kv: bool = False, last_only: bool = False, positions=None):
        """Causal forward over one whole sequence.  Returns logits [T, V] (or [1, V] with last_only, or one row per
        entry of `positions`: the LM head is then applied to those positions only).

        With return_kv also returns [(K_l, V_l)] with K_l, V_l of shape [T, Hkv, hd] (K after RoPE).
        """
        m = self.m
        tokens = np.asarray(tokens, dtype=np.int64)
        T = tokens.shape[0]
        pos = np.arange(T)
        h = self.W("embed")[tokens].astype(self.dtype)
        causal = np.triu(np.ones((T, T), dtype=bool), k=1)          # True above the diagonal: masked
        scale = 1.0 / math.sqrt(m.head_dim)
        kv = []
        for l in range(m.n_layers):
            p = f"layers.{l}."
            a = rmsnorm(h, self.W(p + "attn_norm"), m.rms_eps)
            q, k, v = self.qkv(l, a, pos)
            kv.append((k, v))
            o = np.empty_like(q)
            for j in range(m.n_q_heads):
                g = j // self.n_rep
                s = (q[:, j, :] @ k[:, g, :].T) * scale
                s = np.where(causal, -np.inf, s)
                o[:, j, :] = softmax_lastdim(s) @ v[:, g, :]
            h = h + o.reshape(T, m.q_dim) @ self.W(p + "wo").T
            h = h + self.mlp(l, h)
        if last_only:
            h = h[-1:, :]
        elif positions is not None:
            h = h[np.asarray(positions, dtype=np.int64), :]
        logits = self.logits_from_hidden(h)
        return (logits, kv) if return_kv else logits

    def prefill(self, tokens: np.ndarray):
        """One prompt evaluated once: its KV for every layer and the logits at its last position."""
        logits, kv = self.forward_full(tokens, return_kv=True, last_only=True)
        return kv, logits[0]

    # -- modes 2 and 3: KV-cached decode for the rollouts of one group ----------------------
    def attend_concat(self, q, Kp, Vp, Ks, Vs):
        """One query position q [Hq, hd] over prompt KV [Lp, Hkv, hd] followed by its own suffix KV [n, Hkv, hd]."""
        m = self.m
        K = np.concatenate([Kp, Ks], axis=0)
        V = np.concatenate([Vp, Vs], axis=0)
        scale = 1.0 / math.sqrt(m.head_dim)
        o = np.empty_like(q)
        for j in range(m.n_q_heads):
            g = j // self.n_rep
            s = (K[:, g, :] @ q[j]) * scale
            o[j] = softmax_lastdim(s) @ V[:, g, :]
        return o

    def attend_shared_prefix(self, q, Kp, Vp, Ks, Vs):
        """Same result as attend_concat, computed as two partial softmaxes merged by log-sum-exp.

        (m1, l1, O1) over the prompt part, (m2, l2, O2) over the suffix part;
        M = max(m1, m2), l = l1 e^{m1-M} + l2 e^{m2-M}, O = (O1 l1 e^{m1-M} + O2 l2 e^{m2-M}) / l
        with O1, O2 the normalised partial outputs.
        """
        m = self.m
        scale = 1.0 / math.sqrt(m.head_dim)
        o = np.empty_like(q)
        for j in range(m.n_q_heads):
            g = j // self.n_rep
            parts = []
            for K, V in ((Kp, Vp), (Ks, Vs)):
                s = (K[:, g, :] @ q[j]) * scale
                mx = np.max(s)
                e = np.exp(s - mx)
                l = np.sum(e)
                parts.append((mx, l, (e @ V[:, g, :]) / l))
            (m1, l1, o1), (m2, l2, o2) = parts
            M = max(m1, m2)
            a1, a2 = l1 * math.exp(m1 - M), l2 * math.exp(m2 - M)
            o[j] = (o1 * a1 + o2 * a2) / (a1 + a2)
        return o

    def decode(self, tokens: np.ndarray, pos: np.ndarray, prompt_kv, suffix_kv: List[list],
               shared_prefix: bool = False) -> np.ndarray:
        """One decode step for R rollouts of one group.

        tokens [R]: the input token of each rollout; pos [R]: its absolute position
        (prompt length + number of suffix tokens already cached).  prompt_kv is the
        group's shared [(K_l, V_l)]; suffix_kv[r] is rollout r's own list of
        [K_l, V_l] arrays of shape [n_r, Hkv, hd], extended in place by this call.
        Returns logits [R, V] for the next token of every rollout.
        """
        m = self.m
        tokens = np.asarray(tokens, dtype=np.int64)
        R = tokens.shape[0]
        h = self.W("embed")[tokens].astype(self.dtype)
        attend = self.attend_shared_prefix if shared_prefix else self.attend_concat
        for l in range(m.n_layers):
            p = f"layers.{l}."
            a = rmsnorm(h, self.W(p + "attn_norm"), m.rms_eps)
            q, k, v = self.qkv(l, a, pos)
            o = np.empty_like(q)
            Kp, Vp = prompt_kv[l]
            for r in range(R):
                Ks = np.concatenate([suffix_kv[r][l][0], k[r:r + 1]], axis=0)
                Vs = np.concatenate([suffix_kv[r][l][1], v[r:r + 1]], axis=0)
                suffix_kv[r][l] = [Ks, Vs]
                o[r] = attend(q[r], Kp, Vp, Ks, Vs)
            h = h + o.reshape(R, m.q_dim) @ self.W(p + "wo").T
            h = h + self.mlp(l, h)
        return self.logits_from_hidden(h)

    def empty_suffix(self) -> list:
        m = self.m
        z = np.zeros((0, m.n_kv_heads, m.head_dim), dtype=self.dtype)
        return [[z, z] for _ in range(m.n_layers)]
