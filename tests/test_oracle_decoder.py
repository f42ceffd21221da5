"""Pins for oracle/decoder.py: an independent library model (Hugging Face Qwen2 / Qwen3 built from a
config, CPU, float64) with the same weights, plus mode-against-mode checks and special cases."""
import dataclasses
import math

import numpy as np
import pytest
import torch

from oracle.decoder import Decoder, rmsnorm, rope, silu
from paper_2605_26606_b200 import workloads as wl

MINI2 = wl.ModelShape("mini-qwen2", 2, 64, 4, 2, 16, 96, 512, dtype=wl.DTYPE_F32, tied_embed=True, qkv_bias=True)
MINI3 = wl.ModelShape("mini-qwen3", 2, 64, 4, 2, 32, 96, 512, dtype=wl.DTYPE_F32, rope_theta=1e6, qk_norm=True)


def _hf_model(model, w):
    from transformers import Qwen2Config, Qwen2ForCausalLM, Qwen3Config, Qwen3ForCausalLM
    common = dict(vocab_size=model.vocab, hidden_size=model.d_model, intermediate_size=model.d_ff,
                  num_hidden_layers=model.n_layers, num_attention_heads=model.n_q_heads,
                  num_key_value_heads=model.n_kv_heads, rms_norm_eps=model.rms_eps, rope_theta=model.rope_theta,
                  tie_word_embeddings=model.tied_embed, max_position_embeddings=512, attn_implementation="eager")
    if model.qk_norm:
        hf = Qwen3ForCausalLM(Qwen3Config(head_dim=model.head_dim, attention_bias=False, **common))
    else:
        assert model.head_dim * model.n_q_heads == model.d_model
        hf = Qwen2ForCausalLM(Qwen2Config(**common))
    hf = hf.double().eval()
    t = lambda name: torch.from_numpy(np.asarray(w[name], dtype=np.float64))
    sd = {"model.embed_tokens.weight": t("embed"), "model.norm.weight": t("final_norm")}
    sd["lm_head.weight"] = t("embed") if model.tied_embed else t("lm_head")
    for l in range(model.n_layers):
        a, b = f"model.layers.{l}.", f"layers.{l}."
        for hf_n, n in (("q_proj", "wq"), ("k_proj", "wk"), ("v_proj", "wv"), ("o_proj", "wo")):
            sd[a + f"self_attn.{hf_n}.weight"] = t(b + n)
        if not model.qk_norm:
            for hf_n, n, dim in (("q_proj", "bq", model.q_dim), ("k_proj", "bk", model.kv_dim), ("v_proj", "bv", model.kv_dim)):
                sd[a + f"self_attn.{hf_n}.bias"] = t(b + n) if model.qkv_bias else torch.zeros(dim, dtype=torch.float64)
        else:
            sd[a + "self_attn.q_norm.weight"] = t(b + "q_norm")
            sd[a + "self_attn.k_norm.weight"] = t(b + "k_norm")
        for hf_n, n in (("gate_proj", "w_gate"), ("up_proj", "w_up"), ("down_proj", "w_down")):
            sd[a + f"mlp.{hf_n}.weight"] = t(b + n)
        sd[a + "input_layernorm.weight"] = t(b + "attn_norm")
        sd[a + "post_attention_layernorm.weight"] = t(b + "mlp_norm")
    missing, unexpected = hf.load_state_dict(sd, strict=False)
    assert not unexpected and all("rotary" in k for k in missing), (missing, unexpected)
    return hf


@pytest.mark.parametrize("model", [MINI2, MINI3, dataclasses.replace(MINI2, name="mini-nobias", qkv_bias=False, tied_embed=False)],
                         ids=lambda m: m.name)
def test_full_forward_matches_library_model(model):
    w = wl.gen_weights(model, seed=3, threads=1, gain_jitter=0.2)
    # larger weights than N(0, 0.02) so that attention and the MLP are far from their linear regime
    for n in w.names():
        if w[n].ndim == 2:
            w.put(n, w[n] * 8.0, False)
    dec = Decoder(model, w)
    toks = np.random.default_rng(0).integers(0, model.vocab, size=23)
    mine = dec.forward_full(toks)
    with torch.no_grad():
        ref = _hf_model(model, w)(torch.from_numpy(toks)[None]).logits[0].numpy()
    assert np.std(ref) > 0.1
    # the library model builds its rotary tables in float32, which bounds the agreement
    assert np.max(np.abs(mine - ref)) < 2e-5


@pytest.fixture(scope="module")
def tiny():
    w = wl.gen_weights(wl.TINY, seed=0, threads=2, gain_jitter=0.1)
    return Decoder(wl.TINY, w)


def test_cached_decode_equals_full_recompute(tiny):
    rng = np.random.default_rng(1)
    prompt = rng.integers(0, wl.TINY.vocab, size=9)
    conts = [rng.integers(0, wl.TINY.vocab, size=6) for _ in range(3)]
    pkv, last = tiny.prefill(prompt)
    full0 = tiny.forward_full(prompt)
    assert np.max(np.abs(last - full0[-1])) < 1e-12
    for shared in (False, True):
        suffix = [tiny.empty_suffix() for _ in conts]
        for s in range(6):
            x = np.array([c[s] for c in conts])
            logits = tiny.decode(x, np.full(3, len(prompt) + s), pkv, suffix, shared_prefix=shared)
            for r, c in enumerate(conts):
                ref = tiny.forward_full(np.concatenate([prompt, c[:s + 1]]))[-1]
                assert np.max(np.abs(logits[r] - ref)) < 1e-11


def test_shared_prefix_merge_equals_concatenated_softmax(tiny):
    rng = np.random.default_rng(2)
    m = wl.TINY
    q = rng.normal(size=(m.n_q_heads, m.head_dim)) * 3
    Kp, Vp = rng.normal(size=(2, 11, m.n_kv_heads, m.head_dim))
    Ks, Vs = rng.normal(size=(2, 4, m.n_kv_heads, m.head_dim))
    a = tiny.attend_concat(q, Kp, Vp, Ks, Vs)
    b = tiny.attend_shared_prefix(q, Kp, Vp, Ks, Vs)
    assert np.max(np.abs(a - b)) < 1e-13
    # against a library softmax on the duplicated prefix
    K = torch.from_numpy(np.concatenate([Kp, Ks])); V = torch.from_numpy(np.concatenate([Vp, Vs]))
    for j in range(m.n_q_heads):
        g = j // (m.n_q_heads // m.n_kv_heads)
        p = torch.softmax(K[:, g] @ torch.from_numpy(q[j]) / math.sqrt(m.head_dim), dim=0)
        assert np.max(np.abs((p @ V[:, g]).numpy() - a[j])) < 1e-13


def test_causality(tiny):
    rng = np.random.default_rng(3)
    t = rng.integers(0, wl.TINY.vocab, size=12)
    a = tiny.forward_full(t)
    t2 = t.copy(); t2[8:] = rng.integers(0, wl.TINY.vocab, size=4)
    b = tiny.forward_full(t2)
    assert np.array_equal(a[:8], b[:8]) and not np.allclose(a[8:], b[8:])


def test_degenerate_model_is_one_matmul():
    w = wl.gen_weights(wl.TINY, seed=0, threads=2)
    for l in range(wl.TINY.n_layers):
        for n in ("wo", "w_down"):
            w.put(f"layers.{l}.{n}", np.zeros_like(w[f"layers.{l}.{n}"]), False)
    dec = Decoder(wl.TINY, w)
    t = np.array([5, 17, 1999])
    e = w["embed"][t].astype(np.float64)
    want = (e / np.sqrt((e * e).mean(-1, keepdims=True) + 1e-6)) @ w["lm_head"].astype(np.float64).T
    assert np.max(np.abs(dec.forward_full(t) - want)) < 1e-13


def test_rope_properties():
    rng = np.random.default_rng(4)
    x = rng.normal(size=(1, 3, 64)); y = rng.normal(size=(1, 3, 64))
    assert np.array_equal(rope(x, np.array([0]), 1e4), x)                         # position 0 is the identity
    for m_, n_ in ((5, 2), (105, 102), (1003, 1000)):
        xr, yr = rope(x, np.array([m_]), 1e4), rope(y, np.array([n_]), 1e4)
        assert np.allclose(np.linalg.norm(xr, axis=-1), np.linalg.norm(x, axis=-1))
        dots = np.sum(xr * yr, axis=-1)
        if m_ == 5:
            base = dots
        assert np.allclose(dots, base, atol=1e-9)                                   # depends on m - n only
    # pair (i, i + hd/2) turns by angle t * theta^(-2i/hd)
    e = np.zeros((1, 1, 8)); e[0, 0, 1] = 1.0
    r = rope(e, np.array([3]), 100.0)
    ang = 3 * 100.0 ** (-2 * 1 / 8)
    assert np.allclose(r[0, 0], [0, math.cos(ang), 0, 0, 0, math.sin(ang), 0, 0])


def test_rmsnorm_and_silu_properties():
    rng = np.random.default_rng(5)
    x = rng.normal(size=(4, 32))
    y = rmsnorm(x, np.ones(32), 0.0)
    assert np.allclose(np.sqrt((y * y).mean(-1)), 1.0)
    assert np.allclose(rmsnorm(7.0 * x, np.ones(32), 0.0), y)
    g = rng.normal(size=32)
    assert np.allclose(rmsnorm(x, g, 1e-6), y * g, atol=1e-5)
    assert silu(np.array([0.0]))[0] == 0.0
    assert silu(np.array([40.0]))[0] == pytest.approx(40.0)
    assert silu(np.array([1.0]))[0] == pytest.approx(1.0 / (1.0 + math.exp(-1.0)))
    assert np.allclose(silu(x), torch.nn.functional.silu(torch.from_numpy(x)).numpy())
