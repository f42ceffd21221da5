"""The C-ABI library loads without a GPU and exports every symbol include/pc.h declares; host-side
argument checks answer before any CUDA call."""
import ctypes as C
import os
import re

import pytest

from paper_2605_26606_b200 import binding as B
from paper_2605_26606_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return B._lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "pc.h")).read()
    declared = re.findall(r"PC_API\s+[\w\s\*]+?\b(pc_\w+)\s*\(", header)
    assert sorted(declared) == sorted(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert B.pc_status_string(B.PC_OK) == "ok"
    assert "argument" in B.pc_status_string(B.PC_ERR_INVALID_ARG)
    assert B.pc_status_string(1234) == "unknown status"


def _desc(**kw):
    base = dict(n_layers=1, d_model=64, n_q_heads=2, n_kv_heads=1, head_dim=64, d_ff=64, vocab=32, rms_eps=1e-6,
                rope_theta=1e4, dtype=0, tied_embed=1, qk_norm=0, qkv_bias=0)
    base.update(kw)
    return B.ModelDesc(**base)


def test_create_rejects_bad_arguments_on_the_host(lib):
    out = C.c_void_p()
    w = B.WeightsDesc()
    assert lib.pc_create(None, C.byref(w), C.byref(out)) == B.PC_ERR_INVALID_ARG
    assert lib.pc_create(C.byref(_desc(head_dim=48)), C.byref(w), C.byref(out)) == B.PC_ERR_SHAPE
    assert lib.pc_create(C.byref(_desc(n_q_heads=3, n_kv_heads=2)), C.byref(w), C.byref(out)) == B.PC_ERR_SHAPE
    assert lib.pc_create(C.byref(_desc(dtype=7)), C.byref(w), C.byref(out)) == B.PC_ERR_INVALID_ARG
    assert lib.pc_create(C.byref(_desc()), C.byref(w), C.byref(out)) == B.PC_ERR_INVALID_ARG      # null weight pointers
    assert lib.pc_create(C.byref(_desc(half_gemm=1)), C.byref(w), C.byref(out)) == B.PC_ERR_INVALID_ARG   # half operands need a bf16 model
    assert lib.pc_create(C.byref(_desc(dtype=1, half_gemm=2)), C.byref(w), C.byref(out)) == B.PC_ERR_INVALID_ARG
    assert out.value is None


def test_entry_points_reject_bad_arguments_on_the_host(lib):
    assert lib.pc_sample(None, -1, 8, None, None, 1.0, 0, None, None, None, None, None, None, None, 0) == B.PC_ERR_INVALID_ARG
    assert lib.pc_sample(None, 4, 8, None, None, 1.0, 0, None, None, None, None, None, None, None, 0) == B.PC_ERR_INVALID_ARG
    assert lib.pc_sample(None, 0, 8, None, None, 1.0, 0, None, None, None, None, None, None, None, 0) == B.PC_OK
    assert lib.pc_group_stats(None, 3, None, None, None, None, None, None, None, None, 0) == B.PC_ERR_INVALID_ARG
    assert lib.pc_group_stats(None, 0, None, None, None, None, None, None, None) == B.PC_OK
    assert lib.pc_grpo_advantage(None, 2, None, None, None, None, None) == B.PC_ERR_INVALID_ARG
    assert lib.pc_reward_last_token(None, 5, None, None, None, None) == B.PC_ERR_INVALID_ARG
    prm = B.AllocParams(0.5, 0.25, 1.0, 4, 4)      # p_lower > p_upper
    assert lib.pc_allocate(None, 0, None, None, C.byref(prm), None, None, None, None, None) == B.PC_ERR_INVALID_ARG
    assert lib.pc_decode_step(None, None, 1, *([None] * 6), 1, None, 1, None, None, 0, None, None, 0, None, None) \
        == B.PC_ERR_INVALID_ARG
    assert lib.pc_workspace_bytes(None, 1, 1, None) == B.PC_ERR_INVALID_ARG


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_LIB", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        B.pc_status_string(0)
