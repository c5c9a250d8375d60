"""Boundary checks that need no GPU: the C-ABI library loads, exports every symbol that
include/equiforge.h declares, and rejects bad arguments on the host with status codes."""
import ctypes
import os
import re

import pytest

import paper_2609_12330_b200 as ef
from paper_2609_12330_b200 import build as ef_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ef_build.build()
    return ef.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "equiforge.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ef_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in equiforge.h but not exported"
    assert sorted(ef.EXPORTS) == names


def test_status_strings_and_version(lib):
    assert lib.ef_version() >= 100
    seen = {lib.ef_status_string(c) for c in range(9)}
    assert len(seen) == 9 and lib.ef_status_string(0) == b"ok"


def test_host_side_argument_validation(lib):
    p = ctypes.c_void_p
    one = p(4096)  # non-null, 16-byte aligned fake pointers: validation fails before any dereference
    null = p(0)
    # null pointers
    assert lib.ef_gqa_decode(null, one, one, one, 1, 4, 1, 8, 128, 1.0, one, 1 << 30, null) == 1
    # bad shapes
    assert lib.ef_gqa_decode(one, one, one, one, 1, 5, 2, 8, 128, 1.0, one, 1 << 30, null) == 2   # Hq % Hkv
    assert lib.ef_gqa_decode(one, one, one, one, 0, 4, 1, 8, 128, 1.0, one, 1 << 30, null) == 2
    # unsupported (no fallback)
    assert lib.ef_gqa_decode(one, one, one, one, 1, 4, 1, 8, 64, 1.0, one, 1 << 30, null) == 3    # D != 128
    assert lib.ef_gqa_decode(one, one, one, one, 1, 32, 1, 8, 128, 1.0, one, 1 << 30, null) == 3  # group > 8
    # alignment
    assert lib.ef_gqa_decode(p(4098), one, one, one, 1, 4, 1, 8, 128, 1.0, one, 1 << 30, null) == 4
    # workspace
    assert lib.ef_gqa_decode(one, one, one, one, 1, 4, 1, 8, 128, 1.0, null, 0, null) == 5
    assert lib.ef_gqa_decode(one, one, one, one, 1, 4, 1, 8, 128, 1.0, one, 16, null) == 5
    # the per-sequence-length decode: same rules, plus the length array and the batch limit
    assert lib.ef_gqa_decode_varlen(one, one, one, null, one, 1, 4, 1, 8, 128, 1.0, one, 1 << 30, null) == 1
    assert lib.ef_gqa_decode_varlen(one, one, one, one, one, 1, 5, 2, 8, 128, 1.0, one, 1 << 30, null) == 2
    assert lib.ef_gqa_decode_varlen(one, one, one, one, one, 1025, 4, 1, 8, 128, 1.0, one, 1 << 30, null) == 3   # B > 1024
    assert lib.ef_gqa_decode_varlen(one, one, one, p(4098), one, 1, 4, 1, 8, 128, 1.0, one, 1 << 30, null) == 4
    assert lib.ef_gqa_decode_varlen(one, one, one, one, one, 1, 4, 1, 8, 128, 1.0, one, 16, null) == 5
    # windowed decode, LayerNorm projection, attention with grouped heads / window / sinks
    assert lib.ef_gqa_decode_window(one, one, one, null, 1, 4, 1, 8, 128, 1.0, 4, 0, one, 1 << 30, null) == 1
    assert lib.ef_gqa_decode_window(one, one, one, one, 1, 4, 1, 8, 128, 1.0, -1, 0, one, 1 << 30, null) == 2
    assert lib.ef_gqa_decode_window(one, one, one, one, 1, 4, 1, 8, 64, 1.0, 4, 0, one, 1 << 30, null) == 3
    assert lib.ef_layernorm_matmul(one, one, null, one, one, 4, 64, 8, 1e-5, one, 1 << 30, null) == 1      # beta missing
    assert lib.ef_layernorm_matmul(one, one, one, one, one, 16, 64, 8, 1e-5, one, 1 << 30, null) == 3       # M > 15
    assert lib.ef_layernorm_matmul(one, one, one, one, one, 4, 60, 8, 1e-5, one, 1 << 30, null) == 3        # K % 64
    assert lib.ef_qknorm_attn_ex(one, one, one, one, one, null, 1, 4, 2, 64, 128, 1e-6, 1.0, 1, 0, 0, one, 1 << 30, null) == 1
    assert lib.ef_qknorm_attn_ex(one, one, one, one, one, one, 1, 5, 2, 64, 128, 1e-6, 1.0, 1, 0, 0, one, 1 << 30, null) == 2   # Hq % Hkv
    assert lib.ef_qknorm_attn_ex(one, one, one, one, one, one, 1, 4, 2, 64, 128, 1e-6, 1.0, 0, 16, 0, one, 1 << 30, null) == 3  # window, not causal
    assert lib.ef_qknorm_attn_ex(one, one, one, one, one, one, 1, 4, 2, 64, 128, 1e-6, 1.0, 1, 16, 200, one, 1 << 30, null) == 3  # sinks > 128
    assert lib.ef_qknorm_attn_ex(one, one, one, one, one, one, 1, 4, 2, 64, 128, 1e-6, 0.0, 1, 0, 0, one, 1 << 30, null) == 3   # scale <= 0
    assert lib.ef_workspace_init(null, 4096, null) == 1
    assert lib.ef_workspace_init(one, 16, null) == 5


def test_workspace_queries(lib):
    assert lib.ef_gqa_decode_workspace_bytes(8, 32, 8, 4096, 128) >= 4096
    assert lib.ef_gqa_decode_workspace_bytes(0, 32, 8, 4096, 128) == 0
