"""CPU-only checks of the boundary: the library builds, loads without a GPU, exports every symbol the
header declares, and its host-side planning functions behave.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

import paper_2601_21686_b200 as S
from paper_2601_21686_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return S.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "stief.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(stief_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"stief_prefill_compress", "stief_append", "stief_decode_attention", "stief_split_combine"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in stief.h but not exported"


def test_status_strings_and_version(lib):
    assert S.stief_version() >= 200
    assert S.status_string(0) == "ok"
    assert "workspace" in S.status_string(S.STIEF_ERR_WORKSPACE)
    assert all(S.status_string(i) for i in range(8))


def test_workspace_planning(lib):
    # 128 bytes of control words | counters [n_units] int32, once per section | then per section:
    # partial_o [parts + n_units][8][r_v] fp32 | partial_lse [parts + n_units][8] fp32; four sections
    up = lambda x: (x + 127) // 128 * 128
    size = lambda n_units, parts, r_v: 128 + 4 * up(n_units * 4) + 4 * (up((parts + n_units) * 8 * r_v * 4) + up((parts + n_units) * 8 * 4))
    assert S.stief_decode_workspace_bytes(4, 32, 8, 64, 148) == size(4 * 8 * 1, 148, 64)
    # a group of 16 query heads per KV head is two units per (sequence, KV head)
    assert S.stief_decode_workspace_bytes(2, 32, 2, 96, 10) == size(2 * 2 * 2, 10, 96)
    # the built-in scratch of the workspace-free entry point holds 359 units at one part per SM of a B200 and r_v = 128
    assert size(359, 148, 128) <= S.STATIC_WORKSPACE_BYTES < size(360, 148, 128)
    assert S.stief_decode_workspace_bytes(0, 32, 8, 64, 1) == 0
    assert S.stief_decode_workspace_bytes(4, 30, 8, 64, 1) == 0          # Hq not a multiple of Hkv
    assert S.stief_decode_num_parts() >= 1                                  # 148 when no device is present
    assert S.stief_decode_workspace_bytes(4, 32, 8, 64, 0) == S.stief_decode_workspace_bytes(4, 32, 8, 64, S.stief_decode_num_parts())
    assert S.stief_host_staging_bytes(4, 32, 8) == 2 * 4 * 32 * 128 * 2 + 2 * 4 * 8 * 128 * 2


def test_host_side_argument_checks_need_no_gpu(lib):
    # NULL descriptors are rejected before anything touches CUDA
    assert lib.stief_append(None, None, None, None, None, None) == S.STIEF_ERR_INVALID_ARG
    assert lib.stief_decode_attention(None, None, None, 0, None, 0, 0, None, None, 0, None, None) == S.STIEF_ERR_INVALID_ARG
    assert lib.stief_advance_seq_lens(None, 4, 1, None) == S.STIEF_ERR_INVALID_ARG


def test_product_never_imports_the_oracle():
    for dirpath, _, files in os.walk(os.path.join(ROOT, "paper_2601_21686_b200")):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b|oracle/|stief_oracle", text, flags=re.M), f
