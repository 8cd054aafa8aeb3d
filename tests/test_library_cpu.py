"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol
the header declares, and validates configurations."""
import ctypes as C
import os
import re

import pytest

from paper_2503_09387_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "videoscan.h")).read()
    declared = set(re.findall(r"\b(vs_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name)


def test_status_strings(lib):
    assert binding.status_string(0) == "ok"
    for code in range(-7, 0):
        assert binding.status_string(code) not in ("ok", "unknown status")
    assert binding.status_string(-99) == "unknown status"


def test_struct_layout_matches_header():
    assert C.sizeof(binding.VsConfig) == 23 * 4
    assert C.sizeof(binding.VsWeights) == 10 * 8
    assert C.sizeof(binding.VsBankInfo) == 4 + 4 + 5 * 8 + 4 + 4 + 8 + 8


def test_workspace_bytes_and_config_validation(lib):
    cfg = binding.make_config(1, 3584, 28, 4, 128, 169, 64, 64, 64)
    small = binding.vs_workspace_bytes(cfg)
    cfg2 = binding.make_config(1, 3584, 28, 4, 128, 169, 64, 64, 128)
    bigger = binding.vs_workspace_bytes(cfg2)
    # growing the bank by 64 carriers costs 64 * (K + V + embedding) bytes, nothing else
    assert bigger - small == pytest.approx(64 * (2 * 4 * 128 * 2 + 3584 * 2 + 4 + 4 + 8 + 8), abs=8 * 256)
    bad = [dict(d_model=100), dict(head_dim=96), dict(n_kv_heads=3), dict(max_tokens_per_frame=300),
           dict(n_streams=0), dict(n_streams=65), dict(evict_policy=3), dict(n_layers=2)]
    base = dict(n_layers=1, d_model=256, n_q_heads=4, n_kv_heads=1, head_dim=64, max_tokens_per_frame=16,
                max_prefix=8, max_text=8, bank_capacity=4)
    for change in bad:
        kw = dict(base)
        kw.update(change)
        with pytest.raises(binding.VsError) as e:
            binding.vs_workspace_bytes(binding.make_config(**kw))
        assert e.value.code in (binding.VS_ERR_INVALID_ARG, binding.VS_ERR_UNSUPPORTED)


def test_null_arguments_are_rejected(lib):
    assert lib.vs_workspace_bytes(None, None) == binding.VS_ERR_INVALID_ARG
    assert lib.vs_frame_prefill(None, None, 0, None, 0, None, None, None) == binding.VS_ERR_INVALID_ARG
    assert lib.vs_decode_step(None, None, 0, None, 0, None, None) == binding.VS_ERR_INVALID_ARG
    assert lib.vs_destroy_stream(None) == binding.VS_ERR_INVALID_ARG
    assert lib.vs_end_turn(None, None, 0) == binding.VS_ERR_INVALID_ARG


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(FileNotFoundError):
        binding.load_library(str(tmp_path / "nope.so"))
