"""Host-side checks of the C-ABI library: it loads without a GPU, exports every
symbol the header declares, sizes workspaces on the host, and rejects bad
arguments with a status code before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_2510_18692_b200 import build as moga_build
from paper_2510_18692_b200.inputs import CONFIGS, MogaConfig

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    moga_build.build()
    from paper_2510_18692_b200 import binding as b
    return b


def test_every_declared_symbol_is_exported(binding):
    text = open(os.path.join(ROOT, "include", "moga.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(moga_[a-z_0-9]+)\s*\(", text))
    assert {"moga_route", "moga_permute", "moga_group_attn", "moga_unpermute",
            "moga_forward"} <= declared
    for name in declared:
        assert hasattr(binding.lib, name), name
    assert declared >= set(binding.EXPORTS)


def test_workspace_sizes_are_host_only(binding):
    for cfg in CONFIGS.values():
        sh = binding.make_shape(cfg)
        total, scratch = binding.moga_workspace_bytes(sh), binding.moga_scratch_bytes(sh)
        es = 4 if cfg.dtype == "f32" else 2
        tensors = 4 * cfg.B * cfg.H * cfg.T * cfg.D * es + 5 * 4 * cfg.B * cfg.T   # 4 permuted tensors, 5 routing arrays
        assert scratch > 0 and total >= scratch + tensors
        assert total < tensors + scratch + (1 << 20)
    minute = CONFIGS["minute_bf16"]
    assert binding.moga_workspace_bytes(binding.make_shape(minute)) < 30 * 2**30


def _fake(addr=0x10000):
    return ctypes.c_void_p(addr)


def test_bad_arguments_return_codes_without_launch(binding):
    lib = binding.lib
    cfg = CONFIGS["tiny_f32"]
    sh = binding.make_shape(cfg)
    null = ctypes.c_void_p(0)
    z = ctypes.c_size_t(0)
    # null / misaligned pointers
    assert lib.moga_route(ctypes.byref(sh), null, _fake(), null, _fake(), _fake(), null, null, z, null) == 1
    assert lib.moga_route(ctypes.byref(sh), _fake(0x10004), _fake(), null, _fake(), _fake(), null, null, z, null) == 1
    assert lib.moga_unpermute(ctypes.byref(sh), _fake(), null, _fake(), _fake(), null) == 1
    assert lib.moga_route(None, _fake(), _fake(), null, _fake(), _fake(), null, null, z, null) == 1
    # unsupported shapes
    for kw in (dict(M=65), dict(k=9, M=16), dict(D=96), dict(C=130), dict(k=3, M=2),
               dict(N=2**30, k=2)):
        bad = binding.make_shape(cfg.with_(**kw))
        assert binding.moga_workspace_bytes(bad) == 0
        assert lib.moga_route(ctypes.byref(bad), _fake(), _fake(), null, _fake(), _fake(), null, null, z, null) == 2
    # invalid sizes / enums
    for kw in (dict(B=0), dict(N=-1), dict(gate_mode=7)):
        bad = binding.make_shape(cfg.with_(**kw))
        assert lib.moga_route(ctypes.byref(bad), _fake(), _fake(), null, _fake(), _fake(), null, null, z, null) == 1
    bad = binding.make_shape(cfg, route_mode=5)
    assert lib.moga_route(ctypes.byref(bad), _fake(), _fake(), null, _fake(), _fake(), null, null, z, null) == 1
    # workspace missing or too small: nothing is launched
    need = binding.moga_workspace_bytes(sh)
    args = [ctypes.byref(sh)] + [_fake()] * 2 + [null] + [_fake()] * 4 + [null] * 4
    assert lib.moga_forward(*args, null, ctypes.c_size_t(need), null) == 3
    assert lib.moga_forward(*args, _fake(0x10000), ctypes.c_size_t(need - 1), null) == 3
    assert lib.moga_forward(*args, _fake(0x10010), ctypes.c_size_t(need), null) == 3   # misaligned ws
    assert lib.moga_permute(ctypes.byref(sh), _fake(), null, null, null, _fake(), _fake(), _fake(),
                            null, null, null, _fake(), ctypes.c_size_t(16), null) == 3
    # permute wants all three outputs or none
    assert lib.moga_permute(ctypes.byref(sh), _fake(), _fake(), _fake(), _fake(), _fake(), _fake(),
                            _fake(), _fake(), null, null, _fake(), ctypes.c_size_t(need), null) == 1
    # strides must keep rows 16-byte aligned and D contiguous
    bad = binding.make_shape(cfg, strides=(cfg.H * cfg.N * cfg.D, cfg.N * cfg.D, cfg.D - 1))
    assert lib.moga_unpermute(ctypes.byref(bad), _fake(), _fake(), _fake(), _fake(), null) == 1


def test_status_strings(binding):
    assert binding.status_string(0) == "ok"
    assert "workspace" in binding.status_string(3)
