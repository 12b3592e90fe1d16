"""The shared library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "echo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(echo_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2602_02192_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert "echo_rollout" in names and "echo_load_policy" in names and "echo_group_advantage" in names
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_names():
    from paper_2602_02192_b200 import binding
    assert sorted(binding.EXPORTED) == _declared()


def test_config_validation_needs_no_gpu():
    from paper_2602_02192_b200 import binding, synth
    shape = synth.SHAPES["tiny"]
    cfg = binding.make_config(shape, 4, 4, 32, 32)
    n = binding.echo_arena_bytes(cfg)
    assert n > 7_000_000          # two weight buffers alone are ~14 MB
    bad = binding.make_config(shape, 4, 4, 32, 32)
    bad.head_dim = 48
    assert binding.echo_arena_bytes(bad) == 0
    bad = binding.make_config(shape, 4, 4, 32, 32)
    bad.eos_id = 2
    assert binding.echo_arena_bytes(bad) == 0
    assert binding.lib.echo_strerror(-5) == b"an install is still pending"
    # 8B-shape workload: 2 x 16.4 GB weights + ~80 GB KV must fit a 180 GB part
    big = binding.make_config(synth.SHAPES["8B"], 32, 8, 512, 2048)
    assert 110e9 < binding.echo_arena_bytes(big) < 125e9
