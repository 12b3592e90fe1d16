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


def test_struct_layouts_match_the_header(tmp_path):
    """The ctypes mirrors of echo_config and echo_stats against the C compiler's view of the header:
    size and the offset of every field (a field added on one side only would shift everything after it)."""
    import subprocess
    from paper_2602_02192_b200 import binding
    fields = {"echo_config": binding.EchoConfig, "echo_stats": binding.EchoStats}
    lines = []
    for name, cls in fields.items():
        lines.append(f'printf("{name} %zu\\n", sizeof({name}));')
        for f, _ in cls._fields_:
            lines.append(f'printf("{name}.{f} %zu\\n", offsetof({name}, {f}));')
    src = tmp_path / "layout.c"
    src.write_text('#include <stddef.h>\n#include <stdio.h>\n#include "echo.h"\nint main(void) {\n' + "\n".join(lines) +
                   "\nreturn 0; }\n")
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    out = dict(l.split() for l in subprocess.check_output([str(exe)], text=True).splitlines())
    for name, cls in fields.items():
        assert int(out[name]) == ctypes.sizeof(cls), name
        for f, _ in cls._fields_:
            assert int(out[f"{name}.{f}"]) == getattr(cls, f).offset, (name, f)
    # and the header declares no field the mirror lacks
    text = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "echo.h")).read(), flags=re.S)
    for name, cls in fields.items():
        body = re.search(r"typedef struct %s \{(.*?)\} %s;" % (name, name), text, flags=re.S).group(1)
        declared = [x.strip() for decl in body.split(";") if decl.strip()
                    for x in re.sub(r"^\s*\w+\s+", "", decl.strip()).split(",")]
        assert declared == [f for f, _ in cls._fields_], name


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
    bad.eos_id = shape.vocab                 # the end token must be a token id (or -1)
    assert binding.echo_arena_bytes(bad) == 0
    assert binding.lib.echo_strerror(-5) == b"an install is still pending"
    # 8B-shape workload: 2 x 16.4 GB weights + ~80 GB KV must fit a 180 GB part
    big = binding.make_config(synth.SHAPES["8B"], 32, 8, 512, 2048)
    assert 110e9 < binding.echo_arena_bytes(big) < 125e9


def test_host_page_plan_matches_oracle_bit_for_bit():
    """The library's page plan (host arithmetic, no GPU) against the oracle's on ragged cases."""
    import numpy as np
    from oracle import pages
    from paper_2602_02192_b200 import binding
    rng = np.random.default_rng(11)
    cases = [([32] * 4, 4, 32, 16), ([512] * 32, 8, 2048, 16), ([20, 33, 16, 1], 3, 9, 16), ([5], 2, 1, 16),
             ([17, 31], 2, 40, 8), ([1024] * 16, 8, 2048, 16)]
    for _ in range(20):
        P = int(rng.integers(1, 9))
        cases.append(([int(x) for x in rng.integers(1, 200, size=P)], int(rng.integers(1, 6)),
                      int(rng.integers(1, 70)), int(rng.choice([4, 16, 32]))))
    for lens, G, T, Z in cases:
        plan = pages.build(lens, G, T, Z)
        table, prefill, n_pages = binding.echo_plan_page_table(lens, G, T, Z)
        assert n_pages == plan.n_pages
        assert table.shape[1] == plan.width
        assert np.array_equal(table, plan.table)
        assert np.array_equal(prefill, plan.prefill_table)
