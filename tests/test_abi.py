"""Host-side checks that need no GPU: the C-ABI library loads and exports every
symbol the header declares; the workspace size function rejects bad shapes."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "pacer.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pacer_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2602_01274_b200 import build
    lib = ctypes.CDLL(build.build_lib())
    names = _declared_symbols()
    assert "pacer_generate" in names and "pacer_preverify" in names and len(names) >= 17
    for n in names:
        assert hasattr(lib, n), n


def test_binding_covers_the_header():
    from paper_2602_01274_b200 import build
    build.build_lib()
    from paper_2602_01274_b200 import binding
    assert sorted(binding.exported_symbols()) == _declared_symbols()


def test_workspace_bytes_host_logic():
    from paper_2602_01274_b200 import build, synth
    build.build_lib()
    from paper_2602_01274_b200 import binding as b
    cfg = synth.CONFIGS["7b_68m"]
    n = b.pacer_workspace_bytes(b.make_cfg(cfg.target, cfg.draft, 1, 1024, 16))
    # the target's cache (values + remainders) and the library's own copy of its projection matrices dominate
    big = 2 * cfg.target.kv_bytes_per_token() * 1024 + cfg.target.streamed_weight_bytes()
    assert big < n < big + (1 << 30)
    assert b.pacer_workspace_bytes(b.make_cfg(cfg.target, cfg.draft, 0, 1024, 16)) == 0
    assert b.pacer_workspace_bytes(b.make_cfg(cfg.target, cfg.draft, 1, 1024, 16, block_b=3)) == 0
    assert b.pacer_strerror if hasattr(b, "pacer_strerror") else True
