"""The C-ABI library builds for sm_100a, loads, and exports every symbol include/kdkl.h declares."""
import os
import re

import __graft_entry__ as entry
from paper_2608_03796_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    src = open(os.path.join(ROOT, "include", "kdkl.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(kdkl_[a-z0-9_]+)\s*\(", src)))


def test_library_builds_loads_and_exports_declared_symbols():
    entry.build()
    L = binding.lib()
    names = _declared_symbols()
    assert len(names) >= 8
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(binding.EXPORTS)


def test_sizes_without_a_gpu():
    entry.build()
    # workspace grows linearly with T at fixed chunk: the vocabulary-sized part is per chunk
    a = binding.kdkl_workspace_bytes(32768, 4096, 131072, 100, 4096)
    b = binding.kdkl_workspace_bytes(65536, 4096, 131072, 100, 4096)
    c = binding.kdkl_workspace_bytes(131072, 4096, 131072, 100, 4096)
    assert abs((c - b) - 2 * (b - a)) <= 4096
    per_token = (b - a) / 32768
    assert per_token < 2500                      # bytes of saved state per token at K = 100
    assert a - 32768 * per_token < 1.2 * 2 ** 30  # constant part: one [chunk, V] bf16 buffer + partials
    assert binding.kdkl_workspace_bytes(0, 1, 1, 1) == 0
    assert binding.kdkl_host_arena_bytes(256, 256, 4096, 16, 64) > binding.kdkl_workspace_bytes(256, 256, 4096, 16, 64)


def test_options_struct_layout():
    o = binding.make_options(teacher_mode=1, denom_override=3.0)
    assert o.struct_size == 20 and o.teacher_mode == 1 and o.denom_override == 3.0
