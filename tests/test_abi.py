"""The C-ABI library builds for sm_100a, loads, and exports every function include/confu.h declares.
No compute call is made here (no GPU needed)."""
import os
import re

from paper_2603_08899_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "confu.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(confu_[a-z_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_the_header():
    build.build()
    L = binding.lib()
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(L, n), f"{n} declared in confu.h but not exported"
    assert sorted(binding.EXPORTS) == names, "binding.py and confu.h disagree on the entry points"


def test_status_strings_and_host_side_argument_errors():
    L = binding.lib()
    assert L.confu_status_string(0) == b"ok"
    assert b"workspace" in L.confu_status_string(-4)
    assert b"sibling" in L.confu_status_string(4)
    # pure host-side checks that return before touching CUDA
    assert L.confu_destroy(None) == -1
    assert L.confu_set_workspace(None, None, 0) == -1
    assert L.confu_accept_workspace_bytes(4, 60, 128256) > 0
    assert L.confu_accept_workspace_bytes(-1, 60, 128256) == 0
