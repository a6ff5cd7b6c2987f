"""Host-only checks of the boundary: the library builds for sm_100a, loads, and
exports every function include/saki.h declares.  No compute calls."""
import ctypes
import os
import re

import paper_2609_36601_b200 as P
from paper_2609_36601_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "saki.h")).read()
    return sorted(set(re.findall(r"SAKI_API[^;(]*?\b(saki_\w+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert len(names) >= 10
    for n in names:
        assert hasattr(lib, n), f"{n} declared in saki.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_version_and_error_text_without_a_gpu():
    assert P.version() >= 100
    assert isinstance(P.last_error(), str)


def test_struct_layouts_match_the_header():
    # sizes that the C compiler gives the same structs (checked with a tiny C program)
    import subprocess, tempfile
    src = '#include <stdio.h>\n#include "saki.h"\nint main(){printf("%zu %zu %zu %zu %zu %zu %zu\\n",sizeof(saki_in),sizeof(saki_out),sizeof(saki_spec_in),sizeof(saki_spec_out),sizeof(saki_meta_in),sizeof(saki_meta_out),sizeof(saki_select_in));return 0;}\n'
    with tempfile.TemporaryDirectory() as td:
        c = os.path.join(td, "a.c")
        open(c, "w").write(src)
        exe = os.path.join(td, "a.out")
        subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), c, "-o", exe])
        sizes = [int(v) for v in subprocess.check_output([exe]).split()]
    assert sizes == [ctypes.sizeof(binding.SakiIn), ctypes.sizeof(binding.SakiOut),
                     ctypes.sizeof(binding.SakiSpecIn), ctypes.sizeof(binding.SakiSpecOut),
                     ctypes.sizeof(binding.SakiMetaIn), ctypes.sizeof(binding.SakiMetaOut),
                     ctypes.sizeof(binding.SakiSelectIn)]
