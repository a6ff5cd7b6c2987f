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


def test_argument_validation_returns_codes_before_any_device_work():
    """Bad arguments are rejected, and empty batches accepted, on the host: these calls return before the
    library touches a device, so they behave the same on a machine without a GPU."""
    lib = binding.load_library()
    C = ctypes
    null = C.c_void_p(None)
    assert lib.saki_route_fwd(None, None, null) == 1
    si, so = binding.SakiIn(), binding.SakiOut()
    si.N, si.V, si.dtype, si.eps, si.temperature = 4, 1, 1, 0.1, 1.0          # V < 2
    assert lib.saki_route_fwd(C.byref(si), C.byref(so), null) == 1 and "V" in P.last_error()
    si.V, si.eps = 128, float("nan")
    assert lib.saki_route_fwd(C.byref(si), C.byref(so), null) == 1
    si.eps, si.temperature = 0.1, 0.0
    assert lib.saki_route_fwd(C.byref(si), C.byref(so), null) == 1
    si.temperature, si.dtype = 1.0, 7
    assert lib.saki_route_fwd(C.byref(si), C.byref(so), null) == 1
    si.dtype, si.N, si.ld_s, si.ld_t = 1, 0, 128, 128                          # empty batch: a no-op
    assert lib.saki_route_fwd(C.byref(si), C.byref(so), null) == 0
    assert lib.saki_route_fwd_bwd(C.byref(si), C.byref(so), null, 128, 1.0, null) == 0
    assert lib.saki_route_fwd_bwd(C.byref(si), C.byref(so), null, 64, 1.0, null) == 1      # ld_g < V
    assert lib.saki_route_fwd_bwd_noalloc(C.byref(si), C.byref(so), null, 128, float("inf"), null) == 1
    mi, mo = binding.SakiMetaIn(), binding.SakiMetaOut()
    mi.N, mi.V, mi.dtype, mi.ld_s, mi.temperature = 0, 128, 1, 128, 1.0
    assert lib.saki_route_bwd_from_meta(C.byref(mi), C.byref(mo), null, 128, 1.0, null) == 0
    mi.temperature = -1.0
    assert lib.saki_route_bwd_from_meta(C.byref(mi), C.byref(mo), null, 128, 1.0, null) == 1
    sel = binding.SakiSelectIn()
    sel.N, sel.B, sel.mode = 0, 0, 1
    assert lib.saki_select_tm(C.byref(sel), null, null, null) == 0
    sel.mode = 9
    assert lib.saki_select_tm(C.byref(sel), null, null, null) == 1
    sp, spo = binding.SakiSpecIn(), binding.SakiSpecOut()
    sp.B, sp.K, sp.V, sp.dtype, sp.eps, sp.temperature = 2, 17, 128, 1, 0.1, 1.0           # K outside [1,16]
    assert lib.saki_spec_verify(C.byref(sp), C.byref(spo), null) == 1


def test_new_entry_points_validate_on_the_host():
    """saki_vshard_* and saki_lmhead_lse reject bad arguments, and accept empty batches, before any device work."""
    lib = binding.load_library()
    C = ctypes
    null = C.c_void_p(None)
    vi = binding.SakiVshardIn()
    vi.N, vi.V, vi.V_local, vi.v0, vi.dtype, vi.eps, vi.temperature, vi.rank, vi.world = 0, 1000, 500, 0, 1, 0.1, 1.0, 0, 2
    assert lib.saki_vshard_partial(C.byref(vi), 0, null, null, null, 0, 1.0, null) == 0           # empty batch
    assert lib.saki_vshard_partial(C.byref(vi), 4, null, null, null, 0, 1.0, null) == 1 and "stage" in P.last_error()
    vi.v0 = 600                                                                                    # slice past the vocabulary
    assert lib.saki_vshard_partial(C.byref(vi), 0, null, null, null, 0, 1.0, null) == 1
    vi.v0, vi.rank = 0, 2                                                                          # rank outside the world
    assert lib.saki_vshard_combine(C.byref(vi), 0, null, null, None, null, null) == 1
    vi.rank, vi.N = 1, 4                                                                           # NULL proposal
    n = C.c_int32(0)
    assert lib.saki_vshard_combine_host(C.byref(vi), 0, null, null, None, C.byref(n)) == 1
    li = binding.SakiLmheadIn()
    li.N, li.d, li.V, li.ld_h, li.ld_w, li.temperature = 0, 64, 256, 64, 64, 1.0
    assert lib.saki_lmhead_lse(C.byref(li), null, 256, null, null, null, 0, null) == 0             # empty batch
    li.N = 8
    assert lib.saki_lmhead_lse(C.byref(li), null, 256, null, null, null, 0, null) == 1             # NULL pointers
    li.d = 4
    assert lib.saki_lmhead_lse(C.byref(li), null, 256, null, null, null, 0, null) == 1
    assert lib.saki_lmhead_scratch_bytes(128, 512) == 128 * 2 * 3 * 4 + 256
    assert lib.saki_set_wait_limit(0) == 0 and lib.saki_set_phase_clock(0) == 0
