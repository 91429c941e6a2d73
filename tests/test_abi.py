"""The C-ABI library loads and exports every symbol include/dmx.h declares; argument checks
that need no GPU return their codes. No compute calls here."""
import ctypes
import os
import re

import numpy as np

import paper_2510_08522_b200 as D
from paper_2510_08522_b200 import binding as B
from paper_2510_08522_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dmx.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dmx_[a-z_0-9]+)\s*\(", text)))


def test_library_is_built_and_exports_every_declared_symbol():
    build.build(checked=True)
    names = declared_functions()
    assert set(B.EXPORTS) <= set(names)
    for so in ("libdmx.so", "libdmx_checked.so"):       # the checked build has the same ABI
        lib = ctypes.CDLL(build.lib_path(so))
        for n in names:
            assert hasattr(lib, n), (so, n)
    gen = ctypes.CDLL(build.lib_path("libdmx_gen.so"))
    for n in ("dmxgen_normal_fill", "dmxgen_normal_add", "dmxgen_grad_fill", "dmxgen_read_probe"):
        assert hasattr(gen, n)


def test_binding_mirrors_header_constants():
    text = open(os.path.join(ROOT, "include", "dmx.h")).read()
    for name, val in re.findall(r"\b(DMX_[A-Z0-9_]+)\s*=\s*(-?\d+)", text):
        py = name[4:]
        if hasattr(B, py):
            assert getattr(B, py) == int(val), name
    assert B.ST_HDR == 16 and B.FLAG_INTERNAL == 16 and B.ERR_HANDLE == -7


def test_create_rejects_bad_arguments_without_a_gpu():
    assert D.dmx_create(0, 8, [0, 8])[0] == B.ERR_ARG
    assert D.dmx_create(65, 8, [0, 8])[0] == B.ERR_ARG
    assert D.dmx_create(2, 0, [0, 0])[0] == B.ERR_ARG
    assert D.dmx_create(2, 8, [0, 8], 7)[0] == B.ERR_ARG
    assert D.dmx_create(2, 8, [0, 7])[0] == B.ERR_SEGMENTS
    assert D.dmx_create(2, 8, [1, 8])[0] == B.ERR_SEGMENTS
    assert D.dmx_create(2, 8, [0, 5, 4, 8])[0] == B.ERR_SEGMENTS
    assert B.dmx_state_len(None) == B.ERR_HANDLE
    assert B.dmx_destroy(None) == B.OK
    assert B.dmx_step(None, [16], [1], 16, 32, 0.1, 0.9, 48, 64) == B.ERR_HANDLE
    for code in range(-9, 1):
        assert D.strerror(code) and "unknown" not in D.strerror(code)
    assert "unknown" in D.strerror(-99)


def test_a_pointer_that_is_not_a_live_handle_is_refused_without_being_read():
    # handles are looked up in the table of live handles; an arbitrary (unmapped) address must come
    # back as DMX_ERR_HANDLE from every entry point that takes a handle, not as a crash
    bogus = ctypes.c_void_p(0x10)
    assert B.dmx_state_len(bogus) == B.ERR_HANDLE
    assert B.dmx_partials_len(bogus) == B.ERR_HANDLE
    assert B.dmx_launches_per_step(bogus) == B.ERR_HANDLE
    assert B.dmx_set_profiling(bogus, 1) == B.ERR_HANDLE
    assert B.dmx_get_profile(bogus)[0] == B.ERR_HANDLE
    assert B.dmx_check_guards(bogus) == B.ERR_HANDLE
    assert B.dmx_selftest_wait(bogus, 16)[0] == B.ERR_HANDLE
    assert B.dmx_step(bogus, [16], [1], 16, 32, 0.1, 0.9, 48, 64) == B.ERR_HANDLE
    assert B.dmx_step_adam(bogus, [16], [1], 16, 32, 80, 0.1, 0.9, 0.99, 1e-8, 1, 48, 64) == B.ERR_HANDLE
    assert B.dmx_step_partial(bogus, [16], [1], 16, 32, 0.1, 0.9, 48, 64) == B.ERR_HANDLE
    assert B.dmx_step_host(bogus, [16], [16], [1], 16, 32, 0.1, 0.9, 48, 64, 80) == B.ERR_HANDLE
    assert B.dmx_destroy(bogus) == B.ERR_HANDLE
    assert B.dmx_agg_push(bogus, 16, 32)[0] == B.ERR_HANDLE
    assert B.dmx_agg_destroy(bogus) == B.ERR_HANDLE


def test_workload_tables():
    from paper_2510_08522_b200 import workload as W
    for wl in W.WORKLOADS:
        seg = wl.segment_table()
        assert seg[0] == 0 and seg[-1] == wl.P and len(seg) == wl.S + 1 and np.all(np.diff(seg) >= 1)
        for t in (0, 1, wl.steps - 1):
            b = wl.batch_sizes(t)
            assert b.shape == (wl.K,) and b.min() >= 16 and b.max() <= 1024
    seg3 = W.WORKLOADS[3].segment_table()
    sizes = np.diff(seg3)
    assert abs(sizes[26] / seg3[-1] - 0.65) < 1e-6 and abs(sizes[28] / seg3[-1] - 0.15) < 1e-6
    # log-normal tables put boundaries at every residue mod 8
    assert len(set(int(v) % 8 for v in W.WORKLOADS[4].segment_table())) == 8
    # the generator's normals: mean 0, variance 1, streams independent
    z = W.normals(0, W.TAG_NOISE, 1, 0, 0, 1 << 16)
    z2 = W.normals(0, W.TAG_NOISE, 2, 0, 0, 1 << 16)
    assert abs(z.mean()) < 0.02 and abs(z.var() - 1) < 0.02 and abs(np.corrcoef(z, z2)[0, 1]) < 0.02
    assert np.array_equal(W.normals(0, W.TAG_NOISE, 1, 0, 5, 100), z[5:105])


def test_philox_known_answer():
    # Known-answer vectors of Philox4x32-10 from the Random123 distribution's kat_vectors.
    from paper_2510_08522_b200 import workload as W
    r = W.philox4x32(0, 0, 0, 0, 0, 0)
    assert [int(x) for x in r] == [0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8]
    r = W.philox4x32(0xffffffff, 0xffffffff, 0xffffffff, 0xffffffff, 0xffffffff, 0xffffffff)
    assert [int(x) for x in r] == [0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd]
    r = W.philox4x32(0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344, 0xa4093822, 0x299f31d0)
    assert [int(x) for x in r] == [0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1]


def test_header_compiles_as_plain_c(tmp_path):
    # the boundary is a C ABI: the header must be valid C99 on its own (no C++, no CUDA types)
    import subprocess
    src = tmp_path / "use_dmx.c"
    src.write_text('#include "dmx.h"\n'
                   'int use(void) { dmx_handle* h = 0; int64_t seg[2] = {0, 8};\n'
                   '  int rc = dmx_create(2, 8, seg, 1, DMX_F32, &h);\n'
                   '  return rc == DMX_OK ? dmx_state_len(h) + DMX_ST_HDR + DMX_FLAG_INTERNAL + DMX_CTL_ACTIONS : rc; }\n')
    r = subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-fsyntax-only", "-I", os.path.join(ROOT, "include"), str(src)],
                       capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
