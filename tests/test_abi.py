"""The C-ABI library loads without a GPU and exports every function that
include/difr.h declares; host-only entry points behave."""
import os

import pytest
import re

import paper_2511_02620_b200 as difr
from paper_2511_02620_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "difr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(difr_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_function():
    build()
    L = difr.lib()
    names = _declared()
    assert {"difr_score_gm", "difr_score_ipt", "difr_detect", "difr_workspace_bytes"} <= set(names)
    for name in names:
        assert hasattr(L, name), name
    assert set(names) == set(difr.EXPORTS)


def test_host_only_entry_points():
    assert difr.difr_version() >= 100
    assert difr.difr_status_string(0) == "ok"
    assert "workspace" in difr.difr_status_string(-4)
    assert difr.difr_status_string(-7)
    # plan-derived sizes: one 32-byte record per (row, strip), a 256-byte tail, and per row (padded to 256 rows)
    # six floats of bounds, a counter and 64 eight-byte entries for the ids fp32 cannot decide
    per_row = 6 * 4 + 4 + 64 * 8
    nbytes = difr.difr_workspace_bytes(4096, 3072, 128256)
    assert nbytes > 0 and (nbytes - 256 - per_row * 4096) % (32 * 4096) == 0
    assert (difr.difr_workspace_bytes(4097, 3072, 128256) - 256 - per_row * (4096 + 256)) % (32 * (4096 + 256)) == 0
    assert difr.difr_workspace_bytes(4096, 3076, 128256) == 0  # d not a multiple of 8
    assert difr.difr_workspace_bytes(4096, 3072, 1) == 0
    assert difr.difr_workspace_bytes(0, 3072, 128256) == 0
    assert difr.difr_workspace_bytes(1 << 30, 64, (1 << 31) - 1) == 0  # more work units than 32-bit ids
    small = difr.difr_workspace_bytes(100, 64, 300)  # 100 rows pad to 256; 300 ids are two tiles: at most two strips
    assert small in (256 + per_row * 256 + 32 * 256 * s for s in (1, 2))


def test_bad_arguments_are_refused_on_the_host():
    """Everything the host can check is checked before the device is touched: these calls run without a GPU and
    never dereference the (fake) pointers."""
    import ctypes

    try:
        import torch

        if torch.cuda.is_available():
            # the pointers below are fake: where a device is present, a call that a later change no longer
            # refused on the host would reach it with them
            pytest.skip("host-only check: run it where no CUDA device is visible")
    except ImportError:
        pass
    L = difr.lib()
    p = ctypes.c_void_p(0x10000)  # non-null, 16-byte aligned, never read
    INVALID, SHAPE, OK = -1, -2, 0

    def out(**kw):
        c = difr._COut()
        c.sigma, c.eps, c.score = 0.3, 1e-12, 0x10000
        for k, v in kw.items():
            setattr(c, k, v)
        return c

    def score(fn, h=p, tokens=p, temperature=1.0, T=128, d=64, V=1000, o=None):
        o = o if o is not None else out()
        return getattr(L, fn)(h, p, tokens, p, p, temperature, T, d, V, ctypes.byref(o), None)

    for fn in ("difr_score_gm", "difr_score_ipt", "difr_score_both"):
        assert score(fn, h=None) == INVALID
        assert score(fn, tokens=None) == INVALID
        assert score(fn, T=-1) == INVALID
        assert score(fn, o=out(sigma=0.0)) == INVALID
        assert score(fn, o=out(eps=-1.0)) == INVALID
        assert score(fn, o=out(score=None)) == INVALID
        assert score(fn, temperature=-0.5) == INVALID
        assert score(fn, temperature=float("nan")) == INVALID
    assert score("difr_score_ipt", temperature=0.0) == INVALID   # the IPT sampler needs a distribution
    assert score("difr_score_both", temperature=0.0) == INVALID
    assert score("difr_score_both") == INVALID                   # no score_ipt / sigma_ipt given
    assert score("difr_score_gm", d=60, o=out()) == SHAPE        # d must be a multiple of 8
    assert score("difr_score_gm", V=1) == SHAPE
    assert score("difr_score_gm", T=0) == OK                     # nothing to do
    assert difr.difr_filtered_workspace_bytes(128, 60, 1000) == 0
    assert difr.difr_filtered_workspace_bytes(128, 64, 1000) > difr.difr_workspace_bytes(128, 64, 1000)

    def filtered(top_k, top_p, s, temperature=1.0, o=None):
        f = difr._CFilter(top_k, top_p, s)
        o = o if o is not None else out()
        return L.difr_score_gm_filtered(p, p, p, p, p, temperature, 128, 64, 1000, ctypes.byref(f), ctypes.byref(o), None)

    assert filtered(50, 0.95, 0) == INVALID and filtered(50, 0.95, 9) == INVALID   # 1 <= s <= 8
    assert filtered(50, 0.0, 1) == INVALID and filtered(50, 1.5, 1) == INVALID
    assert filtered(50, 0.95, 4, temperature=0.0) == INVALID
    assert filtered(-1, 0.95, 4) == INVALID
    f_rows = difr._CFilter(50, 0.95, 9, 0x10000, 0x10000)  # per-row values do not excuse a bad s
    assert L.difr_score_gm_filtered(p, p, p, p, p, 1.0, 128, 64, 1000, ctypes.byref(f_rows), ctypes.byref(out()), None) == INVALID

    f0 = difr._CFilter(0, 1.0, 1)
    o = out()
    assert L.difr_score_ipt_filtered(p, p, p, p, p, 1.0, 128, 64, 1000, ctypes.byref(f0), ctypes.byref(o), None) == INVALID

    taus = (ctypes.c_float * 5)(-1.0, -2.0, -3.0, -4.0, -5.0)
    adm = lambda n, sigma=0.3: L.difr_admissible(p, p, p, p, 1.0, 128, 64, 1000, p, p, p, p, sigma, 1e-12, taus, n, p,
                                                 None, p, 1 << 30, None, None)
    assert adm(0) == INVALID and adm(5) == INVALID and adm(2, sigma=0.0) == INVALID
    assert L.difr_exfiltratable_bits(p, p, 0, 1000, None, 1, 128, None, None, None) == INVALID  # R >= 1
    assert L.difr_exfiltratable_bits(None, p, 8, 1000, None, 1, 128, None, None, None) == INVALID
    assert L.difr_detect(None, -1.0, None, None, 0, None, 1, 128, None, None, None) == INVALID
    assert L.difr_detect(p, float("nan"), None, None, 0, None, 1, 128, None, None, None) == INVALID
    assert L.difr_expand_seeds(None, p, None, 1, None, 128, p, None) == INVALID
    assert L.difr_expand_seeds(p, None, None, 1, None, 128, p, None) == INVALID
    assert L.difr_expand_seeds(p, p, None, 1, None, 128, None, None) == INVALID
    assert L.difr_expand_seeds(p, p, None, 1, None, -1, p, None) == INVALID
    assert L.difr_expand_seeds(p, p, None, 1, None, 0, p, None) == OK


def test_header_is_plain_c():
    """include/difr.h is the boundary: it must compile as C99 and as C++ on its own."""
    import subprocess
    import tempfile

    src = '#include "difr.h"\nint main(void) { difr_out o; difr_filter f; (void)o; (void)f; return (int)sizeof(difr_seq_stats) - 16; }\n'
    with tempfile.TemporaryDirectory() as tmp:
        path = os.path.join(tmp, "t.c")
        open(path, "w").write(src)
        inc = os.path.join(ROOT, "include")
        subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-I", inc, path])
        subprocess.check_call(["g++", "-std=c++17", "-Wall", "-Werror", "-fsyntax-only", "-x", "c++", "-I", inc, path])


def test_binding_structs_have_the_headers_layout():
    """The ctypes mirrors of difr_out, difr_filter and difr_seq_stats must place every member where the C compiler
    places it: a C program prints sizeof and offsetof for each, the binding must agree."""
    import ctypes
    import subprocess
    import tempfile

    structs = {"difr_out": difr._COut, "difr_filter": difr._CFilter}
    lines = []
    for cname, cls in structs.items():
        lines.append(f'printf("{cname} %zu\\n", sizeof({cname}));')
        for field, _ in cls._fields_:
            lines.append(f'printf("{cname}.{field} %zu\\n", offsetof({cname}, {field}));')
    src = ('#include <stddef.h>\n#include <stdio.h>\n#include "difr.h"\nint main(void) {\n' + "\n".join(lines)
           + '\nprintf("difr_seq_stats %zu\\n", sizeof(difr_seq_stats));\nreturn 0;\n}\n')
    with tempfile.TemporaryDirectory() as tmp:
        c_path, exe = os.path.join(tmp, "layout.c"), os.path.join(tmp, "layout")
        open(c_path, "w").write(src)
        subprocess.check_call(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), "-o", exe, c_path])
        out = subprocess.check_output([exe], text=True)
    got = dict(line.split() for line in out.splitlines())
    for cname, cls in structs.items():
        assert int(got[cname]) == ctypes.sizeof(cls), cname
        for field, _ in cls._fields_:
            assert int(got[f"{cname}.{field}"]) == getattr(cls, field).offset, (cname, field)
    assert int(got["difr_seq_stats"]) == 16


def test_planning_is_remembered():
    """The work plan of a shape is computed once (small problems simulate their schedule for a few dozen strip
    counts, about a millisecond each time) and then looked up: a thousand repeated size queries take a few
    milliseconds in all, and an explicit override of the planner takes effect at once and is undone at once."""
    import time

    shape = (16384, 4096, 128256)
    first = difr.difr_workspace_bytes(*shape)
    t0 = time.perf_counter()
    for _ in range(1000):
        assert difr.difr_workspace_bytes(*shape) == first
    assert time.perf_counter() - t0 < 0.02  # 20 us per call, most of it the ctypes call itself
    # llama3b-sized problems take the slow planning path (few rounds of work units)
    t0 = time.perf_counter()
    for _ in range(200):
        difr.difr_workspace_bytes(4096, 3072, 128256)
    assert time.perf_counter() - t0 < 0.02
    try:
        difr.difr_debug_plan_override(7, 0, 0)
        T_pad = 16384
        assert difr.difr_workspace_bytes(*shape) == 7 * 32 * T_pad + 256 + (6 * 4 + 4 + 64 * 8) * T_pad
    finally:
        difr.difr_debug_plan_override()
    assert difr.difr_workspace_bytes(*shape) == first
    with pytest.raises(difr.DifrError):
        difr.difr_debug_plan_override(-1)


def test_a_well_formed_call_without_a_device_reports_a_cuda_error():
    """The host-side failure path: every argument is acceptable, but the CUDA runtime cannot give a device
    (none is visible here), so the call returns DIFR_ERR_CUDA before anything is launched.  Runs in a child
    process with the devices hidden, so it means the same on a machine that has GPUs."""
    import subprocess
    import sys

    code = r'''
import ctypes, sys
sys.path.insert(0, %r)
import paper_2511_02620_b200 as difr
L = difr.lib()
p = ctypes.c_void_p(0x10000)
o = difr._COut()
o.sigma, o.eps, o.score, o.workspace, o.workspace_bytes = 0.3, 1e-12, 0x10000, 0x10000, 1 << 40
rc = [L.difr_score_gm(p, p, p, p, p, 1.0, 128, 64, 1000, ctypes.byref(o), None),
      L.difr_score_ipt(p, p, p, p, p, 1.0, 128, 64, 1000, ctypes.byref(o), None),
      L.difr_score_gm_static(p, p, p, p, p, 1.0, 128, 64, 1000, ctypes.byref(o), None),
      L.difr_logits(p, p, 128, 64, 1000, p, None, None)]
print(rc, difr.difr_status_string(rc[0]))
sys.exit(0 if rc == [-5, -5, -5, -5] else 1)
''' % ROOT
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "CUDA call failed" in r.stdout
