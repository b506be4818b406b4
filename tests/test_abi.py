"""The C-ABI library loads without a GPU and exports every function that
include/difr.h declares; host-only entry points behave."""
import os
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
    # plan-derived sizes: one 32-byte record per (row, strip) and four floats per row, rows padded to 256,
    # plus a 256-byte tail
    nbytes = difr.difr_workspace_bytes(4096, 3072, 128256)
    assert nbytes > 0 and (nbytes - 256 - 16 * 4096) % (32 * 4096) == 0
    assert (difr.difr_workspace_bytes(4097, 3072, 128256) - 256 - 16 * (4096 + 256)) % (32 * (4096 + 256)) == 0
    assert difr.difr_workspace_bytes(4096, 3076, 128256) == 0  # d not a multiple of 8
    assert difr.difr_workspace_bytes(4096, 3072, 1) == 0
    assert difr.difr_workspace_bytes(0, 3072, 128256) == 0
    small = difr.difr_workspace_bytes(100, 64, 300)  # 100 rows pad to 256; 300 ids are two tiles: at most two strips
    assert small in (256 + 16 * 256 + 32 * 256 * s for s in (1, 2))
