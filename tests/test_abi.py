"""The C-ABI library loads without a GPU and exports every symbol that include/mfet.h declares."""
import ctypes
import os
import re

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "mfet.h")).read()
    return re.findall(r"MFET_API\s+[\w\s\*]+?\b(mfet_\w+)\s*\(", text)


def test_library_exports_every_declared_symbol():
    from paper_2508_05700_b200 import build, mfet
    build.build()
    names = _declared()
    assert len(names) >= 18 and len(set(names)) == len(names)
    lib = ctypes.CDLL(mfet.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(names) == sorted(mfet.EXPORTS)


def test_host_only_entry_points():
    from paper_2508_05700_b200 import mfet
    assert mfet.row_bytes(32, mfet.F32) == 128 and mfet.row_bytes(64, mfet.F16) == 128
    assert mfet.row_bytes(128, mfet.BF16) == 256 and mfet.row_bytes(64, mfet.INT4) == 48
    assert mfet.row_bytes(8, 77) == 0
    assert mfet.status_string(0) == "ok" and "unknown" in mfet.status_string(-99)
    for code in range(-7, 0):
        assert mfet.status_string(code) not in ("ok", "unknown status")


def test_struct_layouts_match_the_header():
    from paper_2508_05700_b200 import mfet
    assert ctypes.sizeof(mfet.TableDesc) == 48
    assert ctypes.sizeof(mfet.BatchShape) == 32
    assert mfet.TableDesc.hash_seed.offset == 32 and mfet.BatchShape.slot_feature.offset == 16
