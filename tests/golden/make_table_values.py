"""Writes tests/golden/table_values.txt: frozen entries of the synthetic table-value generator.

Calls only the CPU oracle. Run from the repository root:  python tests/golden/make_table_values.py
The frozen values guard the generator against silent change; they are also compared with the
values that the GPU fill kernel writes.
"""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
import oracle as orc  # noqa: E402

CASES = [
    # key, mode, dim, dtype, row, column
    (1, orc.VAL_NORMAL, 32, orc.F32, 0, 0),
    (1, orc.VAL_NORMAL, 32, orc.F32, 99_999, 31),
    (0x9D2C5680A1B2C3D5, orc.VAL_NORMAL, 64, orc.F16, 9_999_999, 17),
    (0x9D2C5680A1B2C3D5, orc.VAL_NORMAL, 64, orc.BF16, 49_999_999, 63),
    (0xFFFFFFFFFFFFFFFF, orc.VAL_NORMAL, 128, orc.BF16, 999_999_999, 127),
    (12345678901234567, orc.VAL_NORMAL, 64, orc.F16, 123_456_789, 5),
    (7, orc.VAL_GRID, 64, orc.BF16, 3, 2),
    (7, orc.VAL_GRID, 32, orc.F16, 1_000_003, 30),
    (7, orc.VAL_GRID, 32, orc.F32, 1_000_003, 30),
]

if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "table_values.txt")
    with open(out, "w") as fh:
        fh.write("# Frozen entries of the synthetic table-value generator (not paper values: the paper's tables\n"
                 "# are private pretrained weights). Written by make_table_values.py from the CPU oracle.\n"
                 "# key mode dim dtype row column stored_bits\n")
        for key, mode, dim, dtype, r, d in CASES:
            bits = orc.table_value_bits(key, mode, dim, dtype, r, d)
            fh.write("0x%016X %d %d %d %d %d 0x%08X\n" % (key, mode, dim, dtype, r, d, bits))
    print("wrote", out)
