"""Writes tests/golden/oracle_freeze.txt from the CPU oracle alone.

The values are not the paper's (it prints no table row and no word/point
pair); they freeze the readings listed in oracle/tetra_oracle.h so that a later
change of a tie-break or a bit position cannot pass unnoticed.
Run:  python tests/golden/make_golden.py
"""
import hashlib
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402


def main():
    o = oracle.get()
    blob = o.table_blob()
    out = ["# written by tests/golden/make_golden.py from oracle/ only",
           "# sha256 <name> <from> <to> <digest>   over the table blob of Sec. 3.4"]
    for name, lo, hi in (("rows", 0, 16384), ("trellis", 16384, 18688), ("integers", 0, 18688), ("all", 0, 18816)):
        out.append("sha256 %s %d %d %s" % (name, lo, hi, hashlib.sha256(blob[lo:hi]).hexdigest()))
    out.append("# decode <word hex> <m> <g> <24 coordinates>")
    for w in (0x000000000001, 0xFFFFFFFFFFFF, 0x123456789ABC, 0x800000000000, 0x5A5A5A5A5A5A, 0x0F1E2D3C4B5A):
        y, m, g = o.decode_word(w)
        out.append("decode %012x %d %d %s" % (w, m, g, " ".join(str(int(v)) for v in y)))
    with open(os.path.join(HERE, "oracle_freeze.txt"), "w") as f:
        f.write("\n".join(out) + "\n")


if __name__ == "__main__":
    main()
