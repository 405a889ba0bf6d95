"""Writes tests/golden/default_code_table.txt from the CPU oracle alone.

The 16 levels are this project's built-in default for the code-table format
(the paper, Sec. 3.2, names a 4-bit normal-quantile type but prints no values).
Run:  python tests/golden/gen_default_code_table.py
"""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
import oracle  # noqa: E402

here = os.path.dirname(os.path.abspath(__file__))
t = oracle.default_code_table()
with open(os.path.join(here, "default_code_table.txt"), "w") as f:
    f.write("# default 16-level table, float32 hex; closed form: ppf(1/2+j/17)/ppf(1/2+8/17), j=0..8 and\n")
    f.write("# -ppf(1/2+j/15)/ppf(1/2+7/15), j=1..7 (standard normal quantile), ascending.\n")
    f.write("# Source: written by gen_default_code_table.py from oracle/ only (paper Sec. 3.2 prints no table).\n")
    for x in t:
        f.write(float(x).hex() + "\n")
