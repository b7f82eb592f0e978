"""Writes tests/golden/smallest_uniform.txt: positions (seed, step, worker, element)
whose rounding uniform takes its smallest value 2^-24 (all 23 Philox bits set),
found by scanning the CPU oracle's stream.  Calls only the oracle.
Usage: python tests/golden/make_smallest_uniform.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402

SEED = 2107
n = 1 << 22
lay = oracle.Layout([n], 4096)
g = np.ones((1, n), np.float32)
norms = oracle.bucket_norms(lay, g)
found = []
for step in range(64):
    _, _, u = oracle.quantize(lay, g, norms, 4, SEED, step, want_frac_u=True)
    for j in np.nonzero(u[0] == np.float32(2.0 ** -24))[0]:
        if j % 32 != 31:
            found.append((SEED, step, 0, int(j)))
    if len(found) >= 3:
        break
with open(os.path.join(ROOT, "tests", "golden", "smallest_uniform.txt"), "w") as fh:
    fh.write("# seed step worker element : positions of the oracle's Philox stream whose rounding\n"
             "# uniform is 2^-24, its smallest value (written by make_smallest_uniform.py from the\n"
             "# oracle alone)\n")
    for row in found:
        fh.write("%d %d %d %d\n" % row)
print(found)
