"""Writes co3_inputs/scale_table.json: the multiplier s*(beta) minimising the expected squared
conversion error (Sec. IV-A (i), Eq. (exp bias)) for a unit-scale generalized-normal input, per
format and shape value.  Calls only the CPU oracle.  Run from the repository root:

    python -m co3_inputs.make_scale_table
"""
import json
import os

import numpy as np

from oracle import bias

FORMATS = ((2, 1), (3, 0), (4, 3), (5, 2))
BETAS = [round(0.3 + 0.05 * i, 2) for i in range(35)]  # 0.30 .. 2.00


def main() -> None:
    table = {"_doc": "s*(beta) = argmin_s E|Q(s G)/s - G|^2, G ~ GenNorm(0, 1, beta); "
                     "written by co3_inputs/make_scale_table.py from the CPU oracle's level set",
             "betas": BETAS, "formats": {}}
    for (e, m) in FORMATS:
        row = []
        for b in BETAS:
            s, _ = bias.optimal_scale(e, m, b)
            row.append(float(np.float32(s)))
        table["formats"]["%d,%d" % (e, m)] = row
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "scale_table.json")
    with open(path, "w") as fh:
        json.dump(table, fh, indent=1)
        fh.write("\n")


if __name__ == "__main__":
    main()
