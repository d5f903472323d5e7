"""Writes tests/golden/config1_oracle.txt: a few numbers of the fp64 oracle on benchmark config 1 (the tiny fp32
block, seed 0), for detecting an unintended change of the oracle's arithmetic or of the input recipe.

The paper prints no number that could serve as a fixture (no worked example, no intermediate value), so the stored
values are the oracle's own: this file calls only `oracle/`, the seeded input generators and the test harness's
prefill helper; nothing of the CUDA path.  A deliberate change of the oracle (which its commit message has to
justify by the passage of the paper it follows) is followed by running this script again:

    python tests/golden/make_oracle_fixture.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_39329_b200 import inputs as gen      # noqa: E402
from tests import helpers as H                       # noqa: E402


def values():
    cfg = gen.benchmark_config(1)
    lay = H.make_problem(cfg)
    x = lay["x0"]
    o = H.run_oracle(cfg, lay, x, x, [0, cfg.N], cfg.lam0)
    dW = o["dW"]
    return [
        ("lambda (Eq. 7)", float(o["lam"])),
        ("tr(S_H)", float(o["tr"])),
        ("||T||_F^2 (Eq. 5)", float(o["T_fro2"])),
        ("||dW||_F (Eq. 8)", float(np.sqrt(np.sum(dW * dW)))),
        ("dW[0][0]", float(dW[0, 0])),
        ("dW[17][101]", float(dW[17, 101])),
        ("dW[255][255]", float(dW[-1, -1])),
        ("sum of xF_next", float(np.sum(o["xF_next"]))),
        ("sum of xC_next", float(np.sum(o["xC_next"]))),
    ]


def main():
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config1_oracle.txt")
    with open(path, "w") as f:
        f.write("# fp64 oracle on benchmark config 1 (tiny fp32 block, seed 0); written by make_oracle_fixture.py\n")
        f.write("# quantity (equation of the paper it belongs to) <tab> value\n")
        for name, v in values():
            f.write("%s\t%.17g\n" % (name, v))
    print("wrote", path)


if __name__ == "__main__":
    main()
