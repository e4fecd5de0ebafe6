"""Writes tests/golden/config1_digests.txt from the CPU oracle alone.

Run from the repository root:  python tests/golden/make_config1_digests.py
Each line: tensor name, sum, sum of absolute values, first and last element in the
flatten order [Tq, H, d] (O, dQ, dK, dV) or [H, Tq] (LSE).  Inputs: configuration 1 from
the canonical seeded generator, loss = sum(O * dO).
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import zl_workloads as W            # noqa: E402
from oracle import attention as A   # noqa: E402


def main():
    p = W.config(1)
    T = {t: np.stack([W.head_tensor_for(p, t, h).astype(np.float64) for h in range(p.n_heads)], 1)
         for t in ("Q", "K", "V", "dO")}
    out = A.placement_fwd(p, T["Q"], T["K"], T["V"])
    g = A.placement_bwd(p, T["Q"], T["K"], T["V"], T["dO"])
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config1_digests.txt")
    with open(path, "w") as f:
        f.write("# configuration 1, fp64 oracle digests: name sum sum_abs first last\n")
        f.write("# written by tests/golden/make_config1_digests.py (calls only oracle/)\n")
        for name, x in (("O", out["O"]), ("LSE", out["LSE"]), ("dQ", g["dQ"]), ("dK", g["dK"]),
                        ("dV", g["dV"])):
            f.write(f"{name} {x.sum():.12e} {np.abs(x).sum():.12e} {x.ravel()[0]:.12e} {x.ravel()[-1]:.12e}\n")
    print(open(path).read())


if __name__ == "__main__":
    main()
