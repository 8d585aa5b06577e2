"""Writes tests/golden/micro_prefill.txt: the oracle's results on a micro workload.

Calls only the oracle.  Inputs come from NumPy's PCG64 stream (stable across
platforms), drawn in the order below; the test regenerates them the same way.
Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import structkv_oracle as O  # noqa: E402

SHAPE = dict(L=5, H=4, Hkv=2, w=4, d=8, N=96, kv_budget=12, struct_budget=24)
TEMPS = (1.0, 0.8, 1.6, 0.6, 1.2)


def micro_inputs():
    s = SHAPE
    rng = np.random.Generator(np.random.PCG64(20260406746))
    layers = []
    for l in range(s["L"]):
        q = rng.standard_normal((s["H"], s["w"], s["d"]))
        k = rng.standard_normal((s["Hkv"], s["N"], s["d"]))
        q = q.astype(np.float32).astype(np.float64)
        k = k.astype(np.float32).astype(np.float64)
        layers.append((q, k, 1.0 / (np.sqrt(s["d"]) * TEMPS[l])))
    return layers


def main():
    s = SHAPE
    r = O.prefill(micro_inputs(), s["w"], s["kv_budget"], s["struct_budget"])
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "micro_prefill.txt")
    with open(out, "w") as f:
        f.write("# Oracle results on the micro workload of tests/golden/make_golden.py "
                "(Algorithm 1 skeleton: Eq. 2-4, 5, 6, 8, 9, 10, 13).\n")
        f.write("pivot %d\n" % r["pivot"])
        for l in range(s["L"]):
            f.write("metrics %d %.17g %.17g %.17g\n" % (l, *r["metrics"][l]))
        f.write("C " + " ".join("%.17g" % x for x in r["C"]) + "\n")
        f.write("i_struct " + " ".join(str(int(x)) for x in r["i_struct"]) + "\n")
        for l in range(s["L"]):
            f.write("i_kv %d " % l + " ".join(str(int(x)) for x in r["i_kv"][l]) + "\n")
    print("wrote", out)


if __name__ == "__main__":
    main()
