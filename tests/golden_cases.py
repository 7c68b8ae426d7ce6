"""Reader of ``tests/golden/quadratic_fitness_order.txt``: the hand-worked
cases that fix the summation order and the term rounding of the quadratic
fitness.  Holds no arithmetic: it only turns the sparse text into dense fp32
arrays (w = 1, tvec = 0, dvec = 0 where a case lists nothing)."""
import os

import numpy as np

from conftest import GOLDEN

FITNESS_ORDER = os.path.join(GOLDEN, "quadratic_fitness_order.txt")


def _number(text):
    return float.fromhex(text) if "x" in text.lower() else float(text)


def fitness_order_cases(path=FITNESS_ORDER):
    """[(name, w[N], dvec[N], tvec[N], expected fp32)] in file order."""
    cases, cur = [], None
    with open(path) as fh:
        for raw in fh:
            line = raw.split("#", 1)[0].strip()
            if not line:
                continue
            key, *rest = line.split()
            if key == "case":
                cur = {"name": rest[0], "w": {}, "d": {}, "t": {}}
                cases.append(cur)
            elif key == "N":
                cur["N"] = int(rest[0])
            elif key in ("w", "d", "t"):
                for item in rest:
                    idx, val = item.split(":")
                    cur[key][int(idx)] = _number(val)
            elif key == "expect":
                cur["expect"] = np.float32(_number(rest[0]))
            else:
                raise ValueError(f"{path}: unknown line {raw!r}")
    out = []
    for c in cases:
        n = c["N"]
        w = np.ones(n, np.float32)
        d = np.zeros(n, np.float32)
        t = np.zeros(n, np.float32)
        for arr, sparse in ((w, c["w"]), (d, c["d"]), (t, c["t"])):
            for idx, val in sparse.items():
                assert 0 <= idx < n and float(np.float32(val)) == val, (c["name"], idx, val)
                arr[idx] = np.float32(val)
        out.append((c["name"], w, d, t, c["expect"]))
    return out
