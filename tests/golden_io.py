"""Reader for the small text fixtures under tests/golden/."""
import os

import numpy as np

_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_fixture(name):
    out = {}
    with open(os.path.join(_DIR, name)) as f:
        lines = [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]
    i = 0
    while i < len(lines):
        tok = lines[i].split()
        key = tok[0]
        if key == "table":
            r, c = int(tok[1]), int(tok[2])
            rows = [[float(x) for x in lines[i + 1 + k].split()] for k in range(r)]
            out["table"] = np.array(rows, dtype=np.float64).reshape(r, c)
            i += 1 + r
            continue
        out[key] = np.array([float(x) for x in tok[1:]], dtype=np.float64)
        i += 1
    return out
