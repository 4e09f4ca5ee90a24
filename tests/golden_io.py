"""Reader for the small text fixtures under tests/golden/ ("name v v ; v v" rows)."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, _, rest = line.partition(" ")
            rows = [[float(v) for v in row.split()] for row in rest.split(";")]
            arr = np.array(rows, dtype=np.float64)
            out[key] = arr[0] if arr.shape[0] == 1 else arr
    return out
