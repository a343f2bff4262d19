"""Reader for the small text fixtures under tests/golden/."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_blocks(name):
    """Parse `name rows cols` blocks into a dict of float64 arrays."""
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        lines = [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]
    i = 0
    while i < len(lines):
        key, r, c = lines[i].split()
        r, c = int(r), int(c)
        rows = [[float(v) for v in lines[i + 1 + k].split()] for k in range(r)]
        a = np.array(rows, dtype=np.float64)
        assert a.shape == (r, c), (name, key)
        out[key] = a
        i += 1 + r
    return out


def read_shapes(name):
    """Parse `layer layers rows cols` lines and the `parameters n` line."""
    shapes, params = [], None
    with open(os.path.join(GOLDEN, name)) as f:
        for ln in f:
            ln = ln.strip()
            if not ln or ln.startswith("#"):
                continue
            parts = ln.split()
            if parts[0] == "parameters":
                params = int(parts[1])
            else:
                shapes.append((parts[0], int(parts[1]), int(parts[2]), int(parts[3])))
    return shapes, params
