"""Reader for the text fixtures under tests/golden/ (one float per line, '#' comments)."""
import os

import numpy as np

GOLDEN_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def load(name, shape=None):
    vals = []
    with open(os.path.join(GOLDEN_DIR, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                vals.append(float(line))
    arr = np.asarray(vals, dtype=np.float64)
    return arr if shape is None else arr.reshape(shape)
