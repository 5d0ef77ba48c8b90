"""Writes tests/golden/egtp_tiny_*.txt: the oracle's outputs on the tiny EGTP configuration.

Run from the repository root:  python tests/golden/make_golden.py
Calls only the CPU oracle and the seeded input generators; never the CUDA path.
Each file is plain text, one value per line (repr of a float64), with a '#' header.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import egtp_oracle as orc                      # noqa: E402
from paper_2602_11812_b200 import inputs as gen            # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))


def write(name, arr, header):
    with open(os.path.join(HERE, name), "w") as f:
        f.write(f"# {header}\n# shape {list(arr.shape)}\n")
        for v in np.asarray(arr, dtype=np.float64).ravel():
            f.write(repr(float(v)) + "\n")


def main():
    wl = gen.config_tiny()
    out = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, wl.alpha)
    src = "oracle.egtp_predict on inputs.config_tiny() (Eq. 2-4 and the scalar head)"
    write("egtp_tiny_H.txt", out["H"], "token entropies, " + src)
    write("egtp_tiny_pooled.txt", out["pooled"], "pooled vectors, " + src)
    write("egtp_tiny_yhat.txt", out["yhat"], "predicted lengths, " + src)
    wb = gen.config_tiny(gen.HEAD_BINS)
    outb = orc.egtp_predict(wb.hidden, wb.offsets, wb.W, wb.head, wb.alpha, H=out["H"])
    write("egtp_tiny_bins_yhat.txt", outb["yhat"],
          "predicted lengths with the K = 20 bin head (Eq. 6), oracle.egtp_predict on inputs.config_tiny(HEAD_BINS)")


if __name__ == "__main__":
    main()
