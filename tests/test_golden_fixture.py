"""The stored tiny-configuration values are what the oracle produces today (they were written by it)."""
import numpy as np

from oracle import egtp_oracle as orc
from paper_2602_11812_b200 import inputs as gen
from tests.golden_io import load


def test_golden_matches_oracle():
    wl = gen.config_tiny()
    out = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, wl.alpha)
    assert np.allclose(out["H"], load("egtp_tiny_H.txt"), rtol=0, atol=1e-12)
    assert np.allclose(out["pooled"], load("egtp_tiny_pooled.txt", (4, 256)), rtol=0, atol=1e-12)
    assert np.allclose(out["yhat"], load("egtp_tiny_yhat.txt"), rtol=0, atol=1e-12)
    wb = gen.config_tiny(gen.HEAD_BINS)
    outb = orc.egtp_predict(wb.hidden, wb.offsets, wb.W, wb.head, wb.alpha, H=out["H"])
    assert np.allclose(outb["yhat"], load("egtp_tiny_bins_yhat.txt"), rtol=0, atol=1e-9)
    # Gaussian-logit plausibility: logits of this configuration have unit variance, so H ~ ln 4096 - 1/2
    assert abs(out["H"].mean() - (np.log(4096) - 0.5)) < 0.05
