"""GPU parity for the paper's pooling comparators (Table 3): average, max and last-token pooling, then the head."""
import numpy as np
import pytest
import torch

from oracle import egtp_oracle as orc
from paper_2602_11812_b200 import binding as egtp
from paper_2602_11812_b200 import inputs as gen
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

MODES = [(egtp.EGTP_POOL_MEAN, orc.POOL_MEAN), (egtp.EGTP_POOL_MAX, orc.POOL_MAX), (egtp.EGTP_POOL_LAST, orc.POOL_LAST)]


def _run(ctx, wl, mode, offsets=None):
    hidden = gu.dev_tensor(wl.hidden, wl.dtype)
    off_np = wl.offsets if offsets is None else np.asarray(offsets, np.int32)
    off = torch.from_numpy(off_np).cuda()
    head = gu.DeviceHead(wl.head, wl.dtype)
    B = off_np.shape[0] - 1
    pooled = torch.full((B, wl.d), float("nan"), device="cuda")
    y = torch.full((B,), float("nan"), device="cuda")
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    egtp.egtp_pool_baseline(ctx, head.c, hidden, off, B, wl.T, mode, pooled_out=pooled, yhat_out=y, status_dev=status)
    torch.cuda.synchronize()
    return pooled.cpu().numpy().astype(np.float64), y.cpu().numpy().astype(np.float64), int(status.item())


@pytest.mark.parametrize("gpu_mode,orc_mode", MODES)
def test_pooling_comparators_match_oracle(gpu_mode, orc_mode):
    ctx = egtp.egtp_create(0, max_tokens=16384, max_batch=64, max_d=2048, max_V=1024)
    try:
        # long-tailed ragged batch (prompts spanning many 64-token chunks) and the tiny fp32 configuration
        for wl in (gen.config_long(B=24, d=1280, V=64, m_h=96, max_len=1500), gen.config_tiny()):
            pooled, y, st = _run(ctx, wl, gpu_mode)
            ref = orc.baseline_predict(wl.hidden, wl.offsets, wl.head, orc_mode)
            assert st == 0
            if orc_mode == orc.POOL_MEAN:
                gu.assert_pooled_close(pooled, ref["pooled"])
            else:
                assert np.array_equal(pooled, ref["pooled"])          # max and last-token pooling select values: exact
            gu.assert_length_close(y, ref["yhat"])
        # empty prompts, tokens outside every prompt, chunk-edge boundaries
        rng = np.random.default_rng(4)
        off = np.array([5, 5, 64, 128, 129, 129, 321, 400], np.int32)
        hidden = gen.round_to_bf16(rng.standard_normal((410, 256)).astype(np.float32))
        wl = gen.EgtpWorkload("edges", "bf16", hidden, off, np.zeros((16, 256), np.float32), gen.make_head(2, 256, 32, 1, "bf16"))
        pooled, y, st = _run(ctx, wl, gpu_mode)
        ref = orc.baseline_predict(hidden, off, wl.head, orc_mode)
        assert st == 0
        gu.assert_pooled_close(pooled[[1, 2, 3, 5, 6]], ref["pooled"][[1, 2, 3, 5, 6]])
        assert np.all(pooled[[0, 4]] == 0)
        gu.assert_length_close(y, ref["yhat"])
        bad = off.copy(); bad[3] = 10
        assert _run(ctx, wl, gpu_mode, offsets=bad)[2] == egtp.EGTP_ERR_BAD_OFFSETS
    finally:
        egtp.egtp_destroy(ctx)
