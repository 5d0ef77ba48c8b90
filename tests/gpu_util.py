"""Helpers for the GPU parity tests: move seeded workloads to the device and call the C ABI through the binding."""
import numpy as np
import torch

from paper_2602_11812_b200 import binding as egtp
from paper_2602_11812_b200 import inputs as gen
from paper_2602_11812_b200.device import DeviceHead, dev_tensor, host_tensor  # noqa: F401


def run_egtp(ctx, wl: gen.EgtpWorkload, W_dev=None, hidden_dev=None, head_dev=None, offsets=None, want_phat=False):
    """egtp_predict on a workload; returns numpy float64 / int32 arrays and the device status."""
    hidden = dev_tensor(wl.hidden, wl.dtype) if hidden_dev is None else hidden_dev
    W = dev_tensor(wl.W, wl.dtype) if W_dev is None else W_dev
    head = DeviceHead(wl.head, wl.dtype) if head_dev is None else head_dev
    off_np = wl.offsets if offsets is None else np.asarray(offsets, dtype=np.int32)
    off = torch.from_numpy(off_np).cuda()
    B, T, d = off_np.shape[0] - 1, hidden.shape[0], hidden.shape[1]
    f = dict(device="cuda", dtype=torch.float32)
    out = dict(H=torch.full((T,), float("nan"), **f), weights=torch.full((T,), float("nan"), **f),
               seg_id=torch.full((T,), -7, device="cuda", dtype=torch.int32),
               pooled=torch.full((B, d), float("nan"), **f), state_m=torch.full((B,), float("nan"), **f),
               state_s=torch.full((B,), float("nan"), **f), yhat=torch.full((B,), float("nan"), **f),
               phat=torch.full((B, head.d_out), float("nan"), **f) if want_phat else None)
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    lm = egtp.make_lm_head(W)
    egtp.egtp_predict(ctx, lm, head.c, hidden, off, B, T, wl.alpha, H_out=out["H"], weights_out=out["weights"],
                      seg_id_out=out["seg_id"], pooled_out=out["pooled"], state_m_out=out["state_m"],
                      state_s_out=out["state_s"], yhat_out=out["yhat"], phat_out=out["phat"], status_dev=status)
    torch.cuda.synchronize()
    res = {k: (None if v is None else v.cpu().numpy()) for k, v in out.items()}
    for k in ("H", "weights", "pooled", "state_m", "state_s", "yhat"):
        res[k] = res[k].astype(np.float64)
    res["status"] = int(status.item())
    return res


# Tolerances (the bar stated for this path): entropy 1e-3 relative, pooled 2e-3 relative, length 0.5 absolute
# (and 1e-3 relative, so that a prediction of a fraction of a token is checked as strictly as one of hundreds).
def assert_entropy_close(H, H_ref):
    err = np.abs(H - H_ref)
    bound = 1e-3 * np.abs(H_ref) + 1e-5
    assert np.all(err <= bound), f"entropy: max err {err.max():.3e}, worst ratio {(err / bound).max():.3f}"


def assert_pooled_close(p, p_ref):
    for b in range(p_ref.shape[0]):
        scale = np.abs(p_ref[b]).max()
        dmax = np.abs(p[b] - p_ref[b]).max()
        assert dmax <= 2e-3 * scale + 1e-30, f"pooled row {b}: max err {dmax:.3e} vs scale {scale:.3e}"
        n_ref = np.linalg.norm(p_ref[b])
        assert np.linalg.norm(p[b] - p_ref[b]) <= 2e-3 * n_ref + 1e-30, f"pooled row {b}: l2 error too large"


def assert_length_close(y, y_ref):
    """Half a token absolute (the stated bar) and, so that the check can fail whatever the size of the
    prediction, 1e-3 relative with a small absolute floor."""
    y, y_ref = np.asarray(y, dtype=np.float64), np.asarray(y_ref, dtype=np.float64)
    err = np.abs(y - y_ref)
    assert np.all(err <= 0.5), f"predicted length: max abs err {err.max():.3e}"
    bound = 1e-3 * np.abs(y_ref) + 1e-4
    assert np.all(err <= bound), f"predicted length: max err {err.max():.3e}, worst ratio {(err / bound).max():.3f}"
