"""GPU parity for the entropy-from-logits path (Eq. 2 on logits already in memory) and plp_step_from_logits."""
import math

import numpy as np
import pytest
import torch

from oracle import egtp_oracle as orc
from paper_2602_11812_b200 import binding as egtp
from paper_2602_11812_b200 import inputs as gen
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = egtp.egtp_create(0, max_tokens=4096, max_batch=512, max_d=512, max_V=160000)
    yield c
    egtp.egtp_destroy(c)


def _entropy(ctx, logits_dev, V):
    H = torch.full((logits_dev.shape[0],), float("nan"), device="cuda")
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    egtp.egtp_entropy_from_logits(ctx, logits_dev, H, V=V, status_dev=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return H.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("dtype,rows,V", [("bf16", 37, 5003), ("f32", 5, 777), ("bf16", 256, 151936), ("bf16", 3, 7),
                                          ("f32", 1030, 4096)])
def test_entropy_from_logits_matches_oracle(ctx, dtype, rows, V):
    rng = np.random.default_rng(rows + V)
    ld = (V + 7) // 8 * 8 + 8                       # padded rows: the row tail must be ignored
    x = gen._maybe_round((rng.standard_normal((rows, ld)) * 3.0).astype(np.float32), dtype)
    x[:, V:] = 50.0                                 # poison beyond V
    dev = gu.dev_tensor(x, dtype)[:, :V]
    H = _entropy(ctx, dev, V)
    gu.assert_entropy_close(H, orc.entropy_from_logits(x[:, :V].astype(np.float64)))


def test_entropy_from_logits_closed_forms(ctx):
    V = 151936
    x = np.zeros((3, V), np.float32)
    x[1, 12345] = 60.0                              # one-hot limit
    x[2, :100] = 7.0                                # two-level: H = ln Z - k a e^a / Z
    H = _entropy(ctx, gu.dev_tensor(x, "bf16"), V)
    Z = 100 * math.exp(7.0) + V - 100
    assert abs(H[0] - math.log(V)) < 1e-4 * math.log(V)
    assert abs(H[1]) < 1e-5
    assert abs(H[2] - (math.log(Z) - 100 * 7.0 * math.exp(7.0) / Z)) < 1e-3 * H[2]
    assert egtp.egtp_entropy_from_logits(ctx, gu.dev_tensor(x, "bf16"), torch.empty(3, device="cuda"), rows=10**6,
                                         check=False) == egtp.EGTP_ERR_CAPACITY


@pytest.mark.parametrize("bind,slots,m_h", [(False, 130, 64), (True, 130, 64), (True, 300, 264)])
def test_plp_step_from_logits_matches_oracle_and_plp_step(ctx, bind, slots, m_h):
    # bind: the state is bound to its head, so W1 h' comes from a launch of the LM-head kernel over the head columns
    # alone (K split over the SMs; 264 hidden units = two column tiles) and one kernel finishes the step
    wl = gen.config_plp_decode(slots=slots, steps=5, d=256, V=9000, m_h=m_h, mu=1.0, sigma=0.6)
    steps, slots, d = wl.steps, wl.slots, wl.d
    W = gu.dev_tensor(wl.W, "bf16")
    head = gu.DeviceHead(wl.head, "bf16")
    hs = gu.dev_tensor(wl.hidden_steps.reshape(-1, d), "bf16").reshape(steps, slots, d)
    reset = torch.from_numpy(wl.reset_src).cuda()
    lm = egtp.make_lm_head(W)
    st_a = egtp.plp_state_create(ctx, slots, d)
    st_b = egtp.plp_state_create(ctx, slots, d)
    if bind:
        egtp.plp_state_bind_head(st_a, head.c)
    f = dict(device="cuda", dtype=torch.float32)
    Ha, za, ya = torch.zeros(steps, slots, **f), torch.zeros(steps, slots, d, **f), torch.zeros(steps, slots, **f)
    Hb, zb, yb = torch.zeros(steps, slots, **f), torch.zeros(steps, slots, d, **f), torch.zeros(steps, slots, **f)
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    logits_all = []
    n0 = egtp.egtp_launch_count(ctx)
    for t in range(steps):
        logits = (hs[t].float() @ W.float().T).to(torch.bfloat16)       # what a serving engine would hold
        logits_all.append(logits.float().cpu().numpy())
        egtp.plp_step_from_logits(ctx, st_a, logits, head.c, hs[t], reset_src=reset[t], Hstep_out=Ha[t], z_out=za[t],
                                  yrem_out=ya[t], status_dev=status)
        egtp.plp_step(ctx, st_b, lm, head.c, hs[t], reset_src=reset[t], Hstep_out=Hb[t], z_out=zb[t], yrem_out=yb[t],
                      status_dev=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # per step: entropy from logits + update + head layer 1 + head output, and the 4 kernels of plp_step; bound:
    # entropy from logits + projection + fused update (and 3 launches once for the projection of the empty state: halves, GEMM, sum)
    assert egtp.egtp_launch_count(ctx) - n0 == ((3 + 4) * steps + 3 if bind else (4 + 4) * steps)
    # oracle on exactly the logits the kernel read (bf16-rounded), followed through the token lists
    H_ref = np.stack([orc.entropy_from_logits(x.astype(np.float64)) for x in logits_all])
    follow = [0, 64, slots - 1]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow, H_steps=H_ref[:, follow])
    Ha_n, za_n, ya_n = (a.cpu().numpy().astype(np.float64) for a in (Ha, za, ya))
    gu.assert_entropy_close(Ha_n.ravel(), H_ref.ravel())
    for t in range(steps):
        gu.assert_pooled_close(za_n[t, follow], ref["z"][t])
    gu.assert_length_close(ya_n[:, follow].ravel(), ref["yrem"].ravel())
    # and against the GEMM-fused path: bf16 rounding of the logits moves the entropy by well under the tolerance
    assert np.abs(Ha_n - Hb.cpu().numpy()).max() < 5e-3
    # (the two paths read different inputs, rounded and unrounded logits: close, not equal to tolerance)
    yb_n = yb.cpu().numpy().astype(np.float64)
    assert np.abs(ya_n - yb_n).max() <= 2e-3 * max(1.0, np.abs(yb_n).max())
    egtp.plp_state_destroy(st_a); egtp.plp_state_destroy(st_b)


def test_entropy_from_logits_many_rows_twice():
    # more rows than a grid dimension of 65535 would hold, and the same context used twice in a row: the per-row
    # arrival counters of the in-kernel merge must be back at zero after every call
    rows, V = 70000, 72
    rng = np.random.default_rng(5)
    x = gen.round_to_bf16((rng.standard_normal((rows, V)) * 2.0).astype(np.float32))
    c = egtp.egtp_create(0, max_tokens=rows, max_batch=64, max_d=64, max_V=1024)
    try:
        dev = gu.dev_tensor(x, "bf16")
        ref = orc.entropy_from_logits(x.astype(np.float64))
        for _ in range(2):
            gu.assert_entropy_close(_entropy(c, dev, V), ref)
    finally:
        egtp.egtp_destroy(c)
