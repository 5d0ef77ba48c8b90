"""GPU parity for the vocabulary-parallel form of Eq. 2: the LM head is cut into row shards, each shard
yields one (m, s, t2) triple per token, and the merged triples must give the entropy of the whole
vocabulary.  The shards run one after the other on the single GPU available here; the exchange
between ranks is a plain all-gather of the triples (see tests/test_shard_gloo.py for that part)."""
import numpy as np
import pytest
import torch

from oracle import egtp_oracle as orc
from paper_2602_11812_b200 import binding as egtp
from paper_2602_11812_b200 import inputs as gen
from paper_2602_11812_b200 import shard
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = egtp.egtp_create(0, max_tokens=4096, max_batch=512, max_d=512, max_V=40000)
    yield c
    egtp.egtp_destroy(c)


def _gathered_partials(ctx, hidden_dev, W_dev, world):
    rows = hidden_dev.shape[0]
    V = W_dev.shape[0]
    out = torch.zeros(world, rows, 3, device="cuda")
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    for r, (v0, v1) in enumerate(shard.vocab_shards(V, world)):
        lm = egtp.make_lm_head(W_dev[v0:v1])
        egtp.egtp_entropy_partials(ctx, lm, hidden_dev, out[r], status_dev=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out


@pytest.mark.parametrize("world", [2, 3, 8])
@pytest.mark.parametrize("rows", [70, 300, 1500])
def test_sharded_entropy_matches_oracle_and_single_gpu(ctx, world, rows):
    d, V = 256, 20000 + 72
    rng = np.random.default_rng(world * 100 + rows)
    hidden = gen.round_to_bf16((rng.standard_normal((rows, d)) * 1.5).astype(np.float32))
    W = gen.round_to_bf16(gen.make_lm_head(7, V, d, "bf16") * np.float32(4.0))
    hd, Wd = gu.dev_tensor(hidden, "bf16"), gu.dev_tensor(W, "bf16")
    sh = shard.vocab_shards(V, world)
    assert sh[0][0] == 0 and sh[-1][1] == V and all(a[1] == b[0] for a, b in zip(sh, sh[1:]))
    gathered = _gathered_partials(ctx, hd, Wd, world)
    H = torch.empty(rows, device="cuda")
    egtp.egtp_entropy_from_partials(ctx, gathered, H)
    torch.cuda.synchronize()
    H = H.cpu().numpy().astype(np.float64)
    gu.assert_entropy_close(H, orc.token_entropy(hidden, W))
    # same answer as the unsharded kernel up to summation order
    wl = gen.EgtpWorkload("x", "bf16", hidden, np.array([0, rows], np.int32), W, gen.make_head(1, d, 16, 1, "bf16"))
    assert np.abs(H - gu.run_egtp(ctx, wl)["H"]).max() < 2e-5


@pytest.mark.parametrize("bind", [False, True])
def test_plp_step_from_partials_matches_plp_step(ctx, bind):
    # bind: both states are bound to the head (the sharded one gets W1 h' from a projection launch, the other from
    # the LM-head kernel's extra columns)
    wl = gen.config_plp_decode(slots=140, steps=4, d=256, V=9000, m_h=64, mu=1.0, sigma=0.6)
    steps, slots, d = wl.steps, wl.slots, wl.d
    Wd = gu.dev_tensor(wl.W, "bf16")
    head = gu.DeviceHead(wl.head, "bf16")
    hs = gu.dev_tensor(wl.hidden_steps.reshape(-1, d), "bf16").reshape(steps, slots, d)
    reset = torch.from_numpy(wl.reset_src).cuda()
    st_a, st_b = egtp.plp_state_create(ctx, slots, d), egtp.plp_state_create(ctx, slots, d)
    if bind:
        egtp.plp_state_bind_head(st_a, head.c)
        egtp.plp_state_bind_head(st_b, head.c)
    f = dict(device="cuda", dtype=torch.float32)
    ya, yb = torch.zeros(steps, slots, **f), torch.zeros(steps, slots, **f)
    za, zb = torch.zeros(steps, slots, d, **f), torch.zeros(steps, slots, d, **f)
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    for t in range(steps):
        gathered = _gathered_partials(ctx, hs[t], Wd, 4)
        egtp.plp_step_from_partials(ctx, st_a, gathered, head.c, hs[t], reset_src=reset[t], z_out=za[t], yrem_out=ya[t],
                                    status_dev=status)
        egtp.plp_step(ctx, st_b, egtp.make_lm_head(Wd), head.c, hs[t], reset_src=reset[t], z_out=zb[t], yrem_out=yb[t],
                      status_dev=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    follow = [0, 77, 139]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow)
    za_n, ya_n = za.cpu().numpy().astype(np.float64), ya.cpu().numpy().astype(np.float64)
    for t in range(steps):
        gu.assert_pooled_close(za_n[t, follow], ref["z"][t])
    gu.assert_length_close(ya_n[:, follow].ravel(), ref["yrem"].ravel())
    assert torch.allclose(za, zb, rtol=1e-4, atol=1e-5) and torch.allclose(ya, yb, atol=1e-3)
    egtp.plp_state_destroy(st_a); egtp.plp_state_destroy(st_b)
