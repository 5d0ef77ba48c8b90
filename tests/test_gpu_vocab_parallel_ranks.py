"""The vocabulary-parallel PLP step as real ranks: two processes, each holding half of the LM head's rows, share
the one GPU and exchange their per-row entropy triples over a gloo group (host memory).  Their kernels never wait
on one another, only the host-side all-gather couples them, so running them on one device is the same orchestration
that runs on two.  Every rank's predictions are compared with the oracle, which knows nothing of shards."""
import os
import socket
import sys
import tempfile

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
WORLD, STEPS, SLOTS, D, V, M_H = 2, 5, 140, 256, 9000 + 40, 64


def _workload():
    from paper_2602_11812_b200 import inputs as gen
    wl = gen.config_plp_decode(slots=SLOTS, steps=STEPS, d=D, V=V, m_h=M_H, mu=1.2, sigma=0.6)
    wl.head = gen.scaled_head(wl.head, "bf16")          # remaining lengths of hundreds of tokens
    return wl


def _rank_main(rank: int, port: int, out_dir: str, bind: bool):
    if ROOT not in sys.path:
        sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist

    from paper_2602_11812_b200 import binding as egtp
    from paper_2602_11812_b200 import device as dev
    from paper_2602_11812_b200 import shard

    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=WORLD)
    try:
        torch.cuda.set_device(0)
        wl = _workload()
        v0, v1 = shard.vocab_shards(V, WORLD)[rank]
        W_shard = dev.dev_tensor(wl.W[v0:v1], "bf16")       # this rank never holds the other rows
        head = dev.DeviceHead(wl.head, "bf16")
        ctx = egtp.egtp_create(0, max_tokens=1024, max_batch=256, max_d=D, max_V=V)
        st = egtp.plp_state_create(ctx, SLOTS, D)
        if bind:
            egtp.plp_state_bind_head(st, head.c)
        lm = egtp.make_lm_head(W_shard)
        f = dict(device="cuda", dtype=torch.float32)
        H, y = torch.zeros(STEPS, SLOTS, **f), torch.zeros(STEPS, SLOTS, **f)
        z = torch.zeros(STEPS, SLOTS, D, **f)
        status = torch.zeros(1, device="cuda", dtype=torch.int32)
        for t in range(STEPS):
            hs = dev.dev_tensor(wl.hidden_steps[t], "bf16")
            reset = torch.from_numpy(wl.reset_src[t].copy()).cuda()
            gathered = shard.plp_step_vocab_parallel(ctx, st, lm, head.c, hs, reset_src=reset, Hstep_out=H[t], z_out=z[t],
                                                     yrem_out=y[t], status_dev=status)
            assert gathered.shape == (WORLD, SLOTS, 3)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), H=H.cpu().numpy(), y=y.cpu().numpy(), z=z.cpu().numpy())
        egtp.plp_state_destroy(st)
        egtp.egtp_destroy(ctx)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("bind", [False, True])
def test_two_ranks_sharing_one_gpu_match_the_oracle(bind):
    import torch.multiprocessing as mp

    from oracle import egtp_oracle as orc
    from tests import gpu_util as gu

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    with tempfile.TemporaryDirectory() as out_dir:
        mp.spawn(_rank_main, args=(port, out_dir, bind), nprocs=WORLD, join=True)
        runs = [np.load(os.path.join(out_dir, f"rank{r}.npz")) for r in range(WORLD)]
        runs = [{k: r[k].astype(np.float64) for k in ("H", "y", "z")} for r in runs]
    wl = _workload()
    follow = [0, 77, SLOTS - 1]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow)
    assert np.abs(ref["yrem"]).min() > 100
    for r in runs:
        gu.assert_entropy_close(r["H"][:, follow].ravel(), ref["H"].ravel())
        for t in range(STEPS):
            gu.assert_pooled_close(r["z"][t, follow], ref["z"][t])
        gu.assert_length_close(r["y"][:, follow].ravel(), ref["yrem"].ravel())
    # replicas of the state advance in lock step: both ranks hold bitwise the same results
    for k in ("H", "y", "z"):
        assert np.array_equal(runs[0][k], runs[1][k]), k
