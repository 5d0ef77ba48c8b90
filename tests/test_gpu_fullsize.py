"""GPU parity at the full sizes of the named configurations, in the launch shapes the benchmark times.

The CUDA path runs each whole workload once.  The fp64 oracle cannot (2 d V flops per token), so it
computes, one by one, outputs that depend on few tokens: whole shortest prompts (entropies, weights,
pooled vector, predicted length) and seeded-random single tokens elsewhere (entropy).  What is
defined without the LM head is checked everywhere: segment ids (bit-exact), weights summing to one
per prompt, and the pooled vectors recomputed in fp64 from the device's own entropies.
"""
import numpy as np
import pytest
import torch

from oracle import egtp_oracle as orc
from paper_2602_11812_b200 import binding as egtp
from paper_2602_11812_b200 import inputs as gen
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _shortest_prompts(wl, n):
    return [int(b) for b in np.argsort(wl.lengths, kind="stable")[:n]]


def _check_egtp_full(ctx, wl, n_prompts=2, n_tokens=32, seed=7):
    W_dev = gu.dev_tensor(wl.W, wl.dtype)
    res = gu.run_egtp(ctx, wl, W_dev=W_dev)
    assert res["status"] == 0
    off = wl.offsets.astype(np.int64)
    T = wl.T
    # segment ids: unique answer, bit-exact everywhere (oracle's linear scan)
    assert np.array_equal(res["seg_id"], orc.segment_ids(off, T))
    # whole shortest prompts against the oracle
    pick = _shortest_prompts(wl, n_prompts)
    rows = np.concatenate([wl.hidden[off[b]:off[b + 1]] for b in pick])
    sub_off = np.concatenate([[0], np.cumsum([off[b + 1] - off[b] for b in pick])])
    ref = orc.egtp_predict(rows, sub_off, wl.W, wl.head, wl.alpha)
    H_gpu = np.concatenate([res["H"][off[b]:off[b + 1]] for b in pick])
    w_gpu = np.concatenate([res["weights"][off[b]:off[b + 1]] for b in pick])
    gu.assert_entropy_close(H_gpu, ref["H"])
    assert np.all(np.abs(w_gpu - ref["weights"]) <= 5e-3 * ref["weights"] + 1e-9)
    gu.assert_pooled_close(res["pooled"][pick], ref["pooled"])
    gu.assert_length_close(res["yhat"][pick], ref["yhat"])
    # seeded-random single tokens anywhere in the batch
    idx = np.sort(np.random.default_rng(seed).choice(T, size=n_tokens, replace=False))
    gu.assert_entropy_close(res["H"][idx], orc.token_entropy(wl.hidden[idx], wl.W))
    # everywhere: plausible entropies, weights sum to one, pooling consistent with the device's entropies
    assert np.all(res["H"] > 0) and np.all(res["H"] <= np.log(wl.V) + 1e-3)
    for b in range(wl.B):
        s, e = off[b], off[b + 1]
        assert abs(res["weights"][s:e].sum() - 1.0) < 1e-4
    check = np.random.default_rng(seed + 1).choice(wl.B, size=min(6, wl.B), replace=False)
    longest = int(np.argmax(wl.lengths))
    for b in set(check.tolist() + [longest]):
        s, e = off[b], off[b + 1]
        w = orc.entropy_weights(res["H"][s:e], wl.alpha)
        gu.assert_pooled_close(res["pooled"][[b]], orc.pool(wl.hidden[s:e], w)[None, :])
    return res, W_dev


def test_mid_configuration_full_size():
    wl = gen.config_mid()
    assert (wl.B, wl.d, wl.V) == (32, 2048, 151936)
    ctx = egtp.egtp_create(0, max_tokens=wl.T, max_batch=64, max_d=wl.d, max_V=wl.V)
    try:
        _check_egtp_full(ctx, wl)
    finally:
        egtp.egtp_destroy(ctx)


def test_long_configuration_full_size():
    wl = gen.config_long()
    assert (wl.B, wl.d, wl.V) == (64, 4096, 151936) and wl.offsets.dtype == np.int32
    ctx = egtp.egtp_create(0, max_tokens=wl.T, max_batch=64, max_d=wl.d, max_V=wl.V)
    try:
        _check_egtp_full(ctx, wl, n_tokens=24)
    finally:
        egtp.egtp_destroy(ctx)


def _run_plp_steps(ctx, wl, W_dev, head, src=None, bind=False):
    steps, slots, d = wl.steps, wl.slots, wl.d
    hs = gu.dev_tensor(wl.hidden_steps.reshape(-1, d), wl.dtype).reshape(steps, slots, d)
    reset = torch.from_numpy(wl.reset_src).cuda()
    st = egtp.plp_state_create(ctx, slots, d)
    if bind:     # the head's first layer rides along in the LM-head kernel, one kernel finishes the step
        egtp.plp_state_bind_head(st, head.c)
    lm = egtp.make_lm_head(W_dev)
    f = dict(device="cuda", dtype=torch.float32)
    H, z, y = torch.zeros(steps, slots, **f), torch.zeros(steps, slots, d, **f), torch.zeros(steps, slots, **f)
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    sm, ss, sp, n_src = (None, None, None, 0) if src is None else src
    for t in range(steps):
        egtp.plp_step(ctx, st, lm, head.c, hs[t], reset_src=reset[t], src_m=sm, src_s=ss, src_pooled=sp, n_src=n_src,
                      Hstep_out=H[t], z_out=z[t], yrem_out=y[t], status_dev=status)
    torch.cuda.synchronize()
    egtp.plp_state_destroy(st)
    assert int(status.item()) == 0
    return H.cpu().numpy().astype(np.float64), z.cpu().numpy().astype(np.float64), y.cpu().numpy().astype(np.float64)


def test_plp_decode_configuration_full_width():
    # 256 live sequences, d = 4096, V = 151936: the decode launch shape; a window of 20 steps with a
    # retire-and-restart event forced into it for one followed slot
    wl = gen.config_plp_decode(steps=20)
    assert (wl.slots, wl.d, wl.V) == (256, 4096, 151936)
    wl.reset_src[7, 3] = gen.RESET_EMPTY
    ctx = egtp.egtp_create(0, max_tokens=1024, max_batch=256, max_d=wl.d, max_V=wl.V)
    try:
        W_dev = gu.dev_tensor(wl.W, "bf16")
        head = gu.DeviceHead(wl.head, "bf16")
        runs = [_run_plp_steps(ctx, wl, W_dev, head, bind=bind) for bind in (False, True)]
    finally:
        egtp.egtp_destroy(ctx)
    follow = [3, 130, 255]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow)
    for H, z, y in runs:       # the ordinary route, then the state bound to its head (the route bench.py times)
        gu.assert_entropy_close(H[:, follow].ravel(), ref["H"].ravel())
        for t in range(wl.steps):
            gu.assert_pooled_close(z[t, follow], ref["z"][t])
        gu.assert_length_close(y[:, follow].ravel(), ref["yrem"].ravel())
        # every slot, every step: z is a convex combination of the tokens seen since the last reset
        assert np.all(np.isfinite(z)) and np.all(H > 0) and np.all(H <= np.log(wl.V) + 1e-3)
        assert np.array_equal(z[7, 3], wl.hidden_steps[7, 3].astype(np.float64))
    # both routes on all 256 slots: same entropies and lengths up to summation order
    gu.assert_entropy_close(runs[1][0].ravel(), runs[0][0].ravel())
    gu.assert_length_close(runs[1][2].ravel(), runs[0][2].ravel())


def test_rl_group_configuration_full_size():
    # 64 shared prompts (d = 5120, V = 152064), then 1024 decode streams that start from their prompt's state
    wl = gen.config_rl_group(steps=4)
    eg = wl.prompts
    assert (eg.B, eg.d, eg.V, wl.slots) == (64, 5120, 152064, 1024)
    ctx = egtp.egtp_create(0, max_tokens=eg.T, max_batch=1024, max_d=eg.d, max_V=eg.V)
    try:
        res, W_dev = _check_egtp_full(ctx, eg, n_prompts=1, n_tokens=16)
        src = (torch.from_numpy(res["state_m"].astype(np.float32)).cuda(),
               torch.from_numpy(res["state_s"].astype(np.float32)).cuda(),
               torch.from_numpy(res["pooled"].astype(np.float32)).cuda(), eg.B)
        head = gu.DeviceHead(wl.head, "bf16")
        runs = [_run_plp_steps(ctx, wl, W_dev, head, src=src, bind=bind) for bind in (False, True)]
    finally:
        egtp.egtp_destroy(ctx)
    b = _shortest_prompts(eg, 1)[0]
    follow = [16 * b, 16 * b + 15]
    off = eg.offsets.astype(np.int64)
    rows = eg.hidden[off[b]:off[b + 1]]
    H_prompt = orc.token_entropy(rows, eg.W)
    reset = wl.reset_src.copy()
    reset[0, follow] = 0
    ref = orc.plp_run(wl.hidden_steps, reset, wl.W, wl.head, slots=follow,
                      prompts=dict(hidden=rows, offsets=np.array([0, rows.shape[0]]), H=H_prompt))
    for H, z, y in runs:       # the ordinary route, then the state bound to its head (1024 rows: 8 row blocks)
        gu.assert_entropy_close(H[:, follow].ravel(), ref["H"].ravel())
        for t in range(wl.steps):
            gu.assert_pooled_close(z[t, follow], ref["z"][t])
        gu.assert_length_close(y[:, follow].ravel(), ref["yrem"].ravel())
        # streams of one group that were fed different tokens differ; all are finite
        assert np.all(np.isfinite(y)) and not np.array_equal(z[-1, follow[0]], z[-1, follow[1]])
    gu.assert_length_close(runs[1][2].ravel(), runs[0][2].ravel())


def test_wide_model_d8192_llama_sized_vocabulary():
    # hidden size 8192 (128 k blocks per tile pass, 16 KB rows) against a 128256-entry vocabulary: a prompt batch
    # (three row blocks) and bound decode steps of 200 streams; the oracle follows sampled tokens and two streams
    d, V, m_h = 8192, 128256, 512
    lengths = [5, 170, 131]
    wl = gen.make_egtp("wide", 9, lengths, d=d, V=V, dtype="bf16", m_h=m_h)
    ctx = egtp.egtp_create(0, max_tokens=1024, max_batch=256, max_d=d, max_V=V)
    try:
        W_dev = gu.dev_tensor(wl.W, "bf16")
        res = gu.run_egtp(ctx, wl, W_dev=W_dev)
        assert res["status"] == 0
        off = wl.offsets.astype(np.int64)
        assert np.array_equal(res["seg_id"], orc.segment_ids(off, wl.T))
        idx = np.array([0, 4, 5, 127, 128, 174, 175, 305])
        gu.assert_entropy_close(res["H"][idx], orc.token_entropy(wl.hidden[idx], wl.W))
        ref0 = orc.egtp_predict(wl.hidden[:5], np.array([0, 5]), wl.W, wl.head)        # the 5-token prompt in full
        gu.assert_pooled_close(res["pooled"][[0]], ref0["pooled"])
        gu.assert_length_close(res["yhat"][[0]], ref0["yhat"])
        for b in (1, 2):
            w = orc.entropy_weights(res["H"][off[b]:off[b + 1]])
            gu.assert_pooled_close(res["pooled"][[b]], orc.pool(wl.hidden[off[b]:off[b + 1]], w)[None, :])
        y_ref, _ = orc.head_forward(res["pooled"], wl.head.W1, wl.head.b1, wl.head.W2, wl.head.b2)
        gu.assert_length_close(res["yhat"], y_ref)
        # decode: 200 streams, 3 steps, state bound to the head
        rng = np.random.Generator(np.random.PCG64(909))
        hs = gen.round_to_bf16(rng.standard_normal((3, 200, d)).astype(np.float32))
        reset = np.full((3, 200), gen.RESET_KEEP, np.int32); reset[0] = gen.RESET_EMPTY
        pw = gen.PlpWorkload("wide_decode", "bf16", hs, reset, wl.W, wl.head)
        H, z, y = _run_plp_steps(ctx, pw, W_dev, gu.DeviceHead(wl.head, "bf16"), bind=True)
    finally:
        egtp.egtp_destroy(ctx)
    follow = [0, 199]
    ref = orc.plp_run(hs, reset, wl.W, wl.head, slots=follow)
    gu.assert_entropy_close(H[:, follow].ravel(), ref["H"].ravel())
    for t in range(3):
        gu.assert_pooled_close(z[t, follow], ref["z"][t])
    gu.assert_length_close(y[:, follow].ravel(), ref["yrem"].ravel())
