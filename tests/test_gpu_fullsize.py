"""GPU parity at the full sizes of the named configurations, in the launch shapes the benchmark times.

The CUDA path runs each whole workload.  The fp64 oracle (2 d V flops per token) follows whole prompts
through its complete chain (Eq. 2 entropies, Eq. 3 weights, Eq. 4 pooled vector, Eq. 6 length): every
prompt of the mid configuration; the two longest, the two shortest, the median and eight seeded-random
prompts of the long-tailed configuration; the shortest, the longest and two random prompts of the RL
configuration; plus seeded-random single tokens elsewhere (entropy).  Decode configurations are followed
slot by slot from explicit token lists (Eq. 8).  Every length is checked twice: with the configuration's
Xavier-initialised head (predictions of a fraction of a token) and with the same head rescaled to predict a
few hundred tokens.  Oracle entropies are memoised on disk by input digest (tests/oracle_cache.py).
What is defined without the LM head is checked everywhere: segment ids (bit-exact) and weights summing to one.
"""
import numpy as np
import pytest
import torch

from oracle import egtp_oracle as orc
from paper_2602_11812_b200 import binding as egtp
from paper_2602_11812_b200 import inputs as gen
from tests import gpu_util as gu
from tests import oracle_cache as oc

pytestmark = pytest.mark.gpu


def _pick_prompts(wl, n_short, n_long, median, n_random, seed=7):
    """Prompt indices: the shortest, the longest, the median one and seeded-random others (ascending)."""
    order = [int(b) for b in np.argsort(wl.lengths, kind="stable")]
    pick = order[:n_short] + (order[len(order) - n_long:] if n_long else []) + ([order[len(order) // 2]] if median else [])
    rest = [b for b in range(wl.B) if b not in pick]
    pick += [int(b) for b in np.random.default_rng(seed).choice(rest, size=min(n_random, len(rest)), replace=False)]
    return sorted(set(pick))


def _whole_prompts(wl, pick):
    off = wl.offsets.astype(np.int64)
    rows = np.concatenate([wl.hidden[off[b]:off[b + 1]] for b in pick])
    sub_off = np.concatenate([[0], np.cumsum([off[b + 1] - off[b] for b in pick])])
    return rows, sub_off


def _gather(x, wl, pick):
    off = wl.offsets.astype(np.int64)
    return np.concatenate([x[off[b]:off[b + 1]] for b in pick])


def _tokens_elsewhere(wl, pick, n_tokens, seed):
    """Seeded-random token indices outside the picked prompts (ascending)."""
    off = wl.offsets.astype(np.int64)
    outside = np.setdiff1d(np.arange(wl.T), np.concatenate([np.arange(off[b], off[b + 1]) for b in pick]))
    return np.sort(np.random.default_rng(seed).choice(outside, size=min(n_tokens, outside.shape[0]), replace=False))


def _check_egtp_full(ctx, wl, pick, n_tokens=0, seed=7):
    """Runs the whole batch on the GPU (once per head) and compares the picked prompts with the oracle's full chain."""
    W_dev = gu.dev_tensor(wl.W, wl.dtype)
    hidden_dev = gu.dev_tensor(wl.hidden, wl.dtype)
    off = wl.offsets.astype(np.int64)
    T = wl.T
    rows, sub_off = _whole_prompts(wl, pick)
    H_ref = oc.token_entropy(rows, wl.W)
    first = None
    for head in (wl.head, gen.scaled_head(wl.head, wl.dtype)):
        res = gu.run_egtp(ctx, wl, W_dev=W_dev, hidden_dev=hidden_dev, head_dev=gu.DeviceHead(head, wl.dtype))
        assert res["status"] == 0
        # segment ids: unique answer, bit-exact everywhere (oracle's linear scan)
        assert np.array_equal(res["seg_id"], orc.segment_ids(off, T))
        ref = orc.egtp_predict(rows, sub_off, wl.W, head, wl.alpha, H=H_ref)
        gu.assert_entropy_close(_gather(res["H"], wl, pick), ref["H"])
        w_gpu = _gather(res["weights"], wl, pick)
        assert np.all(np.abs(w_gpu - ref["weights"]) <= 5e-3 * ref["weights"] + 1e-9)
        gu.assert_pooled_close(res["pooled"][pick], ref["pooled"])
        assert np.allclose(res["state_m"][pick], ref["state_m"], rtol=1e-3)
        assert np.allclose(res["state_s"][pick], ref["state_s"], rtol=5e-3)
        gu.assert_length_close(res["yhat"][pick], ref["yhat"])
        if first is None:
            first = res
            assert np.abs(ref["yhat"]).max() < 5.0          # the configuration's own head: fractions of a token
        else:
            assert np.abs(ref["yhat"]).min() > 100.0        # the rescaled head: hundreds of tokens
            for k in ("H", "weights", "pooled", "seg_id"):  # nothing before the head depends on the head
                assert np.array_equal(res[k], first[k]), k
    res = first
    # seeded-random single tokens of prompts the oracle did not follow
    if n_tokens > 0:
        idx = _tokens_elsewhere(wl, pick, n_tokens, seed)
        gu.assert_entropy_close(res["H"][idx], oc.token_entropy(wl.hidden[idx], wl.W))
    # everywhere: plausible entropies, weights that sum to one per prompt
    assert np.all(res["H"] > 0) and np.all(res["H"] <= np.log(wl.V) + 1e-3)
    for b in range(wl.B):
        assert abs(res["weights"][off[b]:off[b + 1]].sum() - 1.0) < 1e-4
    # prompts the oracle did not follow: internal consistency only (fp64 pooling with the device's own entropies);
    # the parity claim rests on the picked prompts above
    others = [b for b in range(wl.B) if b not in pick]
    for b in np.random.default_rng(seed + 1).choice(others, size=min(4, len(others)), replace=False) if others else []:
        s, e = off[b], off[b + 1]
        gu.assert_pooled_close(res["pooled"][[b]], orc.pool(wl.hidden[s:e], orc.entropy_weights(res["H"][s:e], wl.alpha))[None, :])
    return res, W_dev, dict(rows=rows, offsets=sub_off, H=H_ref, pick=pick)


def test_mid_configuration_full_size():
    # every prompt of the batch goes through the oracle's whole chain
    wl = gen.config_mid()
    assert (wl.B, wl.d, wl.V) == (32, 2048, 151936)
    ctx = egtp.egtp_create(0, max_tokens=wl.T, max_batch=64, max_d=wl.d, max_V=wl.V)
    try:
        _check_egtp_full(ctx, wl, pick=list(range(wl.B)))
    finally:
        egtp.egtp_destroy(ctx)


def test_long_configuration_full_size():
    wl = gen.config_long()
    assert (wl.B, wl.d, wl.V) == (64, 4096, 151936) and wl.offsets.dtype == np.int32
    pick = _pick_prompts(wl, n_short=2, n_long=2, median=True, n_random=8)
    assert len(pick) == 13 and int(np.argmax(wl.lengths)) in pick and wl.lengths[pick].max() > 3000
    ctx = egtp.egtp_create(0, max_tokens=wl.T, max_batch=64, max_d=wl.d, max_V=wl.V)
    try:
        _check_egtp_full(ctx, wl, pick, n_tokens=64)
    finally:
        egtp.egtp_destroy(ctx)


def _steps_on_device(wl):
    return gu.dev_tensor(wl.hidden_steps.reshape(-1, wl.d), wl.dtype).reshape(wl.steps, wl.slots, wl.d)


def _run_plp_steps(ctx, wl, hs, W_dev, head, follow, src=None, bind=False, all_z_steps=0):
    """All steps through plp_step (hs: the steps' hidden rows on the device).  Returns H, y [steps, slots], z of the
    followed slots [steps, len(follow), d] and z of every slot for the first all_z_steps steps."""
    steps, slots, d = wl.steps, wl.slots, wl.d
    reset = torch.from_numpy(wl.reset_src).cuda()
    st = egtp.plp_state_create(ctx, slots, d)
    if bind:     # the head's first layer rides along in the LM-head kernel, one kernel finishes the step
        egtp.plp_state_bind_head(st, head.c)
    lm = egtp.make_lm_head(W_dev)
    f = dict(device="cuda", dtype=torch.float32)
    H, y = torch.zeros(steps, slots, **f), torch.full((steps, slots), float("nan"), **f)
    z_step = torch.zeros(slots, d, **f)
    z_follow = torch.zeros(steps, len(follow), d, **f)
    z_all = torch.zeros(all_z_steps, slots, d, **f)
    fidx = torch.tensor(follow, device="cuda")
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    sm, ss, sp, n_src = (None, None, None, 0) if src is None else src
    for t in range(steps):
        egtp.plp_step(ctx, st, lm, head.c, hs[t], reset_src=reset[t], src_m=sm, src_s=ss, src_pooled=sp, n_src=n_src,
                      Hstep_out=H[t], z_out=z_step, yrem_out=y[t], status_dev=status)
        z_follow[t] = z_step[fidx]
        if t < all_z_steps:
            z_all[t] = z_step
    torch.cuda.synchronize()
    egtp.plp_state_destroy(st)
    assert int(status.item()) == 0
    to64 = lambda a: a.cpu().numpy().astype(np.float64)
    return to64(H), to64(y), to64(z_follow), to64(z_all)


def _compare_followed(run, ref, follow):
    H, y, zf, _ = run
    gu.assert_entropy_close(H[:, follow].ravel(), ref["H"].ravel())
    for t in range(zf.shape[0]):
        gu.assert_pooled_close(zf[t], ref["z"][t])
    gu.assert_length_close(y[:, follow].ravel(), ref["yrem"].ravel())


def test_plp_decode_configuration_full_size():
    # 256 live sequences, d = 4096, V = 151936, all 512 steps of the configuration.  The oracle follows four slots
    # through every step (retire-and-restart events included) and all 256 slots through the first four steps.
    wl = gen.config_plp_decode()
    assert (wl.slots, wl.steps, wl.d, wl.V) == (256, 512, 4096, 151936)
    wl.reset_src[7, 3] = gen.RESET_EMPTY                     # one more restart, early in the run
    retiring = [int(s) for s in np.argwhere((wl.reset_src[1:] == gen.RESET_EMPTY).any(axis=0)).ravel()]
    follow = sorted({3, retiring[len(retiring) // 2], 130, 255})
    assert len(follow) == 4 and (wl.reset_src[1:, follow] == gen.RESET_EMPTY).sum() >= 2
    first_steps = 4
    heads = (wl.head, gen.scaled_head(wl.head, "bf16"))
    ctx = egtp.egtp_create(0, max_tokens=1024, max_batch=256, max_d=wl.d, max_V=wl.V)
    try:
        W_dev = gu.dev_tensor(wl.W, "bf16")
        hs_dev = _steps_on_device(wl)
        runs = {(hi, bind): _run_plp_steps(ctx, wl, hs_dev, W_dev, gu.DeviceHead(head, "bf16"), follow, bind=bind,
                                           all_z_steps=first_steps)
                for hi, head in enumerate(heads) for bind in (False, True)}
    finally:
        egtp.egtp_destroy(ctx)
    H_follow = oc.token_entropy(wl.hidden_steps[:, follow, :].reshape(-1, wl.d), wl.W).reshape(wl.steps, len(follow))
    H_first = oc.token_entropy(wl.hidden_steps[:first_steps].reshape(-1, wl.d), wl.W).reshape(first_steps, wl.slots)
    for hi, head in enumerate(heads):
        ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, head, slots=follow, H_steps=H_follow)
        ref_first = orc.plp_run(wl.hidden_steps[:first_steps], wl.reset_src[:first_steps], wl.W, head, H_steps=H_first)
        assert (np.abs(ref["yrem"]).max() < 5.0) if hi == 0 else (np.abs(ref["yrem"]).min() > 100.0)
        for bind in (False, True):   # the ordinary route, then the state bound to its head (the route bench.py times)
            H, y, zf, z_all = runs[(hi, bind)]
            _compare_followed(runs[(hi, bind)], ref, follow)
            gu.assert_entropy_close(H[:first_steps].ravel(), ref_first["H"].ravel())
            for t in range(first_steps):
                gu.assert_pooled_close(z_all[t], ref_first["z"][t])
            gu.assert_length_close(y[:first_steps].ravel(), ref_first["yrem"].ravel())
            # every slot, every step: finite outputs, entropies in range; a slot that restarts holds its one token
            assert np.all(np.isfinite(y)) and np.all(H > 0) and np.all(H <= np.log(wl.V) + 1e-3)
            assert np.array_equal(zf[7, follow.index(3)], wl.hidden_steps[7, 3].astype(np.float64))
        # both routes on all 256 slots: same entropies and lengths up to summation order
        gu.assert_entropy_close(runs[(hi, True)][0].ravel(), runs[(hi, False)][0].ravel())
        gu.assert_length_close(runs[(hi, True)][1].ravel(), runs[(hi, False)][1].ravel())


def test_rl_group_configuration_full_size():
    # 64 shared prompts (d = 5120, V = 152064), then 1024 decode streams that start from their prompt's state
    steps = 256
    wl = gen.config_rl_group(steps=steps)
    eg = wl.prompts
    assert (eg.B, eg.d, eg.V, wl.slots, wl.steps) == (64, 5120, 152064, 1024, 256)
    pick = _pick_prompts(eg, n_short=1, n_long=1, median=False, n_random=2)
    assert len(pick) == 4
    # four streams of two different groups: the shortest picked prompt's and another picked prompt's
    b0 = min(pick, key=lambda b: eg.lengths[b])
    b1 = [b for b in pick if b != b0 and eg.lengths[b] < 3000][0]
    follow = [16 * b0, 16 * b0 + 15, 16 * b1 + 3, 16 * b1 + 9]
    heads = (wl.head, gen.scaled_head(wl.head, "bf16"))
    ctx = egtp.egtp_create(0, max_tokens=eg.T, max_batch=1024, max_d=eg.d, max_V=eg.V)
    try:
        res, W_dev, followed = _check_egtp_full(ctx, eg, pick, n_tokens=48)
        src = (torch.from_numpy(res["state_m"].astype(np.float32)).cuda(),
               torch.from_numpy(res["state_s"].astype(np.float32)).cuda(),
               torch.from_numpy(res["pooled"].astype(np.float32)).cuda(), eg.B)
        hs_dev = _steps_on_device(wl)
        runs = {(hi, bind): _run_plp_steps(ctx, wl, hs_dev, W_dev, gu.DeviceHead(head, "bf16"), follow, src=src, bind=bind)
                for hi, head in enumerate(heads) for bind in (False, True)}
    finally:
        egtp.egtp_destroy(ctx)
    # the oracle's view of the two prompts: their own rows and entropies (no value from the CUDA path), as prompts 0 and 1
    prompts = dict(hidden=followed["rows"], offsets=followed["offsets"], H=followed["H"])
    reset = wl.reset_src.copy()
    reset[0, follow] = [pick.index(b0), pick.index(b0), pick.index(b1), pick.index(b1)]
    H_follow = oc.token_entropy(wl.hidden_steps[:, follow, :].reshape(-1, wl.d), wl.W).reshape(steps, len(follow))
    for hi, head in enumerate(heads):
        ref = orc.plp_run(wl.hidden_steps, reset, wl.W, head, slots=follow, prompts=prompts, H_steps=H_follow)
        assert (np.abs(ref["yrem"]).max() < 5.0) if hi == 0 else (np.abs(ref["yrem"]).min() > 100.0)
        for bind in (False, True):     # the ordinary route, then the state bound to its head (1024 rows: 8 row blocks)
            _compare_followed(runs[(hi, bind)], ref, follow)
            H, y, zf, _ = runs[(hi, bind)]
            # streams of one group that were fed different tokens differ; all are finite
            assert np.all(np.isfinite(y)) and not np.array_equal(zf[-1, 0], zf[-1, 1])
        gu.assert_length_close(runs[(hi, True)][1].ravel(), runs[(hi, False)][1].ravel())


def test_wide_model_d8192_llama_sized_vocabulary():
    # hidden size 8192 (128 k blocks per tile pass, 16 KB rows) against a 128256-entry vocabulary: a prompt batch
    # (three row blocks) entirely through the oracle, and bound decode steps of 200 streams of which two are followed
    d, V, m_h = 8192, 128256, 512
    lengths = [5, 170, 131]
    wl = gen.make_egtp("wide", 9, lengths, d=d, V=V, dtype="bf16", m_h=m_h)
    ctx = egtp.egtp_create(0, max_tokens=1024, max_batch=256, max_d=d, max_V=V)
    try:
        _, W_dev, _ = _check_egtp_full(ctx, wl, pick=[0, 1, 2])
        # decode: 200 streams, 3 steps, state bound to the head
        rng = np.random.Generator(np.random.PCG64(909))
        hs = gen.round_to_bf16(rng.standard_normal((3, 200, d)).astype(np.float32))
        reset = np.full((3, 200), gen.RESET_KEEP, np.int32); reset[0] = gen.RESET_EMPTY
        pw = gen.PlpWorkload("wide_decode", "bf16", hs, reset, wl.W, wl.head)
        follow = [0, 199]
        heads = (wl.head, gen.scaled_head(wl.head, "bf16"))
        hs_dev = _steps_on_device(pw)
        runs = [_run_plp_steps(ctx, pw, hs_dev, W_dev, gu.DeviceHead(head, "bf16"), follow, bind=True) for head in heads]
    finally:
        egtp.egtp_destroy(ctx)
    H_follow = oc.token_entropy(hs[:, follow, :].reshape(-1, d), wl.W).reshape(3, 2)
    for head, run in zip(heads, runs):
        _compare_followed(run, orc.plp_run(hs, reset, wl.W, head, slots=follow, H_steps=H_follow), follow)
