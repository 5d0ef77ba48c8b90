"""GPU parity: plp_step through the C ABI against the oracle, which recomputes Eq. 8 from explicit token lists."""
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
    c = egtp.egtp_create(0, max_tokens=8192, max_batch=512, max_d=1024, max_V=40000)
    yield c
    egtp.egtp_destroy(c)


def _run_plp(ctx, wl: gen.PlpWorkload, src=None, slot_ids=None, num_slots=None, head=None):
    """All steps of a PLP workload through plp_step; returns H, z, yrem as float64 arrays [steps, slots(, d)]."""
    steps, slots, d = wl.steps, wl.slots, wl.d
    W = gu.dev_tensor(wl.W, wl.dtype)
    head = gu.DeviceHead(wl.head if head is None else head, wl.dtype)
    hs = gu.dev_tensor(wl.hidden_steps.reshape(-1, d), wl.dtype).reshape(steps, slots, d)
    reset = torch.from_numpy(wl.reset_src).cuda()
    st = egtp.plp_state_create(ctx, num_slots or slots, d)
    lm = egtp.make_lm_head(W)
    f = dict(device="cuda", dtype=torch.float32)
    H = torch.zeros(steps, slots, **f)
    z = torch.zeros(steps, slots, d, **f)
    y = torch.zeros(steps, slots, **f)
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    sm, ss, sp, n_src = (None, None, None, 0) if src is None else src
    for t in range(steps):
        egtp.plp_step(ctx, st, lm, head.c, hs[t], slot_ids=slot_ids, reset_src=reset[t], src_m=sm, src_s=ss,
                      src_pooled=sp, n_src=n_src, Hstep_out=H[t], z_out=z[t], yrem_out=y[t], status_dev=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, egtp.status_string(int(status.item()))
    return st, H.cpu().numpy().astype(np.float64), z.cpu().numpy().astype(np.float64), y.cpu().numpy().astype(np.float64)


def _compare(H, z, y, ref, slots):
    gu.assert_entropy_close(H[:, slots].ravel(), ref["H"].ravel())
    for t in range(z.shape[0]):
        gu.assert_pooled_close(z[t, slots], ref["z"][t])
    gu.assert_length_close(y[:, slots].ravel(), ref["yrem"].ravel())


def test_decode_loop_with_retirement_matches_oracle(ctx):
    # the PLP decode configuration's recipe at reduced size: slots retire at lognormal lengths and restart empty
    wl = gen.config_plp_decode(slots=130, steps=40, d=256, V=9000, m_h=64, mu=2.0, sigma=0.8)
    assert (wl.reset_src[1:] == gen.RESET_EMPTY).sum() > 50
    st, H, z, y = _run_plp(ctx, wl)
    follow = [0, 1, 57, 128, 129]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow)
    _compare(H, z, y, ref, follow)
    # the same loop with the head rescaled to predict hundreds of tokens (the first one predicts fractions of one)
    big = gen.scaled_head(wl.head, "bf16")
    st_b, H_b, z_b, y_b = _run_plp(ctx, wl, head=big)
    ref_b = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, big, slots=follow, H_steps=ref["H"])
    assert np.abs(ref_b["yrem"]).min() > 100
    _compare(H_b, z_b, y_b, ref_b, follow)
    egtp.plp_state_destroy(st_b)
    # a slot that was just reset holds exactly its one token: z == h'
    t, s = np.argwhere(wl.reset_src[1:] == gen.RESET_EMPTY)[0]
    assert np.array_equal(z[t + 1, s], wl.hidden_steps[t + 1, s].astype(np.float64))
    egtp.plp_state_destroy(st)


def test_decode_loop_in_cta_pair_mode(ctx):
    wl = gen.config_plp_decode(slots=200, steps=6, d=256, V=9000 + 40, m_h=64, mu=1.0, sigma=0.5)
    egtp.egtp_set_lmhead_mode(ctx, egtp.EGTP_LMHEAD_CTA_PAIRS)
    try:
        st, H, z, y = _run_plp(ctx, wl)
    finally:
        egtp.egtp_set_lmhead_mode(ctx, egtp.EGTP_LMHEAD_AUTO)
    follow = [0, 127, 128, 199]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow)
    _compare(H, z, y, ref, follow)
    egtp.plp_state_destroy(st)


def test_decode_loop_in_single_cta_mode(ctx):
    # 129..256 rows default to CTA pairs on 256 x 512 tiles; the one-CTA form (both row tiles per W tile) stays selectable
    wl = gen.config_plp_decode(slots=200, steps=6, d=256, V=9000 + 40, m_h=64, mu=1.0, sigma=0.5)
    egtp.egtp_set_lmhead_mode(ctx, egtp.EGTP_LMHEAD_SINGLE_CTA)
    try:
        assert egtp.egtp_lmhead_plan(ctx, 200, 256, 9040, egtp.EGTP_BF16)["rows_per_block"] == 256
        st, H, z, y = _run_plp(ctx, wl)
    finally:
        egtp.egtp_set_lmhead_mode(ctx, egtp.EGTP_LMHEAD_AUTO)
    follow = [0, 127, 128, 199]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow)
    _compare(H, z, y, ref, follow)
    egtp.plp_state_destroy(st)


def test_rl_group_sampling_continues_from_egtp_state(ctx):
    # EGTP over shared prompts, then decode streams that start from their prompt's state (fan-out 4)
    wl = gen.config_rl_group(prompts=5, group=4, steps=12, d=256, V=7000, m_h=64, min_len=3, max_len=200)
    eg = wl.prompts
    res = gu.run_egtp(ctx, eg)
    ref_eg = orc.egtp_predict(eg.hidden, eg.offsets, eg.W, eg.head)
    gu.assert_pooled_close(res["pooled"], ref_eg["pooled"])
    src = (torch.from_numpy(res["state_m"].astype(np.float32)).cuda(), torch.from_numpy(res["state_s"].astype(np.float32)).cuda(),
           torch.from_numpy(res["pooled"].astype(np.float32)).cuda(), eg.B)
    st, H, z, y = _run_plp(ctx, wl, src=src)
    follow = [0, 3, 4, 19]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow,
                      prompts=dict(hidden=eg.hidden, offsets=eg.offsets, H=ref_eg["H"]))
    _compare(H, z, y, ref, follow)
    big = gen.scaled_head(wl.head, "bf16")                     # the same streams with a head that predicts hundreds of tokens
    st_b, H_b, z_b, y_b = _run_plp(ctx, wl, src=src, head=big)
    ref_b = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, big, slots=follow, H_steps=ref["H"],
                        prompts=dict(hidden=eg.hidden, offsets=eg.offsets, H=ref_eg["H"]))
    assert np.abs(ref_b["yrem"]).min() > 100
    _compare(H_b, z_b, y_b, ref_b, follow)
    egtp.plp_state_destroy(st_b)
    # streaming state == batch EGTP over the concatenation [prompt 0 ; generated tokens 1..12] of slot 0
    cat = np.concatenate([eg.hidden[eg.offsets[0]:eg.offsets[1]], wl.hidden_steps[:, 0, :]])
    both = orc.egtp_predict(cat, np.array([0, cat.shape[0]]), wl.W, wl.head)
    gu.assert_pooled_close(z[-1, [0]], both["pooled"])
    egtp.plp_state_destroy(st)


def test_identical_streams_stay_bitwise_identical_and_slot_mapping(ctx):
    rng = np.random.default_rng(5)
    d, V, steps = 128, 3000, 6
    one = gen.round_to_bf16(rng.standard_normal((steps, 1, d)).astype(np.float32))
    hs = np.repeat(one, 16, axis=1)
    reset = np.full((steps, 16), gen.RESET_KEEP, np.int32)
    reset[0] = gen.RESET_EMPTY
    wl = gen.PlpWorkload("fan", "bf16", hs, reset, gen.make_lm_head(3, V, d, "bf16"), gen.make_head(4, d, 32, 1, "bf16"))
    # rows are scattered over a larger slot table through slot_ids
    slot_ids = torch.tensor([31 - 2 * i for i in range(16)], dtype=torch.int32, device="cuda")
    st, H, z, y = _run_plp(ctx, wl, slot_ids=slot_ids, num_slots=32)
    for s in range(1, 16):
        assert np.array_equal(z[:, s], z[:, 0]) and np.array_equal(y[:, s], y[:, 0])
    # exported state: used slots hold the same triple, unused slots are still empty
    m = torch.empty(32, device="cuda"); sarr = torch.empty(32, device="cuda"); acc = torch.empty(32, d, device="cuda")
    egtp.plp_state_export(st, m, sarr, acc)
    torch.cuda.synchronize()
    used = slot_ids.cpu().numpy()
    unused = np.setdiff1d(np.arange(32), used)
    assert np.all(sarr.cpu().numpy()[unused] == 0) and np.all(np.isneginf(m.cpu().numpy()[unused]))
    assert np.all(acc.cpu().numpy()[used] == acc.cpu().numpy()[used[0]])
    zz = acc.cpu().numpy()[used[0]].astype(np.float64) / float(sarr.cpu().numpy()[used[0]])
    assert np.allclose(zz, z[-1, 0], rtol=1e-6, atol=1e-7)
    # import into a fresh state and continue: same result as continuing the original
    st2 = egtp.plp_state_create(ctx, 32, d)
    egtp.plp_state_import(st2, m, sarr, acc)
    W = gu.dev_tensor(wl.W, "bf16"); lm = egtp.make_lm_head(W)
    nxt = gu.dev_tensor(gen.round_to_bf16(rng.standard_normal((16, d)).astype(np.float32)), "bf16")
    z1 = torch.empty(16, d, device="cuda"); z2 = torch.empty(16, d, device="cuda")
    egtp.plp_step(ctx, st, lm, None, nxt, slot_ids=slot_ids, z_out=z1)
    egtp.plp_step(ctx, st2, lm, None, nxt, slot_ids=slot_ids, z_out=z2)
    torch.cuda.synchronize()
    assert torch.equal(z1, z2)
    egtp.plp_state_destroy(st); egtp.plp_state_destroy(st2)


def test_plp_errors_and_host_entry_point(ctx):
    wl = gen.config_plp_decode(slots=8, steps=3, d=128, V=2000, m_h=32, mu=1.0, sigma=0.5)
    W = gu.dev_tensor(wl.W, "bf16"); lm = egtp.make_lm_head(W)
    head = gu.DeviceHead(wl.head, "bf16")
    st = egtp.plp_state_create(ctx, 8, 128)
    hs = gu.dev_tensor(wl.hidden_steps[0], "bf16")
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    bad_slots = torch.tensor([0, 1, 2, 3, 4, 5, 6, 8], dtype=torch.int32, device="cuda")
    egtp.plp_step(ctx, st, lm, None, hs, slot_ids=bad_slots, status_dev=status)
    torch.cuda.synchronize()
    assert int(status.item()) == egtp.EGTP_ERR_BAD_SLOT
    status.zero_()
    bad_reset = torch.full((8,), 3, dtype=torch.int32, device="cuda")      # source row 3 but n_src == 0
    egtp.plp_step(ctx, st, lm, None, hs, reset_src=bad_reset, status_dev=status)
    torch.cuda.synchronize()
    assert int(status.item()) == egtp.EGTP_ERR_BAD_SLOT
    # two rows of one step on the same slot would race on its state: refused on the device, on both routes, and the
    # state serves the next (valid) step as before
    for bind in (False, True):
        st_d = egtp.plp_state_create(ctx, 8, 128)
        if bind:
            egtp.plp_state_bind_head(st_d, head.c)
        dup = torch.tensor([0, 1, 2, 3, 4, 5, 6, 3], dtype=torch.int32, device="cuda")
        y = torch.zeros(8, device="cuda")
        status.zero_()
        egtp.plp_step(ctx, st_d, lm, head.c, hs, slot_ids=dup, yrem_out=y, status_dev=status)
        torch.cuda.synchronize()
        assert int(status.item()) == egtp.EGTP_ERR_BAD_SLOT
        status.zero_()
        ok_ids = torch.arange(8, dtype=torch.int32, device="cuda")
        reset_all = torch.full((8,), gen.RESET_EMPTY, dtype=torch.int32, device="cuda")
        z = torch.zeros(8, 128, device="cuda")
        egtp.plp_step(ctx, st_d, lm, head.c, hs, slot_ids=ok_ids, reset_src=reset_all, z_out=z, yrem_out=y, status_dev=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert np.array_equal(z.cpu().numpy(), wl.hidden_steps[0])          # restarted empty: z is the row itself
        egtp.plp_state_destroy(st_d)
    status.zero_()
    assert egtp.plp_step(ctx, st, lm, None, hs, alpha=-1.0, check=False) == egtp.EGTP_ERR_INVALID_ARG
    st_small = egtp.plp_state_create(ctx, 4, 128)
    assert egtp.plp_step(ctx, st_small, lm, None, hs, check=False) == egtp.EGTP_ERR_CAPACITY
    egtp.plp_state_destroy(st_small); egtp.plp_state_destroy(st)
    # host-buffer entry point over all steps against the oracle
    st = egtp.plp_state_create(ctx, 8, 128)
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head)
    y = torch.empty(8, dtype=torch.float32).pin_memory()
    sh = torch.zeros(1, dtype=torch.int32).pin_memory()
    for t in range(3):
        egtp.plp_step_host(ctx, st, lm, head.c, gu.host_tensor(wl.hidden_steps[t], "bf16"),
                           torch.from_numpy(wl.reset_src[t].copy()).pin_memory(), None, None, None, 0, 8, 1.0, y, sh)
        assert int(sh.item()) == 0
        gu.assert_length_close(y.numpy().astype(np.float64), ref["yrem"][t])
    egtp.plp_state_destroy(st)
    # the same steps handed over without waiting in between (copy of step t + 1 next to the kernels of step t),
    # each with its own pinned buffers; one wait at the end
    st = egtp.plp_state_create(ctx, 8, 128)
    hs_host = [gu.host_tensor(wl.hidden_steps[t], "bf16") for t in range(3)]
    rs_host = [torch.from_numpy(wl.reset_src[t].copy()).pin_memory() for t in range(3)]
    ys = [torch.full((8,), float("nan"), dtype=torch.float32).pin_memory() for _ in range(3)]
    shs = [torch.full((1,), 99, dtype=torch.int32).pin_memory() for _ in range(3)]
    for t in range(3):
        egtp.plp_step_host_async(ctx, st, lm, head.c, hs_host[t], rs_host[t], None, None, None, 0, 8, 1.0, ys[t], shs[t])
    torch.cuda.synchronize()
    for t in range(3):
        assert int(shs[t].item()) == 0
        gu.assert_length_close(ys[t].numpy().astype(np.float64), ref["yrem"][t])
    egtp.plp_state_destroy(st)


@pytest.mark.parametrize("slots", [40, 150])
def test_decode_loop_with_fp32_inputs(ctx, slots):
    # fp32 hidden states and weights: the LM-head kernel splits every operand into two tf32 parts (three MMAs per k
    # step); up to 128 rows take the one-row-tile decode shape, more rows the prompt shape
    rng = np.random.default_rng(slots)
    d, V, steps = 64, 1500, 4
    hs = (rng.standard_normal((steps, slots, d)) * 1.5).astype(np.float32)
    W = (rng.standard_normal((V, d)) * 0.3).astype(np.float32)
    reset = np.full((steps, slots), gen.RESET_KEEP, np.int32)
    reset[0] = gen.RESET_EMPTY
    reset[2, ::7] = gen.RESET_EMPTY
    head = gen.scaled_head(gen.make_head(31, d, 24, 1, "f32"), "f32")
    wl = gen.PlpWorkload("f32_decode", "f32", hs, reset, W, head)
    st, H, z, y = _run_plp(ctx, wl)
    follow = [0, 7, slots - 1]
    ref = orc.plp_run(hs, reset, W, head, slots=follow)
    assert np.abs(orc.logits(hs[0], W)).max() > 8           # logits large enough for a single tf32 rounding to show
    _compare(H, z, y, ref, follow)
    egtp.plp_state_destroy(st)
