"""GPU parity: egtp_predict through the C ABI against the fp64 oracle on the same seeded inputs."""
import math

import numpy as np
import pytest
import torch

from oracle import egtp_oracle as orc
from paper_2602_11812_b200 import binding as egtp
from paper_2602_11812_b200 import inputs as gen
from tests import gpu_util as gu
from tests.golden_io import load

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = egtp.egtp_create(0, max_tokens=16384, max_batch=256, max_d=2048, max_V=40000)
    yield c
    egtp.egtp_destroy(c)


def _check_all(res, ref, wl):
    assert res["status"] == 0
    assert np.array_equal(res["seg_id"], ref["seg_id"])                 # bit-exact segment indexing
    gu.assert_entropy_close(res["H"], ref["H"])
    assert np.all(np.abs(res["weights"] - ref["weights"]) <= 5e-3 * ref["weights"] + 1e-9)
    gu.assert_pooled_close(res["pooled"], ref["pooled"])
    gu.assert_length_close(res["yhat"], ref["yhat"])
    ne = np.diff(wl.offsets) > 0
    assert np.allclose(res["state_m"][ne], ref["state_m"][ne], rtol=1e-3)
    assert np.allclose(res["state_s"][ne], ref["state_s"][ne], rtol=5e-3)


def test_tiny_config_matches_oracle_and_golden(ctx):
    wl = gen.config_tiny()
    ref = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, wl.alpha)
    res = gu.run_egtp(ctx, wl)
    _check_all(res, ref, wl)
    big = gen.scaled_head(wl.head, "f32")                      # the same head rescaled to predict hundreds of tokens
    ref_big = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, big, wl.alpha, H=ref["H"])
    assert np.abs(ref_big["yhat"]).min() > 100
    _check_all(gu.run_egtp(ctx, wl, head_dev=gu.DeviceHead(big, "f32")), ref_big, wl)
    gu.assert_entropy_close(res["H"], load("egtp_tiny_H.txt"))
    gu.assert_pooled_close(res["pooled"], load("egtp_tiny_pooled.txt", (4, 256)))
    gu.assert_length_close(res["yhat"], load("egtp_tiny_yhat.txt"))


def test_tiny_config_bins_head(ctx):
    wl = gen.config_tiny(gen.HEAD_BINS)
    ref = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, wl.alpha)
    res = gu.run_egtp(ctx, wl, want_phat=True)
    _check_all(res, ref, wl)
    gu.assert_length_close(res["yhat"], load("egtp_tiny_bins_yhat.txt"))
    assert np.allclose(res["phat"], ref["phat"], atol=2e-4)
    assert np.allclose(res["phat"].sum(axis=1), 1.0, atol=1e-5)


@pytest.mark.parametrize("dtype,V,d", [("bf16", 5000, 512), ("bf16", 256, 64), ("bf16", 1000, 2048),
                                       ("f32", 777, 96), ("bf16", 33000, 256)])
def test_uniform_logits_give_ln_V(ctx, dtype, V, d):
    # W = 0: every entropy is ln V exactly.  V not a multiple of the 256-wide tile catches unmasked padding.
    rng = np.random.default_rng(0)
    lengths = [5, 130, 1, 200]
    hidden = gen._maybe_round(rng.standard_normal((sum(lengths), d)).astype(np.float32), dtype)
    head = gen.make_head(1, d, 32, 1, dtype)
    wl = gen.EgtpWorkload("uniform", dtype, hidden, gen.offsets_from_lengths(lengths), np.zeros((V, d), np.float32), head)
    res = gu.run_egtp(ctx, wl)
    assert res["status"] == 0
    assert np.all(np.abs(res["H"] - math.log(V)) <= 1e-4 * math.log(V))
    # equal entropies: the pool is the plain mean of the prompt's rows
    off = wl.offsets
    for b in range(4):
        mean = hidden[off[b]:off[b + 1]].astype(np.float64).mean(axis=0)
        assert np.abs(res["pooled"][b] - mean).max() <= 2e-3 * np.abs(mean).max() + 1e-6


def test_two_level_closed_form_and_one_hot(ctx):
    # hidden = e_0, W[v, 0] = a for v < k else 0:  H = ln Z - k a e^a / Z, Z = k e^a + V - k
    V, d = 4999, 64
    cases = [(3, 5.0), (100, 7.0), (4000, -2.0), (1, 40.0)]
    rows, Ws = [], None
    hidden = np.zeros((len(cases), d), np.float32)
    expect = []
    res_all = []
    for i, (k, a) in enumerate(cases):
        h = np.zeros((1, d), np.float32)
        h[0, 0] = 1.0
        W = np.zeros((V, d), np.float32)
        W[:k, 0] = a
        wl = gen.EgtpWorkload("two_level", "bf16", h, np.array([0, 1], np.int32), W, gen.make_head(1, d, 16, 1, "bf16"))
        res = gu.run_egtp(ctx, wl)
        Z = k * math.exp(a) + V - k
        exp_H = math.log(Z) - k * a * math.exp(a) / Z
        assert res["status"] == 0
        assert abs(res["H"][0] - exp_H) <= 1e-3 * abs(exp_H) + 1e-5, (k, a, res["H"][0], exp_H)
        assert np.allclose(res["pooled"][0], h[0], atol=1e-6)          # single token: identity


def test_mid_config_scaled(ctx):
    # the mid configuration's recipe (lognormal lengths, 1 % outlier channels x 20, bf16) at reduced d and V;
    # 32 ragged prompts spanning many 128-row tiles, V not a multiple of 128
    wl = gen.config_mid(V=20000 + 72, d=512, m_h=128)
    ref = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, wl.alpha)
    res = gu.run_egtp(ctx, wl)
    _check_all(res, ref, wl)
    assert ref["H"].std() > 0.05                                        # weights are genuinely non-uniform
    big = gen.scaled_head(wl.head, "bf16")                              # predictions of hundreds of tokens
    ref_big = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, big, wl.alpha, H=ref["H"])
    assert np.abs(ref_big["yhat"]).min() > 100
    _check_all(gu.run_egtp(ctx, wl, head_dev=gu.DeviceHead(big, "bf16")), ref_big, wl)
    # the number of vocabulary chunks is a tuning knob: one chunk, an odd count and more chunks than tiles (clamped)
    # give the same result up to summation order
    T, planned = wl.T, egtp.egtp_lmhead_plan(ctx, wl.T, wl.d, wl.V, egtp.EGTP_BF16)["chunks"]
    try:
        for chunks in (1, 7, 500):
            egtp.egtp_set_lmhead_chunks(ctx, chunks)
            got = egtp.egtp_lmhead_plan(ctx, T, wl.d, wl.V, egtp.EGTP_BF16)["chunks"]
            assert got == min(chunks, got) and (chunks > 79 or got == chunks)      # 20072 columns = 79 tiles
            res_c = gu.run_egtp(ctx, wl)
            _check_all(res_c, ref, wl)
            assert np.abs(res_c["H"] - res["H"]).max() < 1e-4
    finally:
        egtp.egtp_set_lmhead_chunks(ctx, 0)
    assert egtp.egtp_lmhead_plan(ctx, T, wl.d, wl.V, egtp.EGTP_BF16)["chunks"] == planned


def test_head_on_tensor_cores_keeps_fp32_accuracy(ctx):
    # bf16 head weights: layer 1 runs on the tensor cores with every fp32 input row split into two bf16 halves.
    # Fed the device's own pooled vectors, the oracle's head must agree to ~1e-5, far inside the 0.5-token bar
    # (a single bf16 rounding of the inputs would be off by ~1e-3 relative).
    wl = gen.config_mid(V=4096 + 8, d=512, m_h=264, B=40, max_len=120)
    big = gen.make_head(21, 512, 264, 1, "bf16")
    big.W2 *= 64.0; big.b2 += 300.0                      # predictions of a few hundred tokens
    big.W2[:] = gen.round_to_bf16(big.W2)
    wl.head = big
    res = gu.run_egtp(ctx, wl)
    assert res["status"] == 0
    y_ref, _ = orc.head_forward(res["pooled"], big.W1, big.b1, big.W2, big.b2)
    assert np.abs(y_ref).max() > 100
    err = np.abs(res["yhat"] - y_ref)
    assert err.max() <= 1e-4 * np.abs(y_ref).max(), err.max()
    # bins head (K = 20) through the same route
    bins = gen.make_head(22, 512, 264, 20, "bf16", mode=gen.HEAD_BINS)
    wl.head = bins
    res = gu.run_egtp(ctx, wl, want_phat=True)
    y_ref, p_ref = orc.head_forward(res["pooled"], bins.W1, bins.b1, bins.W2, bins.b2, mode=bins.mode, centres=bins.centres)
    assert np.abs(res["phat"] - p_ref).max() <= 1e-5 and np.abs(res["yhat"] - y_ref).max() <= 0.05


def test_segment_edge_cases(ctx):
    # leading / trailing tokens outside every prompt, empty prompts, boundaries on and next to a 128-row tile
    # edge and a 64-token pooling chunk edge, a one-token prompt
    rng = np.random.default_rng(3)
    d, V = 128, 3000
    off = np.array([3, 3, 64, 128, 129, 129, 257, 300, 300, 511, 640], np.int32)
    T = 650
    hidden = gen._maybe_round(rng.standard_normal((T, d)).astype(np.float32) * 2, "bf16")
    W = gen.make_lm_head(11, V, d, "bf16") * np.float32(3.0)
    W = gen.round_to_bf16(W)
    head = gen.make_head(12, d, 48, 1, "bf16")
    wl = gen.EgtpWorkload("edges", "bf16", hidden, off, W, head)
    ref = orc.egtp_predict(hidden, off, W, head)
    res = gu.run_egtp(ctx, wl)
    _check_all(res, ref, wl)
    for b in (0, 4, 7):                                                 # empty prompts
        assert np.all(res["pooled"][b] == 0) and res["state_s"][b] == 0 and res["state_m"][b] == -np.inf
    assert np.all(res["weights"][:3] == 0) and np.all(res["weights"][640:] == 0)


def test_alpha_and_determinism(ctx):
    wl = gen.config_mid(V=4096, d=256, m_h=64, B=8)
    wl.alpha = 0.5
    ref = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, wl.alpha)
    r1 = gu.run_egtp(ctx, wl)
    r2 = gu.run_egtp(ctx, wl)
    _check_all(r1, ref, wl)
    for k in ("H", "weights", "pooled", "yhat", "state_m", "state_s"):
        assert np.array_equal(r1[k], r2[k]), k                          # run-to-run bitwise determinism
    # a sharp and a flat temperature: H/alpha up to ~170 (the weights span e^-100..1 inside one prompt, rescaled
    # between 64-token chunks), and weights that are nearly uniform
    for alpha in (0.05, 20.0):
        wl.alpha = alpha
        _check_all(gu.run_egtp(ctx, wl), orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, alpha, H=ref["H"]), wl)


def test_errors_are_reported_not_fatal(ctx):
    wl = gen.config_tiny()
    bad = wl.offsets.copy()
    bad[2] = bad[1] - 1                                                 # decreasing offsets: device-side error
    res = gu.run_egtp(ctx, wl, offsets=bad)
    assert res["status"] == egtp.EGTP_ERR_BAD_OFFSETS
    bad2 = wl.offsets.copy()
    bad2[-1] = wl.T + 1
    assert gu.run_egtp(ctx, wl, offsets=bad2)["status"] == egtp.EGTP_ERR_BAD_OFFSETS
    # host-side errors: returned at once
    W = gu.dev_tensor(wl.W, wl.dtype)
    hidden = gu.dev_tensor(wl.hidden, wl.dtype)
    off = torch.from_numpy(wl.offsets).cuda()
    lm = egtp.make_lm_head(W)
    y = torch.empty(4, device="cuda")
    hd = gu.DeviceHead(wl.head, wl.dtype)
    assert egtp.egtp_predict(ctx, lm, hd.c, hidden, off, 4, wl.T, alpha=0.0, yhat_out=y, check=False) == egtp.EGTP_ERR_INVALID_ARG
    assert egtp.egtp_predict(ctx, lm, hd.c, hidden, off, 4, 10**6, yhat_out=y, check=False) == egtp.EGTP_ERR_CAPACITY
    assert egtp.egtp_predict(ctx, lm, None, hidden, off, 4, wl.T, yhat_out=y, check=False) == egtp.EGTP_ERR_INVALID_ARG
    lm_bad = egtp.make_lm_head(W)
    lm_bad.d = 250
    assert egtp.egtp_predict(ctx, lm_bad, None, hidden, off, 4, wl.T, check=False) == egtp.EGTP_ERR_UNSUPPORTED
    # and the context still works afterwards
    ref = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, wl.alpha)
    _check_all(gu.run_egtp(ctx, wl), ref, wl)


@pytest.mark.parametrize("B", [6, 32])
def test_host_buffer_entry_point(ctx, B):
    # B = 32 gives 9555 tokens: the copy is split into four row ranges that overlap the LM-head kernel
    wl = gen.config_mid(V=3000, d=256, m_h=64, B=B)
    ref = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, wl.alpha)
    W = gu.dev_tensor(wl.W, wl.dtype)
    hd = gu.DeviceHead(wl.head, wl.dtype)
    hidden_host = torch.from_numpy(gen.bf16_bits(wl.hidden).view(np.int16)).view(torch.bfloat16).pin_memory()
    off_host = torch.from_numpy(wl.offsets).pin_memory()
    y = torch.empty(wl.B, dtype=torch.float32).pin_memory()
    pooled = torch.empty(wl.B, wl.d, dtype=torch.float32).pin_memory()
    st = torch.full((1,), 99, dtype=torch.int32).pin_memory()
    egtp.egtp_predict_host(ctx, egtp.make_lm_head(W), hd.c, hidden_host, off_host, wl.B, wl.T, 1.0, y, pooled, st)
    assert int(st.item()) == 0
    gu.assert_pooled_close(pooled.numpy().astype(np.float64), ref["pooled"])
    gu.assert_length_close(y.numpy().astype(np.float64), ref["yhat"])


@pytest.mark.parametrize("mode,tile_cols", [(egtp.EGTP_LMHEAD_CTA_PAIRS, 256), (egtp.EGTP_LMHEAD_CTA_PAIRS_WIDE, 512)])
def test_cta_pair_tile_shape_matches_oracle(mode, tile_cols):
    # the same checks with the LM-head kernel switched to clusters of two CTAs (256 x 256 tiles with two accumulator
    # sets, or 256 x 512 tiles with one set whose two halves are handed back to the MMA warp one after the other)
    c = egtp.egtp_create(0, max_tokens=16384, max_batch=256, max_d=2048, max_V=40000)
    try:
        egtp.egtp_set_lmhead_mode(c, mode)
        plan = egtp.egtp_lmhead_plan(c, 9555, 512, 20072, egtp.EGTP_BF16)
        assert (plan["rows_per_block"], plan["tile_cols"]) == (256, tile_cols)
        wl = gen.config_mid(V=20000 + 72, d=512, m_h=128)
        ref = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, wl.alpha)
        _check_all(gu.run_egtp(c, wl), ref, wl)
        # odd number of 128-row tiles, V not a multiple of 256, W = 0: every entropy is ln V
        rng = np.random.default_rng(1)
        hidden = gen.round_to_bf16(rng.standard_normal((3 * 128 + 5, 256)).astype(np.float32))
        wl0 = gen.EgtpWorkload("uniform", "bf16", hidden, gen.offsets_from_lengths([200, 189]), np.zeros((33000, 256), np.float32),
                               gen.make_head(1, 256, 32, 1, "bf16"))
        res = gu.run_egtp(c, wl0)
        assert res["status"] == 0 and np.all(np.abs(res["H"] - math.log(33000)) <= 1e-4 * math.log(33000))
        # fp32 inputs always run one CTA per SM (operands split into two tf32 parts in shared memory), whatever the mode
        wt = gen.config_tiny()
        big = gen.EgtpWorkload("tiny_x3", "f32", np.concatenate([wt.hidden] * 3), gen.offsets_from_lengths([159, 159, 159]),
                               wt.W, wt.head)
        _check_all(gu.run_egtp(c, big), orc.egtp_predict(big.hidden, big.offsets, big.W, big.head), big)
        assert egtp.load().egtp_set_lmhead_mode(c, 7) == egtp.EGTP_ERR_INVALID_ARG
    finally:
        egtp.egtp_destroy(c)


def test_many_tokens_small_model_64bit_indexing():
    # 300k tokens (2343.75 row tiles, > 2^31 / d / ... byte offsets in play) against a small LM head:
    # entropies are checked on sampled tokens, pooling against fp64 pooling with the device's own entropies
    T, d, V, B = 300_000, 64, 520, 40
    rng = np.random.default_rng(11)
    lengths = rng.multinomial(T - 1000, np.ones(B) / B)
    off = np.concatenate([[500], 500 + np.cumsum(lengths)]).astype(np.int32)
    hidden = gen.make_hidden(21, T, d, "bf16")
    W = gen.round_to_bf16(gen.make_lm_head(22, V, d, "bf16") * np.float32(6.0))
    head = gen.make_head(23, d, 32, 1, "bf16")
    wl = gen.EgtpWorkload("many_tokens", "bf16", hidden, off, W, head)
    c = egtp.egtp_create(0, max_tokens=T, max_batch=64, max_d=d, max_V=V)
    try:
        res = gu.run_egtp(c, wl)
    finally:
        egtp.egtp_destroy(c)
    assert res["status"] == 0
    idx = np.concatenate([[0, 1, T - 1, T - 2, 127, 128, 299_904], rng.choice(T, size=200, replace=False)])
    gu.assert_entropy_close(res["H"][idx], orc.token_entropy(hidden[idx], W))
    ref_seg = np.searchsorted(off, np.arange(T), side="right").astype(np.int32) - 1
    ref_seg[(np.arange(T) < off[0]) | (np.arange(T) >= off[-1])] = -1
    assert np.array_equal(res["seg_id"], ref_seg)
    for b in (0, 17, B - 1):
        s, e = off[b], off[b + 1]
        w = orc.entropy_weights(res["H"][s:e])
        gu.assert_pooled_close(res["pooled"][[b]], orc.pool(hidden[s:e], w)[None, :])
    y_ref, _ = orc.head_forward(res["pooled"], head.W1, head.b1, head.W2, head.b2)
    gu.assert_length_close(res["yhat"], y_ref)


def test_fewer_than_16_rows_in_fp32_and_with_a_row_stride(ctx):
    # batches of fewer than 16 rows go through a zero-padded 16-row staging buffer: fp32 rows (split-tf32 tensor-core path),
    # and bf16 rows that are 3 * d elements apart in memory
    rng = np.random.default_rng(77)
    d, V = 64, 500
    hidden = (rng.standard_normal((7, d)) * 1.5).astype(np.float32)
    W = (rng.standard_normal((V, d)) * 0.3).astype(np.float32)
    head = gen.make_head(6, d, 24, 1, "f32")
    wl = gen.EgtpWorkload("few_f32", "f32", hidden, gen.offsets_from_lengths([3, 4]), W, head)
    res = gu.run_egtp(ctx, wl)
    # fp32 operands are split into two tf32 parts each (three MMAs per k step): logits of a few units, where a
    # single tf32 rounding of the operands would cost 2-3e-3 of entropy, meet the usual tolerance against the oracle
    ref = orc.egtp_predict(hidden, wl.offsets, W, head)
    assert np.abs(orc.logits(hidden, W)).max() > 8 and ref["H"].min() < 5.0
    _check_all(res, ref, wl)
    assert np.abs(res["H"] - ref["H"]).max() <= 1e-4 * ref["H"].max()
    hb = gen.round_to_bf16(hidden); Wb = gen.round_to_bf16(W)
    wide = torch.zeros(7, 3 * d, device="cuda", dtype=torch.bfloat16)
    wide[:, :d] = gu.dev_tensor(hb, "bf16")
    wide[:, d:] = 9.0                                            # poison beside the rows
    H = torch.zeros(7, device="cuda")
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    lm = egtp.make_lm_head(gu.dev_tensor(Wb, "bf16"))
    off = torch.tensor([0, 7], dtype=torch.int32, device="cuda")
    egtp.egtp_predict(ctx, lm, None, wide[:, :d], off, 1, 7, 1.0, H_out=H, status_dev=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    gu.assert_entropy_close(H.cpu().numpy().astype(np.float64), orc.token_entropy(hb, Wb))


@pytest.mark.parametrize("T,d,V", [(3, 16, 40), (129, 32, 300), (256, 48, 1000), (257, 80, 1000), (128, 272, 31), (1, 2048, 9)])
def test_small_and_boundary_shapes(ctx, T, d, V):
    # row counts on both sides of the 128 / 256-row launch shapes, hidden sizes that are not multiples of
    # the 64-element k block, vocabularies smaller than one tile
    rng = np.random.default_rng(T * 1000 + d + V)
    lengths = [T] if T < 4 else [T // 3, T - T // 3 - 1, 1]
    hidden = gen.round_to_bf16((rng.standard_normal((T, d)) * 1.5).astype(np.float32))
    W = gen.round_to_bf16((rng.standard_normal((V, d)) * (2.0 / np.sqrt(d))).astype(np.float32))
    head = gen.make_head(5, d, 24, 1, "bf16")
    wl = gen.EgtpWorkload("small", "bf16", hidden, gen.offsets_from_lengths(lengths), W, head)
    ref = orc.egtp_predict(hidden, wl.offsets, W, head)
    _check_all(gu.run_egtp(ctx, wl), ref, wl)


def test_bounded_wait_reports_timeout_and_context_survives(ctx):
    # a wait on a barrier that nothing signals must end by itself with an error status (no trap, no hang)
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    egtp.egtp_selftest_wait_timeout(ctx, 50, status)
    t1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == egtp.EGTP_ERR_DEVICE_TIMEOUT
    assert 40.0 <= t0.elapsed_time(t1) <= 500.0                         # the 50 ms limit, not the 4 s production limit
    assert egtp.status_string(egtp.EGTP_ERR_DEVICE_TIMEOUT).startswith("a bounded wait")
    # a non-zero status word turns a following call into a no-op instead of computing on top of a failure ...
    wl = gen.config_tiny()
    H = torch.full((wl.T,), -1.0, device="cuda")
    W = gu.dev_tensor(wl.W, wl.dtype); hidden = gu.dev_tensor(wl.hidden, wl.dtype)
    off = torch.from_numpy(wl.offsets).cuda()
    egtp.egtp_predict(ctx, egtp.make_lm_head(W), None, hidden, off, wl.B, wl.T, H_out=H, status_dev=status)
    torch.cuda.synchronize()
    assert torch.all(H == -1.0) and int(status.item()) == egtp.EGTP_ERR_DEVICE_TIMEOUT
    # ... and with a cleared word the same context works as before
    ref = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, wl.alpha)
    _check_all(gu.run_egtp(ctx, wl), ref, wl)
    assert egtp.egtp_selftest_wait_timeout(ctx, 0, status, check=False) == egtp.EGTP_ERR_INVALID_ARG


def test_launch_count_of_a_prediction_and_context_without_host_staging():
    # a whole prediction is six launches (LM head, merge + offsets check + segment ids, pooling, combine + head input,
    # head layer 1, head output); a context created without host staging holds max_tokens * max_d * 4 bytes less,
    # computes the same, and refuses the host-buffer entry points
    wl = gen.config_mid(V=3000, d=256, m_h=64, B=8)
    ref = orc.egtp_predict(wl.hidden, wl.offsets, wl.W, wl.head, wl.alpha)
    full = egtp.egtp_create(0, 4096, 64, 256, 4096)
    lean = egtp.egtp_create_ex(0, 4096, 64, 256, 4096, egtp.EGTP_CREATE_NO_HOST_STAGING)
    try:
        assert egtp.egtp_workspace_bytes(full) - egtp.egtp_workspace_bytes(lean) == 4096 * 256 * 4
        _check_all(gu.run_egtp(lean, wl), ref, wl)
        W = gu.dev_tensor(wl.W, wl.dtype); hidden = gu.dev_tensor(wl.hidden, wl.dtype)
        hd = gu.DeviceHead(wl.head, wl.dtype)
        off = torch.from_numpy(wl.offsets).cuda()
        y = torch.empty(wl.B, device="cuda")
        status = torch.zeros(1, device="cuda", dtype=torch.int32)
        n0 = egtp.egtp_launch_count(lean)
        egtp.egtp_predict(lean, egtp.make_lm_head(W), hd.c, hidden, off, wl.B, wl.T, 1.0, yhat_out=y, status_dev=status)
        torch.cuda.synchronize()
        assert egtp.egtp_launch_count(lean) - n0 == 6 and int(status.item()) == 0
        gu.assert_length_close(y.cpu().numpy().astype(np.float64), ref["yhat"])
        hidden_host = gu.host_tensor(wl.hidden, wl.dtype)
        off_host = torch.from_numpy(wl.offsets).pin_memory()
        yh = torch.empty(wl.B, dtype=torch.float32).pin_memory()
        st = torch.zeros(1, dtype=torch.int32).pin_memory()
        assert egtp.egtp_predict_host(lean, egtp.make_lm_head(W), hd.c, hidden_host, off_host, wl.B, wl.T, 1.0, yh, None, st,
                                      check=False) == egtp.EGTP_ERR_UNSUPPORTED
        assert egtp.egtp_create_ex(0, 4096, 64, 256, 4096, flags=2, check=False) == egtp.EGTP_ERR_INVALID_ARG
    finally:
        egtp.egtp_destroy(full); egtp.egtp_destroy(lean)
