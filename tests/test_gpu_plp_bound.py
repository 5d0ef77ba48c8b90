"""GPU parity of plp_step on a state bound to its head (plp_state_bind_head): W1 h' comes out of the LM-head
kernel as extra output columns and one kernel finishes the step.  Checked against the oracle, which knows nothing
of that shortcut (it recomputes Eq. 8 and the head from explicit token lists), and against the unbound route."""
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


def _run(ctx, wl: gen.PlpWorkload, bind=True, src=None, want_z=True, head=None, W=None):
    steps, slots, d = wl.steps, wl.slots, wl.d
    W = gu.dev_tensor(wl.W, wl.dtype) if W is None else W
    head = gu.DeviceHead(wl.head, wl.dtype) if head is None else head
    hs = gu.dev_tensor(wl.hidden_steps.reshape(-1, d), wl.dtype).reshape(steps, slots, d)
    reset = torch.from_numpy(wl.reset_src).cuda()
    st = egtp.plp_state_create(ctx, slots, d)
    if bind:
        egtp.plp_state_bind_head(st, head.c)
    lm = egtp.make_lm_head(W)
    f = dict(device="cuda", dtype=torch.float32)
    H = torch.zeros(steps, slots, **f)
    z = torch.zeros(steps, slots, d, **f)
    y = torch.full((steps, slots), float("nan"), **f)
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    sm, ss, sp, n_src = (None, None, None, 0) if src is None else src
    n0 = egtp.egtp_launch_count(ctx)
    for t in range(steps):
        egtp.plp_step(ctx, st, lm, head.c, hs[t], reset_src=reset[t], src_m=sm, src_s=ss, src_pooled=sp, n_src=n_src,
                      Hstep_out=H[t], z_out=z[t] if want_z else None, yrem_out=y[t], status_dev=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, egtp.status_string(int(status.item()))
    launches = egtp.egtp_launch_count(ctx) - n0
    to64 = lambda a: a.cpu().numpy().astype(np.float64)
    return st, to64(H), to64(z), to64(y), launches


def _compare(H, z, y, ref, slots):
    gu.assert_entropy_close(H[:, slots].ravel(), ref["H"].ravel())
    for t in range(z.shape[0]):
        gu.assert_pooled_close(z[t, slots], ref["z"][t])
    gu.assert_length_close(y[:, slots].ravel(), ref["yrem"].ravel())


@pytest.mark.parametrize("slots,V,m_h", [(130, 9000, 64),      # two row tiles; V not a multiple of 32: padded gap before W1
                                         (77, 4096 + 32, 40),   # one row tile; m_h not a multiple of 32
                                         (300, 7000, 96)])      # three row blocks of the prompt shape, 256-column boxes
def test_bound_decode_loop_matches_oracle(ctx, slots, V, m_h):
    wl = gen.config_plp_decode(slots=slots, steps=12, d=256, V=V, m_h=m_h, mu=1.5, sigma=0.8)
    assert (wl.reset_src[1:] == gen.RESET_EMPTY).sum() > 10
    st, H, z, y, launches = _run(ctx, wl)
    # first step projects the (empty) state: 3 launches (halves, GEMM, sum); then 2 launches per step (LM head, fused update + head)
    assert launches == 3 + 2 * wl.steps
    follow = sorted({0, 1, slots // 2, slots - 2, slots - 1})
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow)
    _compare(H, z, y, ref, follow)
    egtp.plp_state_destroy(st)
    # the same loop bound to a head that predicts hundreds of tokens (the configuration's own predicts fractions of one)
    big = gen.scaled_head(wl.head, "bf16")
    st_b, H_b, z_b, y_b, _ = _run(ctx, wl, head=gu.DeviceHead(big, "bf16"))
    ref_b = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, big, slots=follow, H_steps=ref["H"])
    assert np.abs(ref_b["yrem"]).min() > 100
    _compare(H_b, z_b, y_b, ref_b, follow)
    egtp.plp_state_destroy(st_b)
    # the unbound route on the same inputs: same entropies bit for bit (same vocabulary columns per tile only when
    # the column split is the same, so compare within tolerance), same lengths within tolerance
    st2, H2, z2, y2, launches2 = _run(ctx, wl, bind=False)
    assert launches2 == 4 * wl.steps
    gu.assert_entropy_close(H.ravel(), H2.ravel())
    assert np.abs(y - y2).max() <= 1e-3 * max(1.0, np.abs(y2).max())
    assert np.array_equal(z, z2) or np.abs(z - z2).max() <= 1e-5 * np.abs(z2).max()
    egtp.plp_state_destroy(st2)


def test_bound_decode_loop_in_single_cta_mode(ctx):
    # 129..256 rows: the default is the CTA-pair kernel with head columns; this is the one-CTA kernel with head columns
    wl = gen.config_plp_decode(slots=190, steps=8, d=256, V=6000 + 8, m_h=72, mu=1.5, sigma=0.8)
    egtp.egtp_set_lmhead_mode(ctx, egtp.EGTP_LMHEAD_SINGLE_CTA)
    try:
        st, H, z, y, launches = _run(ctx, wl)
    finally:
        egtp.egtp_set_lmhead_mode(ctx, egtp.EGTP_LMHEAD_AUTO)
    assert launches == 3 + 2 * wl.steps
    follow = [0, 127, 128, 189]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow)
    _compare(H, z, y, ref, follow)
    egtp.plp_state_destroy(st)


def test_bound_bins_head_without_z(ctx):
    wl = gen.config_plp_decode(slots=140, steps=6, d=256, V=5000, m_h=64, mu=1.5, sigma=0.5)
    head_bins = gen.make_head(11, 256, 64, 20, "bf16", mode=gen.HEAD_BINS)
    wl = gen.PlpWorkload("bins", "bf16", wl.hidden_steps, wl.reset_src, wl.W, head_bins)
    st, H, z, y, _ = _run(ctx, wl, want_z=False)
    assert np.all(z == 0)            # z_out was not requested: nothing is written
    follow = [0, 128, 139]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow)
    gu.assert_length_close(y[:, follow].ravel(), ref["yrem"].ravel())
    c = np.asarray(head_bins.centres, dtype=np.float64)
    assert np.all(y >= c.min() - 1e-3) and np.all(y <= c.max() + 1e-3)
    egtp.plp_state_destroy(st)


def test_bound_rl_group_continues_from_egtp_rows(ctx):
    wl = gen.config_rl_group(prompts=5, group=4, steps=8, d=256, V=7000, m_h=64, min_len=3, max_len=200)
    eg = wl.prompts
    res = gu.run_egtp(ctx, eg)
    ref_eg = orc.egtp_predict(eg.hidden, eg.offsets, eg.W, eg.head)
    src = (torch.from_numpy(res["state_m"].astype(np.float32)).cuda(), torch.from_numpy(res["state_s"].astype(np.float32)).cuda(),
           torch.from_numpy(res["pooled"].astype(np.float32)).cuda(), eg.B)
    st, H, z, y, _ = _run(ctx, wl, src=src)
    follow = [0, 3, 4, 19]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow,
                      prompts=dict(hidden=eg.hidden, offsets=eg.offsets, H=ref_eg["H"]))
    _compare(H, z, y, ref, follow)
    egtp.plp_state_destroy(st)


def test_projection_is_rebuilt_after_other_routes(ctx):
    # bound steps, then an unbound step with another head, an import, and bound steps again: the oracle's
    # answer for the original head must come out every time the bound head is used
    wl = gen.config_plp_decode(slots=40, steps=9, d=128, V=3000, m_h=32, mu=3.0, sigma=0.3)
    W = gu.dev_tensor(wl.W, "bf16"); lm = egtp.make_lm_head(W)
    head = gu.DeviceHead(wl.head, "bf16")
    other = gu.DeviceHead(gen.make_head(99, 128, 48, 1, "bf16"), "bf16")
    hs = gu.dev_tensor(wl.hidden_steps.reshape(-1, 128), "bf16").reshape(wl.steps, 40, 128)
    reset = torch.from_numpy(wl.reset_src).cuda()
    st = egtp.plp_state_create(ctx, 40, 128)
    egtp.plp_state_bind_head(st, head.c)
    y = torch.full((wl.steps, 40), float("nan"), device="cuda")
    y_other = torch.zeros(40, device="cuda")
    m = torch.empty(40, device="cuda"); s = torch.empty(40, device="cuda"); acc = torch.empty(40, 128, device="cuda")
    for t in range(wl.steps):
        if t == 3:       # another head: ordinary route, the projection goes stale
            egtp.plp_step(ctx, st, lm, other.c, hs[t], reset_src=reset[t], yrem_out=y_other)
            continue
        if t == 6:       # checkpoint and restore into the same state
            egtp.plp_state_export(st, m, s, acc)
            egtp.plp_state_import(st, m, s, acc)
        egtp.plp_step(ctx, st, lm, head.c, hs[t], reset_src=reset[t], yrem_out=y[t])
    torch.cuda.synchronize()
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head)
    keep = [t for t in range(wl.steps) if t != 3]
    gu.assert_length_close(y.cpu().numpy().astype(np.float64)[keep].ravel(), ref["yrem"][keep].ravel())
    egtp.plp_state_destroy(st)


def test_bind_rejects_fp32_heads(ctx):
    st = egtp.plp_state_create(ctx, 8, 128)
    head32 = gu.DeviceHead(gen.make_head(5, 128, 32, 1, "f32"), "f32")
    assert egtp.plp_state_bind_head(st, head32.c, check=False) == egtp.EGTP_ERR_UNSUPPORTED
    egtp.plp_state_destroy(st)


def test_bound_step_replayed_from_a_cuda_graph_equals_eager_steps(ctx):
    # the decode step is two launches (the second one with programmatic stream serialization); captured once and
    # replayed with new tokens copied into fixed buffers it must give bit for bit what eager calls give
    wl = gen.config_plp_decode(slots=150, steps=7, d=256, V=5000, m_h=64, mu=3.0, sigma=0.3)
    W = gu.dev_tensor(wl.W, "bf16"); lm = egtp.make_lm_head(W)
    head = gu.DeviceHead(wl.head, "bf16")
    hs = gu.dev_tensor(wl.hidden_steps.reshape(-1, 256), "bf16").reshape(wl.steps, 150, 256)
    reset = torch.from_numpy(wl.reset_src).cuda()
    st_e, st_g = egtp.plp_state_create(ctx, 150, 256), egtp.plp_state_create(ctx, 150, 256)
    egtp.plp_state_bind_head(st_e, head.c); egtp.plp_state_bind_head(st_g, head.c)
    y_e = torch.zeros(wl.steps, 150, device="cuda"); y_g = torch.zeros(wl.steps, 150, device="cuda")
    status = torch.zeros(1, device="cuda", dtype=torch.int32)
    for t in range(wl.steps):
        egtp.plp_step(ctx, st_e, lm, head.c, hs[t], reset_src=reset[t], yrem_out=y_e[t], status_dev=status)
    # step 0 eagerly (it also projects the empty state, which is not part of the steady-state graph)
    h_buf, r_buf, y_buf = hs[0].clone(), reset[0].clone(), torch.zeros(150, device="cuda")
    egtp.plp_step(ctx, st_g, lm, head.c, h_buf, reset_src=r_buf, yrem_out=y_buf, status_dev=status)
    y_g[0].copy_(y_buf)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        egtp.plp_step(ctx, st_g, lm, head.c, h_buf, reset_src=r_buf, yrem_out=y_buf, status_dev=status,
                      stream=torch.cuda.current_stream().cuda_stream)
    for t in range(1, wl.steps):
        h_buf.copy_(hs[t]); r_buf.copy_(reset[t])
        graph.replay()
        y_g[t].copy_(y_buf)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(y_e, y_g)
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=[0, 149])
    gu.assert_length_close(y_g.cpu().numpy().astype(np.float64)[:, [0, 149]].ravel(), ref["yrem"].ravel())
    egtp.plp_state_destroy(st_e); egtp.plp_state_destroy(st_g)


def test_bound_projection_does_not_drift_over_a_long_sequence(ctx):
    # 400 steps without a restart: P = W1 acc is advanced incrementally all the way; the oracle recomputes the pool
    # and the head from the whole token list at every step
    wl = gen.config_plp_decode(slots=8, steps=400, d=128, V=2000, m_h=48, mu=12.0, sigma=0.1)
    assert (wl.reset_src[1:] == gen.RESET_KEEP).all()
    st, H, z, y, _ = _run(ctx, wl)
    follow = [0, 7]
    ref = orc.plp_run(wl.hidden_steps, wl.reset_src, wl.W, wl.head, slots=follow)
    err = np.abs(y[:, follow] - ref["yrem"])
    assert err.max() <= 1e-3 * max(1.0, np.abs(ref["yrem"]).max()), err.max()
    assert err[-50:].max() <= 2.0 * max(err[:50].max(), 1e-5) + 1e-4       # no growth along the sequence
    for t in (0, 199, 399):
        gu.assert_pooled_close(z[t, follow], ref["z"][t])
    egtp.plp_state_destroy(st)


def test_two_contexts_on_two_streams_do_not_disturb_each_other():
    # two contexts (each with its own workspace) driven from two CUDA streams at the same time give bit for bit
    # what each gives alone: the library keeps no per-call state outside the context
    wl = gen.config_plp_decode(slots=140, steps=6, d=256, V=6000, m_h=64, mu=2.0, sigma=0.5)
    W = gu.dev_tensor(wl.W, "bf16"); lm = egtp.make_lm_head(W)
    head = gu.DeviceHead(wl.head, "bf16")
    hs = gu.dev_tensor(wl.hidden_steps.reshape(-1, 256), "bf16").reshape(wl.steps, 140, 256)
    reset = torch.from_numpy(wl.reset_src).cuda()

    def run(ctxs, streams):
        ys, sts, stat = [], [], []
        for c in ctxs:
            st = egtp.plp_state_create(c, 140, 256)
            egtp.plp_state_bind_head(st, head.c)
            sts.append(st); ys.append(torch.zeros(wl.steps, 140, device="cuda"))
            stat.append(torch.zeros(1, device="cuda", dtype=torch.int32))
        torch.cuda.synchronize()
        for t in range(wl.steps):
            for k, c in enumerate(ctxs):
                with torch.cuda.stream(streams[k]):
                    egtp.plp_step(c, sts[k], lm, head.c, hs[t], reset_src=reset[t], yrem_out=ys[k][t], status_dev=stat[k])
        torch.cuda.synchronize()
        for st in sts:
            egtp.plp_state_destroy(st)
        assert all(int(s.item()) == 0 for s in stat)
        return ys

    c1 = egtp.egtp_create(0, max_tokens=1024, max_batch=256, max_d=256, max_V=8192)
    c2 = egtp.egtp_create(0, max_tokens=1024, max_batch=256, max_d=256, max_V=8192)
    try:
        alone = run([c1], [torch.cuda.current_stream()])[0]
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        both = run([c1, c2], [s1, s2])
    finally:
        egtp.egtp_destroy(c1); egtp.egtp_destroy(c2)
    assert torch.equal(both[0], alone) and torch.equal(both[1], alone)
