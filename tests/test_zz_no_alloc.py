"""egtp_head_forward_static: the head for callers that are not allowed to allocate GPU memory.

A serving engine that pre-sizes its memory pool, or a plugin living inside another runtime,
cannot call cudaMalloc and so cannot create an egtp context.  This entry point runs the head with
its scratch in a fixed array inside the library.  The test feeds it the pooled vectors that
egtp_predict produced and checks its predictions against egtp_predict's own and against the fp64
oracle's head on those same vectors, twice in a row (the second call reuses the scratch the first
one left behind, with a different head shape and mode); the amount of free device memory must not
move across a call.  Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest
import torch

from oracle import egtp_oracle as orc
from paper_2602_11812_b200 import binding as egtp
from paper_2602_11812_b200 import inputs as gen
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _reference_through_context(ctx, wl, want_phat):
    res = gu.run_egtp(ctx, wl, want_phat=want_phat)
    assert res["status"] == 0
    return res


def test_static_head_matches_context_head_on_two_calls_in_a_row():
    ctx = egtp.egtp_create(0, max_tokens=8192, max_batch=64, max_d=512, max_V=8192)
    try:
        wl1 = gen.config_mid(V=4096 + 40, d=512, m_h=128, B=24, max_len=300)          # scalar head, bf16 weights
        wl2 = gen.config_tiny(gen.HEAD_BINS)                                            # K = 20 bins, fp32 weights
        ref1 = _reference_through_context(ctx, wl1, False)
        ref2 = _reference_through_context(ctx, wl2, True)
    finally:
        egtp.egtp_destroy(ctx)

    # a third head that predicts hundreds of tokens, so that the relative part of the length tolerance bites
    cases = [(wl1, wl1.head, ref1), (wl2, wl2.head, ref2), (wl1, gen.scaled_head(wl1.head, "bf16"), ref1)]
    for n, (wl, hp, ref) in enumerate(cases):
        head = gu.DeviceHead(hp, wl.dtype)
        z32 = ref["pooled"].astype(np.float32)
        z = torch.from_numpy(z32).cuda()
        y = torch.full((wl.B,), float("nan"), device="cuda")
        phat = torch.full((wl.B, head.d_out), float("nan"), device="cuda") if hp.mode == gen.HEAD_BINS else None
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        egtp.egtp_head_forward_static(head.c, z, wl.B, y_out=y, phat_out=phat)
        torch.cuda.synchronize()
        if n > 0:      # the first call on a device may load the module that holds the scratch array; later calls hold still
            assert torch.cuda.mem_get_info()[0] == free_before
        y64 = y.cpu().numpy().astype(np.float64)
        # the oracle's head on exactly the vectors the entry point was given
        y_ref, p_ref = orc.head_forward(z32, hp.W1, hp.b1, hp.W2, hp.b2, hp.mode, hp.centres)
        gu.assert_length_close(y64, y_ref)
        if hp is wl.head:                                   # and the context path's own prediction for that head
            gu.assert_length_close(y64, ref["yhat"])
        if phat is not None:
            assert np.allclose(phat.cpu().numpy(), p_ref, atol=1e-5)
            assert np.allclose(phat.cpu().numpy(), ref["phat"], atol=1e-5)


def test_static_head_rejects_sizes_beyond_its_scratch():
    wl = gen.config_tiny()
    head = gu.DeviceHead(wl.head, wl.dtype)
    rows = (1 << 20) // wl.head.m_h + 1
    z = torch.zeros(8, wl.d, device="cuda")
    y = torch.zeros(8, device="cuda")
    rc = egtp.egtp_head_forward_static(head.c, z, rows, y_out=y, check=False)           # nothing is launched
    assert rc == egtp.EGTP_ERR_CAPACITY
    assert egtp.egtp_head_forward_static(head.c, z, 8, y_out=None, check=False) == egtp.EGTP_ERR_INVALID_ARG
