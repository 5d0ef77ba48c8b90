"""Host logic of the LM-head kernel's launch plan (no GPU): which kernel form a batch gets, how the vocabulary is
cut into chunks and tiles, and the workspace bounds.  The expected values are either counted by hand from the
tile sizes (128-row blocks, 256-column tiles, 148 SMs, 74 CTA pairs) or invariants every plan must satisfy."""
import math

import pytest

from paper_2602_11812_b200 import binding as egtp

SMS, PAIRS = 148, 74


def plan(T, d, V, **kw):
    return egtp.egtp_lmhead_plan_for(SMS, kw.pop("pairs", PAIRS), T, d, V, **kw)


def test_kernel_form_by_row_count():
    assert plan(1, 4096, 151936)["variant"] == 1 and plan(128, 4096, 151936)["variant"] == 1
    assert plan(129, 4096, 151936)["variant"] == 5 and plan(256, 4096, 151936)["variant"] == 5      # CTA pairs
    assert plan(257, 4096, 151936)["variant"] == 0
    # without co-schedulable pairs, or when single CTAs are asked for, 129..256 rows use the one-CTA decode form
    assert plan(256, 4096, 151936, pairs=0)["variant"] == 2
    assert plan(256, 4096, 151936, mode=egtp.EGTP_LMHEAD_SINGLE_CTA)["variant"] == 2
    # pairs for prompt batches only on request, and never together with head columns
    assert plan(9555, 2048, 151936, mode=egtp.EGTP_LMHEAD_CTA_PAIRS)["variant"] == 4
    assert plan(1024, 5120, 152064, mode=egtp.EGTP_LMHEAD_CTA_PAIRS, head_cols=512)["variant"] == 0
    wide = plan(25629, 4096, 151936, mode=egtp.EGTP_LMHEAD_CTA_PAIRS_WIDE)      # 256 x 512 tiles for prompts on request
    assert (wide["variant"], wide["rows_per_block"], wide["tile_cols"], wide["row_blocks"]) == (6, 256, 512, 101)
    assert wide["n_groups"] == math.ceil(151936 / 512)
    # fp32 rows: prompt shape and one-row-tile decode shape only, never pairs, two stages holding every tile twice
    f = egtp.EGTP_F32
    assert plan(200, 256, 4096, dtype=f)["variant"] == 0 and plan(100, 256, 4096, dtype=f)["variant"] == 1
    assert plan(9555, 256, 4096, dtype=f, mode=egtp.EGTP_LMHEAD_CTA_PAIRS)["variant"] == 0
    assert plan(200, 256, 4096, dtype=f)["smem_bytes"] == 2 * 2 * (128 * 128 + 256 * 128) + 256 + 1024


def test_decode_plans_give_every_worker_one_vocabulary_range():
    p = plan(256, 4096, 151936)
    assert (p["grid"], p["chunks"], p["slots"], p["tile_cols"], p["rows_per_block"]) == (148, 74, 148, 512, 256)
    assert p["col_gran"] == 64 and p["n_groups"] == 151936 // 64                 # 2374 groups of 64 columns
    assert p["k_blocks"] == 4096 * 2 // 128
    q = plan(256, 4096, 151936, head_cols=256)                                  # W1 rows ride along: 4 more groups
    assert q["n_groups"] == p["n_groups"] + 4 and q["chunks"] == 74
    r = plan(100, 4096, 151936)
    assert (r["grid"], r["chunks"], r["slots"], r["col_gran"]) == (148, 148, 296, 32)
    assert r["n_groups"] == 151936 // 32
    # a vocabulary smaller than one range per worker: one chunk per column group, a smaller grid
    s = plan(200, 256, 1000)
    assert s["chunks"] == math.ceil(1000 / 64) and s["grid"] == 2 * s["chunks"]


def test_prompt_plans_at_the_named_sizes():
    mid = plan(9555, 2048, 151936)
    # 75 row blocks x 594 tiles: 33 chunks of 18 tiles fill 16.7 of 17 rounds (306 tile times for an ideal of 301)
    assert (mid["row_blocks"], mid["n_groups"], mid["chunks"], mid["group_rb"]) == (75, 594, 33, 75)
    long_ = plan(25629, 4096, 151936)
    # 8 KB rows: groups of 4 row blocks (4 MB) and the 2 % rule
    assert (long_["row_blocks"], long_["chunks"], long_["group_rb"]) == (201, 8, 4)
    rl = plan(1024, 5120, 152064, head_cols=512)
    # 8 row blocks of 10 KB rows: one round of 8 x 18 = 144 units rather than three rounds of shorter ones
    assert (rl["row_blocks"], rl["chunks"], rl["n_groups"]) == (8, 18, 594 + 2)
    assert rl["row_blocks"] * rl["chunks"] <= SMS


@pytest.mark.parametrize("T", [1, 15, 127, 128, 129, 255, 256, 257, 300, 1000, 4097, 9555, 25629, 136769, 500000])
@pytest.mark.parametrize("d,V,head_cols", [(256, 1000, 0), (2048, 151936, 0), (4096, 151936, 256), (5120, 152064, 512),
                                          (8192, 128256, 0), (64, 40, 24)])
def test_plan_invariants(T, d, V, head_cols):
    p = plan(T, d, V, head_cols=head_cols)
    rows_pad = p["row_blocks"] * p["rows_per_block"]
    assert rows_pad >= T and rows_pad - T < p["rows_per_block"]
    assert p["k_blocks"] == math.ceil(d * 2 / 128)
    assert p["n_groups"] == math.ceil(V / p["col_gran"]) + math.ceil(head_cols / p["col_gran"])
    assert 1 <= p["chunks"] <= p["n_groups"]                       # every chunk owns at least one column group
    assert p["slots"] in (p["chunks"], 2 * p["chunks"])
    assert 1 <= p["grid"] <= SMS and p["smem_bytes"] <= 227 * 1024
    assert 1 <= p["group_rb"] <= p["row_blocks"]
    # the partial buffer of a context sized for T rows holds the plan
    capacity = max(math.ceil(T / 128) * 128 * 48, 256 * SMS * 2, 1 << 21)
    assert rows_pad * p["slots"] <= capacity
    if p["variant"] == 0:
        # the chosen chunk count is never worse than a single chunk, and never far from the best over 1..64
        workers = min(SMS, p["row_blocks"] * p["n_groups"])
        mk = lambda S: math.ceil(p["row_blocks"] * S / workers) * math.ceil(p["n_groups"] / S)
        best = min(mk(S) for S in range(1, min(64, p["n_groups"]) + 1))
        assert mk(p["chunks"]) <= 1.06 * best + 1e-9


def test_plan_argument_checks():
    info_err = egtp.EGTP_ERR_INVALID_ARG
    lib = egtp.load()
    import ctypes as C
    buf = (C.c_int32 * 12)()
    assert lib.egtp_lmhead_plan_for(0, 74, 100, 256, 1000, egtp.EGTP_BF16, 0, 0, buf) == info_err
    assert lib.egtp_lmhead_plan_for(148, 74, 0, 256, 1000, egtp.EGTP_BF16, 0, 0, buf) == info_err
    assert lib.egtp_lmhead_plan_for(148, 74, 100, 256, 1000, 7, 0, 0, buf) == egtp.EGTP_ERR_UNSUPPORTED
    assert lib.egtp_lmhead_plan_for(148, 74, 100, 256, 1000, egtp.EGTP_BF16, 9, 0, buf) == info_err
