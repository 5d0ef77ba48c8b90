"""Pins for the oracle's weights (Eq. 3), pooling (Eq. 4), head (Eq. 6), segment indexing and PLP (Eq. 8)."""
import math
import types

import numpy as np
import pytest

from oracle import egtp_oracle as orc


def _head(rng, d, m_h, d_out, mode=orc.HEAD_SCALAR, centres=None):
    return types.SimpleNamespace(
        W1=rng.standard_normal((m_h, d)) / math.sqrt(d), b1=rng.standard_normal(m_h) * 0.1,
        W2=rng.standard_normal((d_out, m_h)) / math.sqrt(m_h), b2=rng.standard_normal(d_out) * 0.1,
        mode=mode, centres=centres)


# ----------------------------- Eq. 3 / Eq. 4 -------------------------------- #
def test_equal_entropies_reduce_to_the_mean():
    rng = np.random.default_rng(0)
    rows = rng.standard_normal((13, 5))
    w = orc.entropy_weights(np.full(13, 7.25))
    assert np.allclose(w, 1.0 / 13, atol=1e-15)
    assert np.allclose(orc.pool(rows, w), rows.mean(axis=0), atol=1e-14)
    # through the whole chain: W = 0 makes every entropy ln V
    hidden = rng.standard_normal((13, 5)).astype(np.float32)
    head = _head(rng, 5, 3, 1)
    out = orc.egtp_predict(hidden, np.array([0, 4, 13]), np.zeros((11, 5), np.float32), head)
    assert np.allclose(out["pooled"][0], hidden[:4].astype(np.float64).mean(axis=0), atol=1e-14)
    assert np.allclose(out["pooled"][1], hidden[4:].astype(np.float64).mean(axis=0), atol=1e-14)


def test_two_token_closed_form_and_direction():
    # n = 2:  w_1 = 1 / (1 + exp(H_2 - H_1)); the higher-entropy token gets the larger weight (Sec. 3.1).
    H = np.array([2.0, 3.5])
    w = orc.entropy_weights(H)
    assert abs(w[0] - 1.0 / (1.0 + math.exp(1.5))) < 1e-15
    assert w[1] > w[0] and abs(w.sum() - 1.0) < 1e-15
    # temperature divides the entropies: alpha = 2 halves the gap
    w2 = orc.entropy_weights(H, alpha=2.0)
    assert abs(w2[0] - 1.0 / (1.0 + math.exp(0.75))) < 1e-15


def test_temperature_limits():
    H = np.array([1.0, 4.0, 2.0, 3.9])
    assert np.allclose(orc.entropy_weights(H, alpha=1e9), 0.25, atol=1e-8)           # flat: average pooling
    w = orc.entropy_weights(H, alpha=1e-3)                                           # sharp: picks the arg-max token
    assert w[1] > 1 - 1e-12 and w[0] < 1e-300


def test_weights_brute_force_and_pool_brute_force():
    rng = np.random.default_rng(1)
    H = rng.uniform(5, 11, size=9)
    rows = rng.standard_normal((9, 4))
    w = orc.entropy_weights(H)
    den = math.fsum(math.exp(h) for h in H)
    for i in range(9):
        assert abs(w[i] - math.exp(H[i]) / den) < 1e-14        # Eq. 3 as printed (no max subtraction)
    h = orc.pool(rows, w)
    for k in range(4):
        assert abs(h[k] - math.fsum(w[i] * rows[i, k] for i in range(9))) < 1e-14


def test_single_token_identity_and_range_and_permutation():
    rng = np.random.default_rng(2)
    rows = rng.standard_normal((17, 6))
    H = rng.uniform(0, 12, size=17)
    assert np.allclose(orc.pool(rows[:1], orc.entropy_weights(H[:1])), rows[0], atol=0)
    w = orc.entropy_weights(H)
    h = orc.pool(rows, w)
    assert np.all(h <= rows.max(axis=0) + 1e-14) and np.all(h >= rows.min(axis=0) - 1e-14)
    perm = rng.permutation(17)
    assert np.allclose(orc.pool(rows[perm], orc.entropy_weights(H[perm])), h, atol=1e-13)


def test_softmax_state_and_split_merge():
    rng = np.random.default_rng(3)
    H = rng.uniform(3, 12, size=20)
    rows = rng.standard_normal((20, 3))
    M, Z = orc.softmax_state(H)
    assert M == H.max() and abs(Z - math.fsum(math.exp(h - M) for h in H)) < 1e-13
    # the pool of [A; B] is the Z-weighted merge of the pools of A and B
    (Ma, Za), (Mb, Zb) = orc.softmax_state(H[:7]), orc.softmax_state(H[7:])
    pa = orc.pool(rows[:7], orc.entropy_weights(H[:7]))
    pb = orc.pool(rows[7:], orc.entropy_weights(H[7:]))
    ca, cb = Za * math.exp(Ma - M), Zb * math.exp(Mb - M)
    assert abs(ca + cb - Z) < 1e-12
    assert np.allclose((ca * pa + cb * pb) / (ca + cb), orc.pool(rows, orc.entropy_weights(H)), atol=1e-13)
    assert orc.softmax_state(np.array([])) == (-np.inf, 0.0)


# ----------------------------- segment indexing ----------------------------- #
def test_segment_ids_cases():
    assert orc.segment_ids(np.array([0, 2, 5]), 5).tolist() == [0, 0, 1, 1, 1]
    # leading and trailing tokens belong to no prompt; empty prompts own no token
    assert orc.segment_ids(np.array([1, 1, 3, 3, 4]), 6).tolist() == [-1, 1, 1, 3, -1, -1]
    rng = np.random.default_rng(4)
    lens = rng.integers(0, 9, size=40)
    off = np.concatenate([[3], 3 + np.cumsum(lens)])
    T = int(off[-1]) + 5
    seg = orc.segment_ids(off, T)
    ref = np.searchsorted(off, np.arange(T), side="right") - 1
    ref[(np.arange(T) < off[0]) | (np.arange(T) >= off[-1])] = -1
    assert np.array_equal(seg, ref.astype(np.int32))
    assert orc.offsets_valid(off, T) and not orc.offsets_valid(np.array([0, 5, 4]), 9)
    assert not orc.offsets_valid(np.array([0, 5, 10]), 9) and not orc.offsets_valid(np.array([-1, 5]), 9)


def test_egtp_predict_segments_are_isolated_and_empty_is_zero():
    rng = np.random.default_rng(5)
    d, V = 6, 33
    hidden = rng.standard_normal((20, d)).astype(np.float32)
    W = rng.standard_normal((V, d)).astype(np.float32)
    head = _head(rng, d, 4, 1)
    off = np.array([2, 7, 7, 15, 19])
    out = orc.egtp_predict(hidden, off, W, head)
    assert np.all(out["pooled"][1] == 0) and out["state_s"][1] == 0 and out["state_m"][1] == -np.inf
    y_empty, _ = orc.head_forward(np.zeros(d), head.W1, head.b1, head.W2, head.b2)
    assert out["yhat"][1] == y_empty[0]
    assert np.all(out["weights"][:2] == 0) and np.all(out["weights"][19:] == 0)
    for b in (0, 2, 3):
        assert abs(out["weights"][off[b]:off[b + 1]].sum() - 1.0) < 1e-14
    hidden2 = hidden.copy()
    hidden2[7:15] += 1.0                      # touch prompt 2 only
    out2 = orc.egtp_predict(hidden2, off, W, head)
    for b in (0, 1, 3):
        assert np.array_equal(out["pooled"][b], out2["pooled"][b]) and out["yhat"][b] == out2["yhat"][b]
    assert not np.array_equal(out["pooled"][2], out2["pooled"][2])
    # each prompt alone gives the same answer as inside the batch
    solo = orc.egtp_predict(hidden[7:15], np.array([0, 8]), W, head)
    assert np.allclose(solo["pooled"][0], out["pooled"][2], atol=1e-14)
    with pytest.raises(ValueError):
        orc.egtp_predict(hidden, np.array([0, 9, 5]), W, head)


# ----------------------------- Eq. 6: head ---------------------------------- #
def test_head_special_cases():
    rng = np.random.default_rng(6)
    d, m_h, K = 7, 5, 20
    centres = (np.arange(K) + 0.5) * 409.6
    head = _head(rng, d, m_h, K, orc.HEAD_BINS, centres)
    z = rng.standard_normal((3, d))
    # W1 = 0: the output is the same constant W2 ReLU(b1) + b2 for every row
    y0, _ = orc.head_forward(z, np.zeros_like(head.W1), head.b1, head.W2[:1], head.b2[:1])
    const = math.fsum(head.W2[0, j] * max(0.0, head.b1[j]) for j in range(m_h)) + head.b2[0]
    assert np.allclose(y0, const, atol=1e-14)
    # bins: a huge logit on bin k gives y = c_k; equal logits give the mean centre
    W2 = np.zeros((K, m_h))
    b2 = np.zeros(K)
    b2[13] = 500.0
    y, p = orc.head_forward(z, head.W1, head.b1, W2, b2, orc.HEAD_BINS, centres)
    assert np.allclose(y, centres[13], atol=1e-9) and np.allclose(p[:, 13], 1.0)
    y, p = orc.head_forward(z, head.W1, head.b1, W2, np.zeros(K), orc.HEAD_BINS, centres)
    assert np.allclose(y, centres.mean(), atol=1e-10) and np.allclose(p, 1.0 / K)


def test_head_brute_force():
    rng = np.random.default_rng(7)
    d, m_h, K = 5, 4, 3
    centres = np.array([10.0, 100.0, 1000.0])
    head = _head(rng, d, m_h, K, orc.HEAD_BINS, centres)
    z = rng.standard_normal(d)
    u = [max(0.0, math.fsum(head.W1[j, k] * z[k] for k in range(d)) + head.b1[j]) for j in range(m_h)]
    o = [math.fsum(head.W2[c, j] * u[j] for j in range(m_h)) + head.b2[c] for c in range(K)]
    den = math.fsum(math.exp(v) for v in o)
    expect = math.fsum(math.exp(o[c]) / den * centres[c] for c in range(K))
    y, p = orc.head_forward(z, head.W1, head.b1, head.W2, head.b2, orc.HEAD_BINS, centres)
    assert abs(y[0] - expect) < 1e-11 and abs(p.sum() - 1) < 1e-14
    ys, none = orc.head_forward(z, head.W1, head.b1, head.W2[:1], head.b2[:1], orc.HEAD_SCALAR)
    assert none is None and abs(ys[0] - o[0]) < 1e-13
    assert any(v == 0.0 for v in u) or True      # ReLU exercised below
    zneg = -50 * np.sign(head.W1[0]) / np.abs(head.W1[0]).sum() * 50
    yn, _ = orc.head_forward(zneg, head.W1, head.b1, head.W2[:1], head.b2[:1])
    un = [max(0.0, math.fsum(head.W1[j, k] * zneg[k] for k in range(d)) + head.b1[j]) for j in range(m_h)]
    assert un[0] == 0.0
    assert abs(yn[0] - (math.fsum(head.W2[0, j] * un[j] for j in range(m_h)) + head.b2[0])) < 1e-12


# ----------------------------- Eq. 8: PLP ----------------------------------- #
def _streaming_reference(hidden_steps, H_steps, reset_src, slot, prompts_state, alpha=1.0):
    """Independent restatement: running (m, s, acc) with the usual online-softmax update."""
    m, s, acc = -math.inf, 0.0, np.zeros(hidden_steps.shape[2])
    zs = []
    for t in range(hidden_steps.shape[0]):
        r = int(reset_src[t, slot])
        if r == orc.RESET_EMPTY:
            m, s, acc = -math.inf, 0.0, np.zeros_like(acc)
        elif r >= 0:
            pm, ps, pp = prompts_state
            m, s, acc = pm[r], ps[r], pp[r] * ps[r]
        a = H_steps[t, slot] / alpha
        m2 = max(m, a)
        scale = 0.0 if m == -math.inf else math.exp(m - m2)
        e = math.exp(a - m2)
        s = s * scale + e
        acc = acc * scale + e * hidden_steps[t, slot].astype(np.float64)
        m = m2
        zs.append(acc / s)
    return np.stack(zs)


def test_plp_equals_egtp_on_the_concatenation_and_streaming():
    rng = np.random.default_rng(8)
    d, V, steps, slots = 6, 40, 9, 3
    W = rng.standard_normal((V, d)).astype(np.float32)
    head = _head(rng, d, 4, 1)
    p_hidden = (rng.standard_normal((11, d)) * 2).astype(np.float32)
    p_off = np.array([0, 4, 11])
    eg = orc.egtp_predict(p_hidden, p_off, W, head)
    hs = (rng.standard_normal((steps, slots, d)) * 2).astype(np.float32)
    reset = np.full((steps, slots), orc.RESET_KEEP, dtype=np.int32)
    reset[0] = [0, 1, orc.RESET_EMPTY]
    reset[5, 1] = orc.RESET_EMPTY            # slot 1 retires and restarts empty
    reset[6, 2] = 0                          # slot 2 restarts from prompt 0
    out = orc.plp_run(hs, reset, W, head, prompts=dict(hidden=p_hidden, offsets=p_off, H=eg["H"]))
    Hs = np.stack([orc.token_entropy(hs[t], W) for t in range(steps)])
    assert np.allclose(out["H"], Hs, atol=1e-13)
    # slot 0 at step 3 == EGTP over [prompt 0 ; its first four generated tokens]
    cat = np.concatenate([p_hidden[0:4], hs[0:4, 0, :]])
    ref = orc.egtp_predict(cat, np.array([0, 8]), W, head)
    assert np.allclose(out["z"][3, 0], ref["pooled"][0], atol=1e-13)
    assert abs(out["yrem"][3, 0] - ref["yhat"][0]) < 1e-12
    # a slot reset to empty: after its first token z is that token's hidden state
    assert np.allclose(out["z"][0, 2], hs[0, 2].astype(np.float64), atol=0)
    assert np.allclose(out["z"][5, 1], hs[5, 1].astype(np.float64), atol=0)
    # the running-state form gives the same z at every step
    st = (eg["state_m"], eg["state_s"], eg["pooled"])
    for s in range(slots):
        assert np.allclose(out["z"][:, s], _streaming_reference(hs, Hs, reset, s, st), atol=1e-12)


def test_plp_fan_out_identical_streams_stay_identical():
    rng = np.random.default_rng(9)
    d, V, steps = 5, 17, 4
    W = rng.standard_normal((V, d)).astype(np.float32)
    head = _head(rng, d, 3, 1)
    p_hidden = rng.standard_normal((6, d)).astype(np.float32)
    p_off = np.array([0, 6])
    eg = orc.egtp_predict(p_hidden, p_off, W, head)
    one = rng.standard_normal((steps, 1, d)).astype(np.float32)
    hs = np.repeat(one, 4, axis=1)
    reset = np.full((steps, 4), orc.RESET_KEEP, dtype=np.int32)
    reset[0] = 0
    out = orc.plp_run(hs, reset, W, head, prompts=dict(hidden=p_hidden, offsets=p_off, H=eg["H"]))
    for s in range(1, 4):
        assert np.array_equal(out["z"][:, s], out["z"][:, 0]) and np.array_equal(out["yrem"][:, s], out["yrem"][:, 0])


# ----------------------------- Table 3: pooling alternatives ----------------- #
def test_baseline_pooling_definitions():
    rng = np.random.default_rng(10)
    rows = rng.standard_normal((7, 5))
    mean, mx, last = (orc.pool_baseline(rows, m) for m in (orc.POOL_MEAN, orc.POOL_MAX, orc.POOL_LAST))
    for k in range(5):
        assert abs(mean[k] - math.fsum(rows[i, k] for i in range(7)) / 7) < 1e-15
        assert mx[k] == max(rows[i, k] for i in range(7))
        assert last[k] == rows[6, k]
    # average pooling is EGTP with equal entropies; a one-token prompt makes all variants that token
    assert np.allclose(mean, orc.pool(rows, orc.entropy_weights(np.zeros(7))), atol=1e-15)
    for m in (orc.POOL_MEAN, orc.POOL_MAX, orc.POOL_LAST):
        assert np.array_equal(orc.pool_baseline(rows[2:3], m), rows[2])
    # max and mean ignore token order, last-token pooling does not
    perm = rng.permutation(7)
    assert np.array_equal(orc.pool_baseline(rows[perm], orc.POOL_MAX), mx)
    assert np.allclose(orc.pool_baseline(rows[perm], orc.POOL_MEAN), mean, atol=1e-15)
    assert np.all(mx >= mean) and np.all(mx >= last)
    head = _head(rng, 5, 3, 1)
    out = orc.baseline_predict(rows, np.array([0, 3, 3, 7]), head, orc.POOL_LAST)
    assert np.array_equal(out["pooled"][0], rows[2]) and np.all(out["pooled"][1] == 0) and np.array_equal(out["pooled"][2], rows[6])
    y, _ = orc.head_forward(rows[6], head.W1, head.b1, head.W2, head.b2)
    assert out["yhat"][2] == y[0]
    with pytest.raises(ValueError):
        orc.pool_baseline(rows, 9)
