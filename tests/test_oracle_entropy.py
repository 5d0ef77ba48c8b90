"""Pins for the oracle's logits and token entropy (Eq. 2): closed forms, invariants, library routines, brute force."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import egtp_oracle as orc


def test_uniform_logits_give_ln_V():
    # W = 0 makes every logit 0, so the distribution is uniform and H = ln V exactly.
    for V, d, expect in [(4096, 8, 8.317766166719343), (151936, 4, 11.931214658529285), (152064, 4, 11.932056763842207)]:
        assert abs(expect - math.log(V)) < 1e-12
        hidden = np.random.default_rng(0).standard_normal((3, d)).astype(np.float32)
        H = orc.token_entropy(hidden, np.zeros((V, d), dtype=np.float32))
        assert np.allclose(H, expect, rtol=0, atol=1e-11)
    # hidden = 0 does the same
    W = np.random.default_rng(1).standard_normal((777, 5)).astype(np.float32)
    assert np.allclose(orc.token_entropy(np.zeros((2, 5), np.float32), W), math.log(777), atol=1e-12)


def test_one_hot_limit_is_zero():
    V = 1000
    x = np.zeros((2, V))
    x[0, 17] = 60.0
    x[1, 999] = 800.0       # would overflow without the max subtraction; p underflows to exactly 0 elsewhere
    H = orc.entropy_from_logits(x)
    assert 0.0 <= H[0] < 1e-20 * V * 100
    assert H[1] == 0.0


def test_two_level_closed_form():
    # k columns at logit a, V-k at 0:  H = ln Z - k a e^a / Z,  Z = k e^a + V - k.
    for V, k, a in [(4096, 3, 5.0), (151936, 100, 7.0), (50, 49, -2.0), (1024, 512, 1.0)]:
        hidden = np.zeros((1, 4), dtype=np.float32)
        hidden[0, 0] = 1.0
        W = np.zeros((V, 4), dtype=np.float32)
        W[:k, 0] = a
        W[:, 1:] = 3.0        # multiplied by hidden zeros: must not matter
        Z = k * math.exp(a) + V - k
        expect = math.log(Z) - k * a * math.exp(a) / Z
        H = orc.token_entropy(hidden, W)
        assert abs(H[0] - expect) < 1e-12 * max(1.0, expect)


def test_logits_index_order_brute_force():
    # x[i, v] = sum_k hidden[i, k] W[v, k] with V != d so that a transposed operand cannot pass.
    rng = np.random.default_rng(2)
    hidden = rng.standard_normal((3, 4))
    W = rng.standard_normal((7, 4))
    x = orc.logits(hidden, W)
    assert x.shape == (3, 7)
    for i in range(3):
        for v in range(7):
            assert abs(x[i, v] - math.fsum(hidden[i, k] * W[v, k] for k in range(4))) < 1e-14
    # square, non-symmetric case
    Wsq = rng.standard_normal((4, 4))
    xs = orc.logits(hidden, Wsq)
    assert abs(xs[1, 2] - math.fsum(hidden[1, k] * Wsq[2, k] for k in range(4))) < 1e-14


def _entropy_python(xrow):
    m = max(xrow)
    e = [math.exp(v - m) for v in xrow]
    s = math.fsum(e)
    p = [v / s for v in e]
    return -math.fsum(pi * math.log(pi) for pi in p if pi > 0.0)


def test_entropy_brute_force_tiny():
    rng = np.random.default_rng(3)
    for V, d in [(2, 1), (3, 2), (8, 4), (5, 3)]:
        hidden = rng.standard_normal((6, d)).astype(np.float32) * 3
        W = rng.standard_normal((V, d)).astype(np.float32)
        H = orc.token_entropy(hidden, W)
        for i in range(6):
            xr = [math.fsum(float(hidden[i, k]) * float(W[v, k]) for k in range(d)) for v in range(V)]
            assert abs(H[i] - _entropy_python(xr)) < 1e-13


def test_entropy_matches_library_routines():
    # scipy.stats.entropy(softmax(x)) and the identity H = logsumexp(x) - sum softmax(x) x.
    rng = np.random.default_rng(4)
    x = rng.standard_normal((5, 300)) * 4.0
    H = orc.entropy_from_logits(x)
    p = scipy.special.softmax(x, axis=1)
    assert np.allclose(H, scipy.stats.entropy(p, axis=1), rtol=1e-12, atol=1e-12)
    lse = scipy.special.logsumexp(x, axis=1)
    assert np.allclose(H, lse - (p * x).sum(axis=1), rtol=1e-11, atol=1e-11)


def test_shift_and_permutation_invariance_and_bounds():
    rng = np.random.default_rng(5)
    V, d = 257, 6
    hidden = rng.standard_normal((9, d)).astype(np.float32) * 2
    W = rng.standard_normal((V, d)).astype(np.float32)
    H = orc.token_entropy(hidden, W)
    assert np.all(H >= 0.0) and np.all(H <= math.log(V) + 1e-12)
    # one extra hidden channel times a constant W column adds the same constant to every logit of a token
    hidden2 = np.concatenate([hidden, rng.standard_normal((9, 1)).astype(np.float32)], axis=1)
    W2 = np.concatenate([W, np.full((V, 1), 2.5, dtype=np.float32)], axis=1)
    assert np.allclose(orc.token_entropy(hidden2, W2), H, rtol=0, atol=1e-11)
    # relabelling the vocabulary leaves every entropy unchanged
    perm = rng.permutation(V)
    assert np.allclose(orc.token_entropy(hidden, W[perm]), H, rtol=0, atol=1e-12)
    # a constant added to a raw logit row
    x = rng.standard_normal((2, 50))
    assert np.allclose(orc.entropy_from_logits(x + 123.0), orc.entropy_from_logits(x), atol=1e-11)


def test_scaling_logits_moves_entropy_the_right_way():
    # sharper distribution (logits x 4) has lower entropy; flatter (x 0.25) has higher: catches a sign slip.
    rng = np.random.default_rng(6)
    x = rng.standard_normal((4, 100))
    H1 = orc.entropy_from_logits(x)
    assert np.all(orc.entropy_from_logits(4 * x) < H1)
    assert np.all(orc.entropy_from_logits(0.25 * x) > H1)


def test_row_blocking_does_not_matter():
    rng = np.random.default_rng(7)
    hidden = rng.standard_normal((37, 8)).astype(np.float32)
    W = rng.standard_normal((65, 8)).astype(np.float32)
    a = orc.token_entropy(hidden, W, rows_per_block=64)
    b = orc.token_entropy(hidden, W, rows_per_block=5)
    assert np.array_equal(a, b) or np.allclose(a, b, rtol=0, atol=1e-14)


def test_gaussian_logit_sanity():
    # logits ~ N(0, s^2), large V:  H ~ ln V - s^2 / 2  (not a gate on the method, a plausibility check)
    rng = np.random.default_rng(8)
    V, s = 100000, 1.0
    x = rng.standard_normal((4, V)) * s
    H = orc.entropy_from_logits(x)
    assert np.all(np.abs(H - (math.log(V) - s * s / 2)) < 0.02)
