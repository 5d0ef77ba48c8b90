"""Seeded synthetic inputs for the EGTP / PLP hot path.

This module only *draws* inputs: prompt lengths, hidden states, LM-head weights,
regression-head parameters and PLP retire schedules.  It holds none of the
method's arithmetic (no entropy, no pooling, no head evaluation), so both the
CPU oracle's tests and the CUDA path's tests can use it without sharing any of
the code under test.

All tensors are numpy float32 arrays.  When ``dtype == "bf16"`` every value has
been rounded (round-to-nearest-even) to a bfloat16-representable number, so that
widening it to fp64 on the CPU side and narrowing it to bf16 bits for the device
are both exact: the oracle and the kernels read the same real numbers.

Length recipes follow the paper's description of long-tailed prompt and response
lengths (Sec. 4.1 and the dataset-statistics appendix); the datasets themselves
are not used anywhere.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

HEAD_SCALAR = 0
HEAD_BINS = 1

RESET_KEEP = -2
RESET_EMPTY = -1


# --------------------------------------------------------------------------- #
# bf16 helpers (pure bit manipulation)
# --------------------------------------------------------------------------- #
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 value (ties to even), returned as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    if np.any(u & np.uint32(0xFFFF)):
        raise ValueError("values are not bf16-representable; call round_to_bf16 first")
    return (u >> np.uint32(16)).astype(np.uint16)


def _maybe_round(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(f"unknown dtype {dtype!r}")


def _normal(rng: np.random.Generator, shape, scale: float, dtype: str, rows_per_block: int = 8192) -> np.ndarray:
    """N(0, scale^2) float32 array drawn block by block (bounded temporary memory)."""
    out = np.empty(shape, dtype=np.float32)
    flat = out.reshape(shape[0], -1) if len(shape) > 1 else out.reshape(-1, 1)
    for r0 in range(0, flat.shape[0], rows_per_block):
        r1 = min(flat.shape[0], r0 + rows_per_block)
        blk = rng.standard_normal((r1 - r0, flat.shape[1]), dtype=np.float32)
        if scale != 1.0:
            blk *= np.float32(scale)
        flat[r0:r1] = _maybe_round(blk, dtype)
    return out


# --------------------------------------------------------------------------- #
# containers
# --------------------------------------------------------------------------- #
@dataclass
class HeadParams:
    """Two-layer regression head d -> m_h -> d_out (ReLU in between)."""
    W1: np.ndarray            # [m_h, d]   values in the workload dtype
    b1: np.ndarray            # [m_h]      float32
    W2: np.ndarray            # [d_out, m_h]
    b2: np.ndarray            # [d_out]    float32
    mode: int = HEAD_SCALAR   # HEAD_SCALAR (d_out == 1) or HEAD_BINS (d_out == K)
    centres: Optional[np.ndarray] = None   # [d_out] float32 bin centres when mode == HEAD_BINS

    @property
    def d(self) -> int:
        return int(self.W1.shape[1])

    @property
    def m_h(self) -> int:
        return int(self.W1.shape[0])

    @property
    def d_out(self) -> int:
        return int(self.W2.shape[0])


@dataclass
class EgtpWorkload:
    name: str
    dtype: str                # "f32" or "bf16"
    hidden: np.ndarray        # [T_total, d] packed ragged rows
    offsets: np.ndarray       # int32 [B+1], token units
    W: np.ndarray             # [V, d] LM-head weight, row v = vocabulary entry v
    head: HeadParams
    alpha: float = 1.0
    seed: int = 0

    @property
    def B(self) -> int:
        return int(self.offsets.shape[0] - 1)

    @property
    def T(self) -> int:
        return int(self.hidden.shape[0])

    @property
    def d(self) -> int:
        return int(self.hidden.shape[1])

    @property
    def V(self) -> int:
        return int(self.W.shape[0])

    @property
    def lengths(self) -> np.ndarray:
        return np.diff(self.offsets)


@dataclass
class PlpWorkload:
    name: str
    dtype: str
    hidden_steps: np.ndarray  # [steps, slots, d]: one decode token per live slot per step
    reset_src: np.ndarray     # int32 [steps, slots]: RESET_KEEP, RESET_EMPTY or an EGTP row >= 0
    W: np.ndarray             # [V, d]
    head: HeadParams          # remaining-length head
    alpha: float = 1.0
    seed: int = 0
    prompts: Optional[EgtpWorkload] = None   # prompts whose EGTP state seeds the slots (RL group sampling)
    retire_len: Optional[np.ndarray] = None  # int64 [n_sequences] drawn response lengths (bookkeeping only)

    @property
    def steps(self) -> int:
        return int(self.hidden_steps.shape[0])

    @property
    def slots(self) -> int:
        return int(self.hidden_steps.shape[1])

    @property
    def d(self) -> int:
        return int(self.hidden_steps.shape[2])

    @property
    def V(self) -> int:
        return int(self.W.shape[0])


# --------------------------------------------------------------------------- #
# building blocks
# --------------------------------------------------------------------------- #
def offsets_from_lengths(lengths) -> np.ndarray:
    lengths = np.asarray(lengths, dtype=np.int64)
    off = np.zeros(lengths.shape[0] + 1, dtype=np.int64)
    np.cumsum(lengths, out=off[1:])
    if off[-1] >= 2**31:
        raise ValueError("token count does not fit int32 offsets")
    return off.astype(np.int32)


def lengths_lognormal(seed: int, n: int, mu: float, sigma: float, lo: int, hi: int) -> np.ndarray:
    rs = np.random.RandomState(seed)
    return np.clip(np.rint(rs.lognormal(mu, sigma, size=n)), lo, hi).astype(np.int64)


def lengths_pareto(seed: int, n: int, shape: float, x_m: int, lo: int, hi: int) -> np.ndarray:
    """Classical Pareto(shape, x_m): x_m * (1 + Lomax(shape)), floored and clipped."""
    rs = np.random.RandomState(seed)
    return np.clip(np.floor(x_m * (1.0 + rs.pareto(shape, size=n))), lo, hi).astype(np.int64)


def lengths_uniform(seed: int, n: int, lo: int, hi: int) -> np.ndarray:
    rs = np.random.RandomState(seed)
    return rs.randint(lo, hi + 1, size=n).astype(np.int64)


def make_hidden(seed: int, T: int, d: int, dtype: str, outlier_frac: float = 0.0,
                outlier_gain: float = 1.0) -> np.ndarray:
    """Rows ~ N(0, 1); a seeded subset of channels (outlier_frac of d) is multiplied by outlier_gain."""
    rng = np.random.Generator(np.random.PCG64(seed))
    n_out = int(round(outlier_frac * d))
    gain = np.ones(d, dtype=np.float32)
    if n_out > 0:
        ch = rng.choice(d, size=n_out, replace=False)
        gain[ch] = np.float32(outlier_gain)
    out = np.empty((T, d), dtype=np.float32)
    for r0 in range(0, T, 8192):
        r1 = min(T, r0 + 8192)
        blk = rng.standard_normal((r1 - r0, d), dtype=np.float32) * gain
        out[r0:r1] = _maybe_round(blk, dtype)
    return out


def make_lm_head(seed: int, V: int, d: int, dtype: str) -> np.ndarray:
    """W[v, k] ~ N(0, 1/d)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return _normal(rng, (V, d), float(1.0 / np.sqrt(d)), dtype)


def make_head(seed: int, d: int, m_h: int, d_out: int, dtype: str, mode: int = HEAD_SCALAR,
              bin_range: float = 8192.0) -> HeadParams:
    """Xavier-uniform weights, U(+-1/sqrt(fan_in)) biases; uniform bin centres over [0, bin_range)."""
    rng = np.random.Generator(np.random.PCG64(seed))

    def xavier(fan_out, fan_in):
        a = np.sqrt(6.0 / (fan_in + fan_out))
        return _maybe_round(rng.uniform(-a, a, size=(fan_out, fan_in)).astype(np.float32), dtype)

    def bias(n, fan_in):
        a = 1.0 / np.sqrt(fan_in)
        return rng.uniform(-a, a, size=n).astype(np.float32)

    W1 = xavier(m_h, d)
    b1 = bias(m_h, d)
    W2 = xavier(d_out, m_h)
    b2 = bias(d_out, m_h)
    centres = None
    if mode == HEAD_BINS:
        width = bin_range / d_out
        centres = ((np.arange(d_out, dtype=np.float64) + 0.5) * width).astype(np.float32)
    elif d_out != 1:
        raise ValueError("scalar head needs d_out == 1")
    return HeadParams(W1=W1, b1=b1, W2=W2, b2=b2, mode=mode, centres=centres)


def scaled_head(head: HeadParams, dtype: str, gain: float = 64.0, shift: float = 300.0) -> HeadParams:
    """The same scalar head with its output layer rescaled: W2 * gain (kept representable in `dtype`), b2 + shift.

    A Xavier-initialised head predicts a fraction of a token, so an absolute tolerance of half a token says
    nothing about it; rescaled like this it predicts a few hundred tokens, the range real lengths live in.
    """
    if head.mode != HEAD_SCALAR:
        raise ValueError("only scalar heads are rescaled (a bins head already predicts in token units)")
    W2 = _maybe_round(head.W2 * np.float32(gain), dtype)
    b2 = (head.b2 + np.float32(shift)).astype(np.float32)
    return HeadParams(W1=head.W1, b1=head.b1, W2=W2, b2=b2, mode=head.mode, centres=head.centres)


def make_egtp(name: str, seed: int, lengths, d: int, V: int, dtype: str, m_h: int, d_out: int = 1,
              mode: int = HEAD_SCALAR, outlier_frac: float = 0.0, outlier_gain: float = 1.0,
              alpha: float = 1.0, W: Optional[np.ndarray] = None) -> EgtpWorkload:
    """Streams: seed*1000 + {1 hidden, 2 W, 3 head}. A ready-made LM head `W` [V, d] may be passed in."""
    offsets = offsets_from_lengths(lengths)
    T = int(offsets[-1])
    hidden = make_hidden(seed * 1000 + 1, T, d, dtype, outlier_frac, outlier_gain)
    if W is None:
        W = make_lm_head(seed * 1000 + 2, V, d, dtype)
    assert W.shape == (V, d)
    head = make_head(seed * 1000 + 3, d, m_h, d_out, dtype, mode)
    return EgtpWorkload(name=name, dtype=dtype, hidden=hidden, offsets=offsets, W=W, head=head,
                        alpha=alpha, seed=seed)


def retire_schedule(seed: int, steps: int, slots: int, mu: float, sigma: float, first_src=None):
    """Reset table for a decode loop that keeps the batch full.

    Every slot starts a sequence at step 0.  A sequence's response length is
    max(1, round(lognormal(mu, sigma))); when a slot has produced that many tokens
    the next step starts a new sequence in it (a reset before that step's token).
    ``first_src`` optionally gives the EGTP row each slot starts from (else empty).
    Returns (reset_src [steps, slots] int32, retire_len list).
    """
    rs = np.random.RandomState(seed)
    reset = np.full((steps, slots), RESET_KEEP, dtype=np.int32)
    drawn = []

    def draw():
        L = max(1, int(np.rint(rs.lognormal(mu, sigma))))
        drawn.append(L)
        return L

    for s in range(slots):
        t = 0
        first = True
        while t < steps:
            if first and first_src is not None:
                reset[t, s] = int(first_src[s])
            else:
                reset[t, s] = RESET_EMPTY
            first = False
            t += draw()
    return reset, np.asarray(drawn, dtype=np.int64)


# --------------------------------------------------------------------------- #
# the five named configurations (and scaled-down forms of each for tests)
# --------------------------------------------------------------------------- #
def config_tiny(mode: int = HEAD_SCALAR) -> EgtpWorkload:
    """4 prompts of lengths {16, 31, 48, 64}, d = 256 fp32, V = 4096, head 256 -> 128 -> 1, seed 0."""
    d_out = 20 if mode == HEAD_BINS else 1
    return make_egtp("egtp_tiny", 0, [16, 31, 48, 64], d=256, V=4096, dtype="f32", m_h=128,
                     d_out=d_out, mode=mode)


def config_mid(seed: int = 1, B: int = 32, d: int = 2048, V: int = 151936, m_h: int = 512,
               max_len: int = 2048) -> EgtpWorkload:
    """32 prompts, lengths lognormal(5.5, 0.8) clipped to [32, 2048]; 1 % outlier channels x 20."""
    lengths = lengths_lognormal(seed * 1000, B, 5.5, 0.8, 32, max_len)
    return make_egtp("egtp_mid", seed, lengths, d=d, V=V, dtype="bf16", m_h=m_h,
                     outlier_frac=0.01, outlier_gain=20.0)


def config_long(seed: int = 1, B: int = 64, d: int = 4096, V: int = 151936, m_h: int = 1024,
                max_len: int = 8192, W: Optional[np.ndarray] = None) -> EgtpWorkload:
    """64 prompts, lengths Pareto(1.2, x_m = 128) clipped to [128, 8192]; packed ragged rows."""
    lengths = lengths_pareto(seed * 1000, B, 1.2, 128, 128, max_len)
    return make_egtp("egtp_long", seed, lengths, d=d, V=V, dtype="bf16", m_h=m_h,
                     outlier_frac=0.01, outlier_gain=20.0, W=W)


def config_plp_decode(seed: int = 4, slots: int = 256, steps: int = 512, d: int = 4096,
                      V: int = 151936, m_h: int = 256, mu: float = 6.0, sigma: float = 1.0) -> PlpWorkload:
    """256 live sequences, one token per step; retire lengths lognormal(6, 1); batch kept full."""
    rng = np.random.Generator(np.random.PCG64(seed * 1000 + 1))
    hs = _normal(rng, (steps * slots, d), 1.0, "bf16").reshape(steps, slots, d)
    W = make_lm_head(seed * 1000 + 2, V, d, "bf16")
    head = make_head(seed * 1000 + 3, d, m_h, 1, "bf16")
    reset, drawn = retire_schedule(seed * 1000 + 4, steps, slots, mu, sigma)
    return PlpWorkload(name="plp_decode", dtype="bf16", hidden_steps=hs, reset_src=reset, W=W,
                       head=head, seed=seed, retire_len=drawn)


def config_rl_group(seed: int = 5, prompts: int = 64, group: int = 16, steps: int = 256, d: int = 5120,
                    V: int = 152064, m_h: int = 512, min_len: int = 256, max_len: int = 4096) -> PlpWorkload:
    """GRPO-style group sampling: EGTP over shared prompts, then `group` decode streams per prompt.

    Every slot starts from its prompt's EGTP state at step 0 and runs for all steps
    (no retirement inside the window); one head serves both phases.
    """
    lengths = lengths_uniform(seed * 1000, prompts, min_len, max_len)
    eg = make_egtp("rl_group_prompts", seed, lengths, d=d, V=V, dtype="bf16", m_h=m_h)
    slots = prompts * group
    rng = np.random.Generator(np.random.PCG64(seed * 1000 + 5))
    hs = _normal(rng, (steps * slots, d), 1.0, "bf16").reshape(steps, slots, d)
    reset = np.full((steps, slots), RESET_KEEP, dtype=np.int32)
    reset[0, :] = np.repeat(np.arange(prompts, dtype=np.int32), group)
    return PlpWorkload(name="rl_group", dtype="bf16", hidden_steps=hs, reset_src=reset, W=eg.W,
                       head=eg.head, seed=seed, prompts=eg)
