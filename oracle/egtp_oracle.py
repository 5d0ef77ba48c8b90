"""CPU oracle for Entropy-Guided Token Pooling (EGTP) and Progressive Length Prediction (PLP).

TEST INFRASTRUCTURE ONLY.  This file is the parity authority for the CUDA path and
the timed CPU baseline; it is deliberately plain, slow and written to be checked
against the paper by eye.  Only the tests, the smoke check and the benchmark's CPU
baseline leg may import it.  It shares no code with the CUDA path and imports
nothing from the package.

Everything is computed in float64 with numpy.  Inputs (float32 arrays whose
values are exactly the numbers the device reads) are widened exactly; nothing is
re-rounded.  `numpy.matmul` is used as the library primitive for the dot
products; tokens are handled in row blocks only to bound memory (each token's
result depends on that token alone).

Every function below is pinned by closed forms, invariants and brute force in
tests/test_oracle_*.py; no function is "parity unpinned".

Readings of the paper taken here (the paper leaves these open):
  * the logarithm of Eq. 2 is natural (entropy in nats);
  * the temperature alpha that the text of Sec. 3.1 mentions divides the
    entropies inside the softmax of Eq. 3; alpha = 1 is Eq. 3 as printed;
  * H_i is the entropy of softmax(W h_i), the distribution emitted at position i;
    logits are hidden . W^T with no bias, norm or temperature;
  * the head is a two-layer ReLU MLP whose output is either a scalar or K bin
    logits turned into an expectation over bin centres (Eq. 6);
  * PLP's Aggregate (Eq. 8) concatenates along the token axis: z_t is the
    entropy-weighted pool over the prompt's tokens followed by the generated
    tokens 1..t, computed from the explicit token list every step.
"""
from __future__ import annotations

import numpy as np

HEAD_SCALAR = 0
HEAD_BINS = 1
RESET_KEEP = -2
RESET_EMPTY = -1
POOL_MEAN = 1
POOL_MAX = 2
POOL_LAST = 3


# --------------------------------------------------------------------------- #
# Eq. 2: token entropy
# --------------------------------------------------------------------------- #
def logits(hidden_rows: np.ndarray, W: np.ndarray) -> np.ndarray:
    """x[i, v] = sum_k hidden[i, k] * W[v, k]  (Sec. 3.1: next-token distribution over the vocabulary)."""
    h = np.asarray(hidden_rows, dtype=np.float64)
    w = np.asarray(W, dtype=np.float64)
    return h @ w.T


def entropy_from_logits(x: np.ndarray) -> np.ndarray:
    """Eq. 2, two passes per row: p = softmax(x); H = -sum_v p_v ln p_v, with 0 ln 0 = 0."""
    x = np.asarray(x, dtype=np.float64)
    m = x.max(axis=1, keepdims=True)
    e = np.exp(x - m)
    s = e.sum(axis=1, keepdims=True)
    p = e / s
    with np.errstate(divide="ignore", invalid="ignore"):
        plogp = np.where(p > 0.0, p * np.log(p), 0.0)
    return -plogp.sum(axis=1)


def token_entropy(hidden: np.ndarray, W: np.ndarray, rows_per_block: int = 64) -> np.ndarray:
    """H[i] for every row of `hidden` (Eq. 2). Row blocks only bound the size of the logits buffer."""
    T = hidden.shape[0]
    W64 = np.asarray(W, dtype=np.float64)
    H = np.empty(T, dtype=np.float64)
    for r0 in range(0, T, rows_per_block):
        r1 = min(T, r0 + rows_per_block)
        H[r0:r1] = entropy_from_logits(logits(hidden[r0:r1], W64))
    return H


# --------------------------------------------------------------------------- #
# segment indexing
# --------------------------------------------------------------------------- #
def offsets_valid(offsets: np.ndarray, T: int) -> bool:
    off = np.asarray(offsets, dtype=np.int64)
    return bool(off[0] >= 0 and off[-1] <= T and np.all(np.diff(off) >= 0))


def segment_ids(offsets: np.ndarray, T: int) -> np.ndarray:
    """seg[i] = the b with offsets[b] <= i < offsets[b+1] (linear scan), -1 if token i is in no prompt."""
    off = np.asarray(offsets, dtype=np.int64)
    seg = np.full(T, -1, dtype=np.int32)
    for i in range(T):
        for b in range(off.shape[0] - 1):
            if off[b] <= i < off[b + 1]:
                seg[i] = b
                break
    return seg


# --------------------------------------------------------------------------- #
# Eq. 3 and Eq. 4: weights and pooling
# --------------------------------------------------------------------------- #
def entropy_weights(H_seg: np.ndarray, alpha: float = 1.0) -> np.ndarray:
    """Eq. 3: w_i = exp(H_i / alpha) / sum_j exp(H_j / alpha) over the tokens of one prompt."""
    a = np.asarray(H_seg, dtype=np.float64) / float(alpha)
    e = np.exp(a - a.max())
    return e / e.sum()


def pool(hidden_seg: np.ndarray, w: np.ndarray) -> np.ndarray:
    """Eq. 4: h = sum_i w_i h_i."""
    h = np.asarray(hidden_seg, dtype=np.float64)
    return np.asarray(w, dtype=np.float64) @ h


def softmax_state(H_seg: np.ndarray, alpha: float = 1.0):
    """(M, Z) with M = max_i H_i/alpha and Z = sum_i exp(H_i/alpha - M): the normaliser of Eq. 3."""
    if len(H_seg) == 0:
        return -np.inf, 0.0
    a = np.asarray(H_seg, dtype=np.float64) / float(alpha)
    M = float(a.max())
    return M, float(np.exp(a - M).sum())


def pool_baseline(hidden_seg: np.ndarray, mode: int) -> np.ndarray:
    """The pooling alternatives of the paper's ablation (Table 3): average, max and last-token pooling."""
    h = np.asarray(hidden_seg, dtype=np.float64)
    if mode == POOL_MEAN:
        return h.sum(axis=0) / h.shape[0]
    if mode == POOL_MAX:
        return h.max(axis=0)
    if mode == POOL_LAST:
        return h[-1].copy()
    raise ValueError("unknown pooling mode")


def baseline_predict(hidden, offsets, head, mode: int):
    """Table 3 comparators over a ragged batch: pooled [B, d] (zeros for an empty prompt) and the head's prediction."""
    hidden = np.asarray(hidden)
    off = np.asarray(offsets, dtype=np.int64)
    if not offsets_valid(off, hidden.shape[0]):
        raise ValueError("offsets must be non-decreasing and lie in [0, T]")
    B = off.shape[0] - 1
    pooled = np.zeros((B, hidden.shape[1]), dtype=np.float64)
    for b in range(B):
        if off[b + 1] > off[b]:
            pooled[b] = pool_baseline(hidden[off[b]:off[b + 1]], mode)
    yhat, phat = head_forward(pooled, head.W1, head.b1, head.W2, head.b2, head.mode, head.centres)
    return dict(pooled=pooled, yhat=yhat, phat=phat)


# --------------------------------------------------------------------------- #
# Eq. 6: prediction head
# --------------------------------------------------------------------------- #
def head_forward(z: np.ndarray, W1, b1, W2, b2, mode: int = HEAD_SCALAR, centres=None):
    """u = ReLU(W1 z + b1); o = W2 u + b2; scalar mode: y = o_0; bins mode: p = softmax(o), y = sum_k p_k c_k (Eq. 6).

    z may be one vector [d] or rows [B, d]. Returns (y, p) where p is None in scalar mode.
    """
    z = np.atleast_2d(np.asarray(z, dtype=np.float64))
    u = np.maximum(0.0, z @ np.asarray(W1, dtype=np.float64).T + np.asarray(b1, dtype=np.float64))
    o = u @ np.asarray(W2, dtype=np.float64).T + np.asarray(b2, dtype=np.float64)
    if mode == HEAD_SCALAR:
        return o[:, 0].copy(), None
    e = np.exp(o - o.max(axis=1, keepdims=True))
    p = e / e.sum(axis=1, keepdims=True)
    y = p @ np.asarray(centres, dtype=np.float64)
    return y, p


# --------------------------------------------------------------------------- #
# EGTP over a ragged batch
# --------------------------------------------------------------------------- #
def egtp_predict(hidden, offsets, W, head, alpha: float = 1.0, H=None):
    """Eq. 2 -> 3 -> 4 -> head for every prompt of a packed ragged batch.

    `head` is any object with W1, b1, W2, b2, mode, centres.  `H` may be passed in
    when the caller already computed the entropies of exactly these rows.
    An empty prompt pools to the zero vector with state (M, Z) = (-inf, 0).
    Returns a dict: H [T], seg_id [T], weights [T] (0 outside prompts), pooled [B, d],
    state_m [B], state_s [B], yhat [B], phat [B, K] or None.
    """
    hidden = np.asarray(hidden)
    T, d = hidden.shape
    off = np.asarray(offsets, dtype=np.int64)
    if not offsets_valid(off, T):
        raise ValueError("offsets must be non-decreasing and lie in [0, T]")
    B = off.shape[0] - 1
    if H is None:
        H = token_entropy(hidden, W)
    H = np.asarray(H, dtype=np.float64)
    weights = np.zeros(T, dtype=np.float64)
    pooled = np.zeros((B, d), dtype=np.float64)
    state_m = np.full(B, -np.inf, dtype=np.float64)
    state_s = np.zeros(B, dtype=np.float64)
    for b in range(B):
        s, e = int(off[b]), int(off[b + 1])
        if e == s:
            continue
        w = entropy_weights(H[s:e], alpha)
        weights[s:e] = w
        pooled[b] = pool(hidden[s:e], w)
        state_m[b], state_s[b] = softmax_state(H[s:e], alpha)
    yhat, phat = head_forward(pooled, head.W1, head.b1, head.W2, head.b2, head.mode, head.centres)
    return dict(H=H, seg_id=segment_ids(off, T), weights=weights, pooled=pooled,
                state_m=state_m, state_s=state_s, yhat=yhat, phat=phat)


# --------------------------------------------------------------------------- #
# Eq. 8: PLP, recomputed from the explicit token list every step
# --------------------------------------------------------------------------- #
class PlpSequence:
    """The tokens one live sequence has contributed since its last reset.

    A sequence that starts from a prompt whose tokens are not part of the decode
    call is represented by that prompt's entropies and hidden rows (given by the
    caller) placed in front of the generated tokens, so that z_t is literally the
    EGTP pool over the concatenated list.
    """

    def __init__(self, d: int):
        self.d = d
        self.rows = []   # hidden rows (float64 arrays of length d)
        self.H = []      # their entropies

    def reset(self, prompt_rows=None, prompt_H=None):
        self.rows = [] if prompt_rows is None else [np.asarray(r, dtype=np.float64) for r in prompt_rows]
        self.H = [] if prompt_H is None else [float(h) for h in prompt_H]

    def append(self, row, H):
        self.rows.append(np.asarray(row, dtype=np.float64))
        self.H.append(float(H))

    def aggregate(self, alpha: float = 1.0) -> np.ndarray:
        """z_t of Eq. 8: Eq. 3-4 over the whole list."""
        w = entropy_weights(np.asarray(self.H), alpha)
        return pool(np.stack(self.rows), w)


def plp_run(hidden_steps, reset_src, W, head, alpha: float = 1.0, slots=None, prompts=None, H_steps=None):
    """Follow `slots` (default: all) through every step of a decode loop.

    hidden_steps [steps, n_slots, d]; reset_src [steps, n_slots] with RESET_KEEP,
    RESET_EMPTY or r >= 0 (start from prompt r of `prompts`, a dict with
    hidden, offsets and H of the prompt batch).  At step t, slot s first applies its
    reset, then appends the step's token, then z_t and the remaining-length
    prediction are recomputed from the full list (Eq. 8 then Eq. 6).
    Returns dict: H [steps, len(slots)], z [steps, len(slots), d], yrem [steps, len(slots)].
    """
    hidden_steps = np.asarray(hidden_steps)
    steps, n_slots, d = hidden_steps.shape
    slots = list(range(n_slots)) if slots is None else list(slots)
    Hs = np.empty((steps, len(slots)), dtype=np.float64)
    zs = np.empty((steps, len(slots), d), dtype=np.float64)
    ys = np.empty((steps, len(slots)), dtype=np.float64)
    W64 = np.asarray(W, dtype=np.float64)
    seqs = [PlpSequence(d) for _ in slots]
    for t in range(steps):
        rows = hidden_steps[t, slots, :]
        Ht = token_entropy(rows, W64) if H_steps is None else np.asarray(H_steps[t], dtype=np.float64)
        for j, s in enumerate(slots):
            r = int(reset_src[t, s])
            if r == RESET_EMPTY:
                seqs[j].reset()
            elif r >= 0:
                po = np.asarray(prompts["offsets"], dtype=np.int64)
                a, b = int(po[r]), int(po[r + 1])
                seqs[j].reset(np.asarray(prompts["hidden"][a:b], dtype=np.float64), prompts["H"][a:b])
            seqs[j].append(rows[j], Ht[j])
            z = seqs[j].aggregate(alpha)
            zs[t, j] = z
            Hs[t, j] = Ht[j]
        y, _ = head_forward(zs[t], head.W1, head.b1, head.W2, head.b2, head.mode, head.centres)
        ys[t] = y
    return dict(H=Hs, z=zs, yrem=ys)
