"""Memo of the oracle's token entropies (Eq. 2), so that the full-size parity tests stay affordable.

The fp64 oracle needs 2 d V flops per token: a few hundred tokens per second.  The full-size tests send
thousands of whole prompts' tokens through it, always the same seeded ones, so the entropies are kept on
disk between runs.  A stored array is only ever written by `oracle.egtp_oracle.token_entropy` itself and is
keyed by a digest of everything that determines it: the bytes of the rows, the bytes of the LM head and
the oracle's own source text.  A missing or unreadable entry is simply recomputed.  Nothing here knows about
the CUDA path.
"""
from __future__ import annotations

import hashlib
import inspect
import os

import numpy as np

from oracle import egtp_oracle as orc

CACHE_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), ".oracle_cache")
_w_digests = {}


def _digest_array(a: np.ndarray) -> str:
    a = np.ascontiguousarray(a)
    h = hashlib.blake2b(digest_size=16)
    h.update(str((a.dtype.str, a.shape)).encode())
    flat = a.reshape(-1).view(np.uint8)
    step = 1 << 26
    for i in range(0, flat.shape[0], step):
        h.update(flat[i:i + step].data)
    return h.hexdigest()


def w_digest(W: np.ndarray) -> str:
    """Digest of an LM head, remembered per array object (hashing 1.5 GB takes a second or two)."""
    key = (id(W), W.shape)
    if key not in _w_digests:
        _w_digests[key] = _digest_array(W)
    return _w_digests[key]


def token_entropy(rows: np.ndarray, W: np.ndarray) -> np.ndarray:
    """oracle.token_entropy(rows, W), read from disk when these exact inputs were seen before."""
    src = inspect.getsource(orc.logits) + inspect.getsource(orc.entropy_from_logits) + inspect.getsource(orc.token_entropy)
    key = hashlib.blake2b((_digest_array(rows) + w_digest(W) + src).encode(), digest_size=16).hexdigest()
    path = os.path.join(CACHE_DIR, f"H_{key}.npy")
    if os.path.exists(path):
        try:
            H = np.load(path)
            if H.shape == (rows.shape[0],) and H.dtype == np.float64:
                return H
        except Exception:
            pass
    H = orc.token_entropy(rows, W)
    try:
        os.makedirs(CACHE_DIR, exist_ok=True)
        tmp = f"{path}.tmp{os.getpid()}.npy"
        np.save(tmp, H)
        os.replace(tmp, path)
    except OSError:
        pass
    return H
