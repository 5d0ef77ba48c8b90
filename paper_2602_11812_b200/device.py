"""Moves seeded host inputs into device memory (torch tensors) and wraps them for the C ABI. Marshalling only."""
import numpy as np
import torch

from . import binding as egtp
from . import inputs as gen


def dev_tensor(x: np.ndarray, dtype: str) -> torch.Tensor:
    """float32 numpy values -> device tensor in the workload dtype (exact for bf16-representable values)."""
    if dtype == "bf16":
        bits = gen.bf16_bits(x).view(np.int16)
        return torch.from_numpy(bits).cuda().view(torch.bfloat16).reshape(x.shape)
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()


def host_tensor(x: np.ndarray, dtype: str) -> torch.Tensor:
    """Pinned host tensor in the workload dtype."""
    if dtype == "bf16":
        return torch.from_numpy(gen.bf16_bits(x).view(np.int16)).view(torch.bfloat16).reshape(x.shape).pin_memory()
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).pin_memory()


class DeviceHead:
    """Regression-head parameters resident on the device plus the C struct that points at them."""

    def __init__(self, head: gen.HeadParams, dtype: str):
        self.W1 = dev_tensor(head.W1, dtype)
        self.W2 = dev_tensor(head.W2, dtype)
        self.b1 = torch.from_numpy(head.b1).cuda()
        self.b2 = torch.from_numpy(head.b2).cuda()
        self.centres = None if head.centres is None else torch.from_numpy(head.centres).cuda()
        self.c = egtp.make_head(self.W1, self.b1, self.W2, self.b2, head.mode, self.centres)
        self.d_out = head.d_out
