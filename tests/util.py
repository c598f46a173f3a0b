"""Test-side helpers.  BF16 conversion goes through torch (a library routine
independent of the oracle's own widening / rounding code)."""
import numpy as np
import torch


def bf16_bits(x) -> np.ndarray:
    """Values -> BF16 bit patterns via torch's float32 -> bfloat16 rounding."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_value(bits) -> np.ndarray:
    """BF16 bit patterns -> float64 values via torch."""
    b = np.ascontiguousarray(np.asarray(bits, dtype=np.uint16))
    t = torch.from_numpy(b.view(np.int16)).view(torch.bfloat16)
    return t.to(torch.float64).numpy()


def finite_bf16_patterns() -> np.ndarray:
    """All BF16 patterns that are not NaN (the two infinities included)."""
    allp = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    nan = ((allp & 0x7F80) == 0x7F80) & ((allp & 0x007F) != 0)
    return allp[~nan]


def read_golden(name):
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", name)
    with open(path) as f:
        return [ln.split("#")[0].split() for ln in f if ln.split("#")[0].strip()]
