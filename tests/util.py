"""Helpers shared by the tests: raw-code views of torch tensors for the oracle."""
import numpy as np
import torch


def codes(t: torch.Tensor) -> np.ndarray:
    """Raw storage codes of a bf16 / float8_e4m3fn tensor as a NumPy array (uint16 / uint8)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    if t.dtype == torch.float8_e4m3fn:
        return t.view(torch.uint8).numpy()
    raise TypeError(t.dtype)


def f32(t):
    return None if t is None else t.detach().cpu().contiguous().to(torch.float32).numpy()


def bf16_codes_from_f64(a) -> np.ndarray:
    """bf16 codes of values that are exactly representable in bf16 (asserted)."""
    t = torch.as_tensor(np.asarray(a, dtype=np.float64)).to(torch.bfloat16)
    assert np.array_equal(t.to(torch.float64).numpy(), np.asarray(a, dtype=np.float64)), "not exact in bf16"
    return codes(t)
