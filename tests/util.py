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


# ---------------------------------------------------------------- parity criteria
RTOL_BF16 = 2e-3     # stated tolerance for bf16 inputs (relative)
RTOL_FP8 = 3e-2      # stated tolerance for e4m3 inputs


def row_scale(o_row: np.ndarray) -> float:
    """RMS of a row's oracle scores: the floor under the relative tolerance, so that
    scores that cancel to ~0 are not held to a zero tolerance."""
    return float(np.sqrt(np.mean(np.square(o_row)))) if o_row.size else 0.0


def assert_scores_close(g_row: np.ndarray, o_row: np.ndarray, rtol: float, what=""):
    """|g - o| <= rtol * max(|o|, rms(o_row)) elementwise; returns the largest error in units of the bound."""
    rho = row_scale(o_row)
    bound = rtol * np.maximum(np.abs(o_row), rho)
    err = np.abs(g_row.astype(np.float64) - o_row)
    if o_row.size and not np.all(err <= bound):
        i = int(np.argmax(err - bound))
        raise AssertionError(f"{what}: score {i}: gpu {g_row[i]!r} oracle {o_row[i]!r} bound {bound[i]!r}")
    return float(np.max(err / np.maximum(bound, 1e-300))) if o_row.size else 0.0


def assert_topk_valid(g_idx: np.ndarray, o_row: np.ndarray, k_top: int, rtol: float, what="") -> bool:
    """Checks a GPU index row against the oracle's scores of that row (length n = candidates).
    Unique part: size, order, range, padding, and membership outside the tolerance band around the
    oracle's k-th score. Returns True when the set equals the oracle's exactly."""
    n = o_row.shape[0]
    kk = min(k_top, n)
    sel = g_idx[:kk]
    assert np.all(g_idx[kk:] == -1), f"{what}: padding"
    assert np.all(sel >= 0) and np.all(sel < n), f"{what}: index out of range"
    assert np.all(np.diff(sel) > 0), f"{what}: not strictly ascending"
    if kk == n:
        return True
    order = np.argsort(-o_row, kind="stable")
    theta = o_row[order[kk - 1]]
    tau = rtol * max(abs(theta), row_scale(o_row))
    chosen = np.zeros(n, dtype=bool)
    chosen[sel] = True
    must = o_row > theta + tau
    must_not = o_row < theta - tau
    assert np.all(chosen[must]), f"{what}: misses a position clearly above the k-th score"
    assert not np.any(chosen[must_not]), f"{what}: holds a position clearly below the k-th score"
    return bool(np.array_equal(np.sort(order[:kk]), sel))
