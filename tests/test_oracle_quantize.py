"""Pins for the oracle's per-token FP8 quantiser (the step in front of the indexer, Sec. 2.1)."""
import numpy as np
import torch

import oracle
from tests.util import bf16_codes_from_f64, codes


def _library_quantize(x: torch.Tensor):
    """The same definition through torch's own float8 conversion (round to nearest even, after clamping)."""
    flat = x.reshape(x.shape[0], -1)
    scale = (flat.abs().amax(dim=1).clamp_min(1e-12) / 448.0).to(torch.float32)
    y = (flat / scale[:, None]).clamp_(-448.0, 448.0)
    return y.to(torch.float8_e4m3fn).reshape(x.shape), scale


def test_matches_library_conversion_bit_for_bit():
    g = torch.Generator().manual_seed(3)
    for shape, mul in [((50, 128), 1.0), ((7, 4, 64), 30.0), ((9, 8), 1e-3), ((3, 256), 1e4)]:
        x = (torch.randn(shape, generator=g) * mul).to(torch.bfloat16)
        want_codes, want_scale = _library_quantize(x.to(torch.float32))
        got_codes, got_scale = oracle.quantize_e4m3(codes(x))
        assert np.array_equal(got_scale, want_scale.numpy())
        a, b = got_codes.reshape(-1), codes(want_codes).reshape(-1)
        assert np.array_equal(a & 0x7F, b & 0x7F)                      # codes, up to the sign of zero
        assert np.array_equal((a >> 7)[(a & 0x7F) != 0], (b >> 7)[(b & 0x7F) != 0])


def test_closed_forms():
    # the largest magnitude of a row maps to +-448 (code 0x7E / 0xFE); powers of two below it are exact
    x = np.array([[448.0, -224.0, 112.0, 0.0, 56.0, -448.0, 1.75, 0.015625]])
    c, s = oracle.quantize_e4m3(bf16_codes_from_f64(x))
    assert s[0] == np.float32(1.0)
    assert c[0].tolist() == [0x7E, 0xF6, 0x6E, 0x00, 0x66, 0xFE, 0x3E, 0x08]
    # scaling a row by a power of two scales the scale and leaves the codes alone
    c2, s2 = oracle.quantize_e4m3(bf16_codes_from_f64(x * 8.0))
    assert s2[0] == np.float32(8.0) and np.array_equal(c2, c)
    # an all-zero row: scale floor 1e-12 / 448, codes zero
    c0, s0 = oracle.quantize_e4m3(bf16_codes_from_f64(np.zeros((2, 16))))
    assert np.all(c0 == 0) and np.all(s0 == np.float32(1e-12) / np.float32(448.0))


def test_dequantised_values_are_within_half_a_step():
    g = torch.Generator().manual_seed(5)
    x = torch.randn(64, 128, generator=g).to(torch.bfloat16)
    c, s = oracle.quantize_e4m3(codes(x))
    deq = np.vectorize(oracle.e4m3_to_f64)(c) * s[:, None].astype(np.float64)
    xd = x.to(torch.float64).numpy()
    # e4m3 has 3 mantissa bits: relative half-step 2^-4 for normal codes, absolute 2^-10 * scale below 2^-6
    err = np.abs(deq - xd)
    bound = np.maximum(np.abs(xd) * 2.0 ** -4, s[:, None] * 2.0 ** -10) * (1 + 1e-6)
    assert np.all(err <= bound)
