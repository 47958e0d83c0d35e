"""Pins for the oracle's own number-format code: every bf16 and e4m3 code against
the format definition written as exact rational arithmetic, and the encoders
against a library conversion (torch) and the round-to-nearest-even rule."""
import struct
from fractions import Fraction

import numpy as np
import torch

import oracle


def _bf16_by_definition(bits):
    s, e, m = bits >> 15, (bits >> 7) & 0xFF, bits & 0x7F
    if e == 0xFF:
        return None
    if e == 0:
        v = Fraction(m, 128) * Fraction(2) ** (-126)
    else:
        v = (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127)
    return -v if s else v


def test_bf16_decode_all_codes_match_definition():
    for bits in range(1 << 16):
        want = _bf16_by_definition(bits)
        got = oracle.bf16_to_f64(bits)
        if want is None:
            assert not np.isfinite(got)
        else:
            assert Fraction(got) == want, hex(bits)


def test_bf16_decode_is_upper_half_of_binary32():
    for bits in (0x0000, 0x8000, 0x3F80, 0xBF80, 0x4049, 0x0001, 0x7F7F, 0x0080):
        want = struct.unpack("<f", struct.pack("<I", bits << 16))[0]
        assert oracle.bf16_to_f64(bits) == want


def _e4m3_by_definition(code):
    s, e, m = code >> 7, (code >> 3) & 0xF, code & 7
    if e == 15 and m == 7:
        return None
    if e == 0:
        v = Fraction(m, 8) * Fraction(2) ** (-6)
    else:
        v = (1 + Fraction(m, 8)) * Fraction(2) ** (e - 7)
    return -v if s else v


def test_e4m3_decode_all_codes_match_definition_and_torch():
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    for code in range(256):
        want = _e4m3_by_definition(code)
        got = oracle.e4m3_to_f64(code)
        if want is None:
            assert np.isnan(got) and np.isnan(lib[code])
        else:
            assert Fraction(got) == want, hex(code)
            assert got == lib[code]
    assert oracle.e4m3_to_f64(0x7E) == 448.0
    assert oracle.e4m3_to_f64(0x01) == 2.0 ** -9


def test_encoders_round_trip_every_code():
    for bits in range(1 << 16):
        v = _bf16_by_definition(bits)
        if v is None:
            continue
        assert oracle.f32_to_bf16(float(v)) == bits or (v == 0)
    for code in range(256):
        v = _e4m3_by_definition(code)
        if v is None or v == 0:
            continue
        assert oracle.f32_to_e4m3(float(v)) == code


def test_encoders_round_to_nearest_even_and_saturate():
    # bf16: 1 + 2^-8 is the midpoint between 1 (even mantissa) and 1 + 2^-7 -> 1
    assert oracle.f32_to_bf16(1.0 + 2.0 ** -8) == 0x3F80
    # 1 + 3*2^-8 is the midpoint between 1+2^-7 (odd) and 1+2^-6 (even) -> 1+2^-6
    assert oracle.f32_to_bf16(1.0 + 3 * 2.0 ** -8) == 0x3F82
    # e4m3: 1.0625 is the midpoint of 1.0 (m=0) and 1.125 (m=1) -> even -> 1.0
    assert oracle.f32_to_e4m3(1.0625) == 0x38
    assert oracle.f32_to_e4m3(1.1875) == 0x3A      # midpoint of 1.125 (m=1) and 1.25 (m=2) -> 1.25
    assert oracle.f32_to_e4m3(1e6) == 0x7E and oracle.f32_to_e4m3(-1e6) == 0xFE
    assert oracle.f32_to_e4m3(460.0) == 0x7E


def test_encoders_match_torch_on_random_values():
    g = torch.Generator().manual_seed(7)
    x = torch.randn(4000, generator=g) * torch.tensor([1e-3, 1.0, 30.0, 400.0]).repeat(1000)
    b = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    f8 = x.clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    for i in range(x.numel()):
        assert oracle.f32_to_bf16(float(x[i])) == int(b[i])
        got = oracle.f32_to_e4m3(float(x[i]))
        if (got & 0x7F) == 0 and (int(f8[i]) & 0x7F) == 0:
            continue                                  # signed zeros compare equal
        assert got == int(f8[i]), (float(x[i]), got, int(f8[i]))
