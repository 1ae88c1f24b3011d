"""Pins of the oracle's 8-bit floating-point decode and of the expansion of an fp8 offline cache."""
import math

import numpy as np
import torch

import oracle


def test_decode_matches_the_library_conversion_for_all_256_bytes():
    ref = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy()
    got = np.array([oracle.e4m3_decode(b) for b in range(256)], dtype=np.float32)
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(got[ok].view(np.uint32), ref[ok].view(np.uint32))


def test_decode_matches_the_stated_values_of_the_format():
    # 1 sign, 4 exponent (bias 7), 3 mantissa bits; no infinities; one NaN pattern per sign
    assert oracle.e4m3_decode(0x00) == 0.0 and math.copysign(1.0, oracle.e4m3_decode(0x80)) == -1.0
    assert oracle.e4m3_decode(0x38) == 1.0 and oracle.e4m3_decode(0xB8) == -1.0
    assert oracle.e4m3_decode(0x01) == 2.0 ** -9            # smallest subnormal
    assert oracle.e4m3_decode(0x07) == 7 * 2.0 ** -9        # largest subnormal
    assert oracle.e4m3_decode(0x08) == 2.0 ** -6            # smallest normal
    assert oracle.e4m3_decode(0x7E) == 448.0                # largest finite
    assert oracle.e4m3_decode(0x3C) == 1.5 and oracle.e4m3_decode(0x40) == 2.0
    assert math.isnan(oracle.e4m3_decode(0x7F)) and math.isnan(oracle.e4m3_decode(0xFF))
    finite = [oracle.e4m3_decode(b) for b in range(0x7F)]
    assert all(a < b for a, b in zip(finite, finite[1:])), "positive codes are strictly increasing"


def test_expansion_with_unit_scale_is_exact_widening_and_scales_round_once_to_bf16():
    rng = np.random.default_rng(5)
    b = rng.integers(0, 256, size=(37, 3, 16), dtype=np.uint8)
    b[(b & 0x7F) == 0x7F] = 0x10                             # no NaN codes in a cache
    wide = torch.from_numpy(b).view(torch.float8_e4m3fn).float().numpy()
    assert np.array_equal(oracle.dequant_fp8(b), wide)                       # scale 1: every value is a bf16 value
    assert np.array_equal(oracle.dequant_fp8(b, np.ones(3, np.float32)), wide)
    # power-of-two scales stay exact; a general scale is one fp32 product rounded to bf16 (library rounding)
    sc = np.array([0.5, 4.0, 0.3], dtype=np.float32)
    got = oracle.dequant_fp8(b, sc)
    ref = (torch.from_numpy(wide) * torch.from_numpy(sc).view(1, 3, 1)).to(torch.bfloat16).float().numpy()
    assert np.array_equal(got, ref)
    assert np.array_equal(got[:, 0], wide[:, 0] * 0.5) and np.array_equal(got[:, 1], wide[:, 1] * 4.0)
