"""Pins for the oracle's scalar formats: e4m3 against torch's float8_e4m3fn, fp16 against numpy."""
import numpy as np
import torch

import oracle


def test_e4m3_decode_all_256_codes_match_torch():
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).to(torch.float32).numpy()
    for b in range(256):
        got = oracle.e4m3_decode(b)
        if np.isnan(ref[b]):
            assert np.isnan(got) and b in (0x7F, 0xFF)
        else:
            assert got == float(ref[b]), b
    assert oracle.e4m3_decode(0x7E) == 448.0 and oracle.e4m3_decode(0x01) == 2.0 ** -9


def test_e4m3_encode_all_bf16_patterns_match_torch_inside_finite_range():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    x = oracle.bf16_bits_to_f32(bits)
    t = torch.from_numpy(x.copy())
    ref = t.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    finite = np.isfinite(x) & (np.abs(x) < 464.0)      # torch does not saturate; beyond this the readings differ
    n = 0
    for i in np.nonzero(finite)[0]:
        assert oracle.e4m3_encode(x[i]) == int(ref[i]), (hex(int(bits[i])), float(x[i]))
        n += 1
    assert n > 34000


def test_e4m3_encode_saturates_and_keeps_nan_and_signed_zero():
    for v in (448.0, 449.0, 463.9, 464.0, 480.0, 1e9, np.inf):
        assert oracle.e4m3_encode(v) == 0x7E
        assert oracle.e4m3_encode(-v) == 0xFE
    assert oracle.e4m3_encode(np.nan) & 0x7F == 0x7F
    assert oracle.e4m3_encode(0.0) == 0x00 and oracle.e4m3_encode(-0.0) == 0x80
    # ties go to the even mantissa: 0.0009765625 = 2^-10 lies midway between 0 and 2^-9
    assert oracle.e4m3_encode(2.0 ** -10) == 0x00
    assert oracle.e4m3_encode(3 * 2.0 ** -10) == 0x02
    # 17 lies midway between 16 (0x58) and 18 (0x59)
    assert oracle.e4m3_encode(17.0) == 0x58 and oracle.e4m3_encode(19.0) == 0x5A


def test_fp16_conversion_matches_numpy_and_saturates():
    rng = np.random.default_rng(0)
    xs = np.concatenate([rng.standard_normal(2000).astype(np.float32) * s for s in (1e-6, 1e-3, 1.0, 100.0, 3e4)])
    xs = np.concatenate([xs, np.float32([0.0, -0.0, 65504.0, 65519.9, 5.9604645e-8, 2.9802322e-8, 1.0009765625])])
    for x in xs:
        ref = np.float32(np.clip(x, -65504, 65504)).astype(np.float16)
        assert oracle.f32_to_f16_sat(x) == int(ref.view(np.uint16)), float(x)
    assert oracle.f32_to_f16_sat(1e9) == 0x7BFF and oracle.f32_to_f16_sat(-1e9) == 0xFBFF
    for u in rng.integers(0, 65536, 3000):
        h = np.uint16(u).view(np.float16)
        if np.isfinite(h):
            assert oracle.f16_to_f32(int(u)) == float(h)


def test_bf16_widening_matches_torch():
    bits = np.arange(0, 65536, 7, dtype=np.uint32).astype(np.uint16)
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).numpy()
    got = oracle.bf16_bits_to_f32(bits)
    ok = np.isnan(ref) | (ref == got)
    assert ok.all()
