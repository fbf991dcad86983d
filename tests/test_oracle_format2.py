"""Pins for record format 2 of the oracle's TQ3 codec (e4m3-exact key codebook, re-cut key section) and
the tie rule of the key quantiser in both formats.

Nothing here re-types the encoder: the codebook is checked against the 8-bit float format itself
(torch.float8_e4m3fn), against a Lloyd iteration and against the closed-form distortion integral of a
scalar quantiser of N(0,1); the codec by exact round trips on inputs built to sit on the codebook, by
norm preservation and the distortion law of a norm-corrected decoder; the packer by a bit-level
bijection; ties by vectors whose rotated coordinate sits exactly on a decision threshold."""
import math

import numpy as np
import pytest
import torch

import oracle
from _util import read_golden
from test_oracle_tq3 import hadamard, lloyd_max_gaussian

FORMATS = [1, 2]


def gaussian_quantiser_mse(C, B):
    """Distortion of the symmetric scalar quantiser with positive levels C and thresholds B on N(0,1):
    2 * sum over the cells of the integral of (x - c)^2 phi(x), in closed form."""
    phi = lambda x: math.exp(-0.5 * x * x) / math.sqrt(2 * math.pi)
    Phi = lambda x: 0.5 * (1 + math.erf(x / math.sqrt(2)))
    edges = [0.0] + [float(b) for b in B] + [math.inf]
    total = 0.0
    for j, c in enumerate(float(x) for x in C):
        lo, hi = edges[j], edges[j + 1]
        P = (1.0 if math.isinf(hi) else Phi(hi)) - Phi(lo)
        m1 = phi(lo) - (0.0 if math.isinf(hi) else phi(hi))
        m2 = P + lo * phi(lo) - (0.0 if math.isinf(hi) else hi * phi(hi))
        total += m2 - 2 * c * m1 + c * c * P
    return 2 * total


def test_format2_codebook_is_the_lloyd_max_quantiser_moved_onto_e4m3():
    with oracle.record_format(2):
        C, B = oracle.codebook()
    # every level survives a round trip through the 8-bit float, in torch's codec and in the oracle's own
    as_e4m3 = torch.tensor(C, dtype=torch.float32).to(torch.float8_e4m3fn)
    assert np.array_equal(as_e4m3.to(torch.float32).numpy(), C)
    for c in C:
        assert oracle.e4m3_decode(oracle.e4m3_encode(float(c))) == float(c)
    # it is the e4m3 number nearest to the Lloyd optimum, level by level
    opt, _ = lloyd_max_gaussian()
    grid = np.array(sorted({oracle.e4m3_decode(b) for b in range(0x7F)}))
    for j in range(4):
        assert grid[np.argmin(np.abs(grid - opt[j]))] == float(C[j])
    assert C.tolist() == [0.25, 0.75, 1.375, 2.25]
    for j in range(3):
        assert float(B[j]) == (float(C[j]) + float(C[j + 1])) / 2      # exact midpoints
    # distortion: about 1 % above the optimum (textbook value in the golden file), never below it
    gold = read_golden("lloyd_max_gaussian_8.txt")
    D2 = gaussian_quantiser_mse(C, B)
    assert gold["mse"] * 0.9999 < D2 < gold["mse"] * 1.0115
    with oracle.record_format(1):
        C1, B1 = oracle.codebook()
    assert abs(gaussian_quantiser_mse(C1, B1) - gold["mse"]) < 2e-5


def test_format_selection_is_checked_and_restored():
    assert oracle.get_format() == 1
    with oracle.record_format(2):
        assert oracle.get_format() == 2
    assert oracle.get_format() == 1
    with pytest.raises(ValueError):
        oracle.set_format(3)


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("d", [128, 256])
def test_key_on_codebook_round_trips_exactly_in_both_formats(d, fmt):
    rng = np.random.default_rng(100 * fmt + d)
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    H = hadamard(d)
    with oracle.record_format(fmt):
        C, _ = oracle.codebook()
        for trial in range(10):
            # magnitudes drawn with the Gaussian cell probabilities; the encoder sees c * r with
            # r = sqrt(d) / |c|, and every level stays inside its own cell for 0.82 < r < 1.29
            while True:
                mag = rng.choice(4, size=d, p=[0.3833, 0.3230, 0.2132, 0.0805])
                r = math.sqrt(d) / np.linalg.norm(C[mag].astype(np.float64))
                if 0.85 < r < 1.25:
                    break
            sgn = rng.integers(0, 2, d)
            c = np.where(sgn == 1, -1.0, 1.0) * C[mag].astype(np.float64)
            x64 = sigma * (H @ c) / d
            code, g = oracle.tq3_encode_key(x64.astype(np.float32), sigma)
            assert np.array_equal(code & 3, mag.astype(np.uint8)) and np.array_equal(code >> 2, sgn.astype(np.uint8))
            xhat = oracle.tq3_decode_key(code, g, sigma)
            assert abs(oracle.f16_to_f32(g) * math.sqrt(d) - 1.0) < 2.0 ** -10
            assert np.abs(xhat - x64).max() <= (2.0 ** -10) * np.abs(x64).max() + 1e-7


@pytest.mark.parametrize("d", [128, 256])
def test_format2_norm_is_preserved_and_distortion_follows_its_own_quantiser(d):
    rng = np.random.default_rng(70 + d)
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    with oracle.record_format(2):
        C, B = oracle.codebook()
        D = gaussian_quantiser_mse(C, B)
        rel = []
        for trial in range(300):
            x = rng.standard_normal(d).astype(np.float32) * np.float32(10.0 ** rng.uniform(-2, 2))
            code, g = oracle.tq3_encode_key(x, sigma)
            xhat = oracle.tq3_decode_key(code, g, sigma)
            nx = np.linalg.norm(x.astype(np.float64))
            assert abs(np.linalg.norm(xhat) / nx - 1.0) < 2.0 ** -11 + 1e-5
            rel.append(np.sum((xhat - x) ** 2) / nx ** 2)
    expect = 2 * (1 - math.sqrt(1 - D))
    assert abs(np.mean(rel) - expect) < 0.0015, (np.mean(rel), expect)


@pytest.mark.parametrize("d", [128, 256])
def test_format2_packed_record_is_a_bijection_and_differs_from_format1_in_the_key_section_only(d):
    rng = np.random.default_rng(d)
    kc = rng.integers(0, 8, (16, d)).astype(np.uint8)
    vc = rng.integers(0, 8, (16, d)).astype(np.uint8)
    g = rng.integers(0, 65536, 16).astype(np.uint16)
    sc = rng.integers(0, 65536, d).astype(np.uint16)
    zp = rng.integers(0, 65536, d).astype(np.uint16)
    rec1 = oracle.tq3_pack_record(kc, g, vc, sc, zp)
    with oracle.record_format(2):
        rec2 = oracle.tq3_pack_record(kc, g, vc, sc, zp)
        out = oracle.tq3_unpack_record(rec2, d)
        for a, b in zip(out, (kc, g, vc, sc, zp)):
            assert np.array_equal(a, b)
        full = oracle.tq3_pack_record(np.full((16, d), 7, np.uint8), np.full(16, 0xFFFF, np.uint16),
                                      np.full((16, d), 7, np.uint8), np.full(d, 0xFFFF, np.uint16), np.full(d, 0xFFFF, np.uint16))
        assert np.all(full == 0xFF)
        seen = np.zeros(6 * d * 8, bool)
        z16, zd, z = np.zeros(16, np.uint16), np.zeros(d, np.uint16), np.zeros((16, d), np.uint8)
        for t in range(16):
            for i in range(0, d, 3):
                for bit in range(3):
                    a = z.copy()
                    a[t, i] = 1 << bit
                    bits = np.unpackbits(oracle.tq3_pack_record(a, z16, z, zd, zd), bitorder="little")
                    assert bits.sum() == 1
                    pos = int(np.argmax(bits))
                    assert pos < 6 * d * 8 and not seen[pos]          # inside the key section, never reused
                    seen[pos] = True
        # four consecutive dims of a token sit in the four nibbles of one 16-bit half-word, code bits at the
        # low three bits of each nibble (or: two magnitude bits there and the sign in another word)
        a = z.copy()
        a[5, 8:12] = [1, 2, 3, 1]
        bits = np.unpackbits(oracle.tq3_pack_record(a, z16, z, zd, zd), bitorder="little")
        pos = np.nonzero(bits)[0]
        assert pos.max() - pos.min() < 16 and pos.min() // 16 == pos.max() // 16
    assert not np.array_equal(rec1[:6 * d], rec2[:6 * d]) and np.array_equal(rec1[6 * d:], rec2[6 * d:])


# Vectors x (eight non-zero entries, the rest zero, rotation signs +1) whose squares sum to N^2 and whose
# entries sum to `on`: the rotated coordinate of every dim i with i % 8 == 0 is then exactly `on`, which is
# exactly threshold j times |x| = N.  Found by a random search; the test checks both properties itself.
TIES = [
    (1, 4096, 2050, 0, [29, -2011, -1376, 867, 700, 1462, 2711, -332]),
    (1, 4096, 4300, 1, [-1441, 1598, 1612, 47, 82, -1422, 2233, 1591]),
    (1, 4096, 7160, 2, [1869, 1795, -50, 1116, 1987, -573, 1926, -910]),
    (2, 16, 8, 0, [4, 5, -7, 0, 8, 7, -2, -7]),
    (2, 32, 34, 1, [-11, 12, -11, 5, -2, 8, 17, 16]),
    (2, 32, 58, 2, [13, -4, 11, 11, 1, -2, 24, 4]),
]


@pytest.mark.parametrize("fmt,N,on,j,head", TIES)
@pytest.mark.parametrize("d", [128, 256])
def test_a_coordinate_exactly_on_a_threshold_takes_the_lower_magnitude(d, fmt, N, on, j, head):
    """Reading of the tie rule: the comparison with a threshold is strict, so a rotated coordinate that equals
    threshold j * |x| keeps magnitude j (the level below the threshold), for either sign."""
    assert sum(v * v for v in head) == N * N and sum(head) == on
    with oracle.record_format(fmt):
        _, B = oracle.codebook()
        assert float(B[j]) * N == on                              # exact in fp32: the threshold really is met
        for sign in (1.0, -1.0):
            x = np.zeros(d, np.float32)
            x[:8] = np.float32(head) * np.float32(sign)
            code, g = oracle.tq3_encode_key(x, np.ones(d, np.int8))
            w = hadamard(d) @ x.astype(np.float64)
            assert np.all(w[::8] == sign * on)
            assert np.all((code[::8] & 3) == j) and np.all((code[::8] >> 2) == (1 if sign < 0 else 0))
            # a coordinate one fp32 step above the threshold does cross it
            others = np.abs(w) > float(B[j]) * N
            assert np.all((code[others] & 3) > j)
