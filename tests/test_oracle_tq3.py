"""Pins for the oracle's TQ3 codec (Section 3.1 "Stale", Section 4.1 record contents).

Nothing here re-types the encoder: the checks are the textbook Lloyd-Max quantiser, closed forms
(norm preservation, Hadamard orthogonality, quantiser distortion), exact round trips on inputs
built to sit on codebook values, bounds of the uniform value quantiser, and a bit-level bijection
of the packed record."""
import math

import numpy as np
import pytest

import oracle
from _util import read_golden


def hadamard(d):
    H = np.array([[1.0]])
    while H.shape[0] < d:
        H = np.block([[H, H], [H, -H]])
    return H


def lloyd_max_gaussian(levels=4, iters=3000):
    """Positive half of the symmetric 2*levels-level minimum-MSE quantiser of N(0,1), fp64."""
    phi = lambda x: math.exp(-0.5 * x * x) / math.sqrt(2 * math.pi)
    Phi = lambda x: 0.5 * (1 + math.erf(x / math.sqrt(2)))
    c = [0.3, 0.9, 1.5, 2.3][:levels]
    for _ in range(iters):
        b = [0.0] + [(c[i] + c[i + 1]) / 2 for i in range(levels - 1)] + [float("inf")]
        c = [(phi(b[i]) - (0.0 if math.isinf(b[i + 1]) else phi(b[i + 1]))) /
             ((1.0 if math.isinf(b[i + 1]) else Phi(b[i + 1])) - Phi(b[i])) for i in range(levels)]
    b = [(c[i] + c[i + 1]) / 2 for i in range(levels - 1)]
    return c, b


def test_codebook_is_the_textbook_lloyd_max_quantiser_rounded_to_fp16():
    C, B = oracle.codebook()
    gold = read_golden("lloyd_max_gaussian_8.txt")
    for j in range(4):
        assert abs(float(C[j]) - gold[f"level_{j}"]) < 6e-4          # table is printed to 4 decimals
    for j in range(3):
        assert abs(float(B[j]) - gold[f"threshold_{j}"]) < 6e-4
    c, b = lloyd_max_gaussian()
    for j in range(4):
        assert np.float32(c[j]).astype(np.float16) == np.float16(C[j])   # nearest fp16 to the optimum
        assert float(np.float16(C[j])) == float(C[j])                    # levels are fp16-exact
    for j in range(3):
        assert float(B[j]) == (float(C[j]) + float(C[j + 1])) / 2        # thresholds are exact midpoints
        assert abs(float(B[j]) - b[j]) < 3e-4


def test_hadamard_orthogonality_closed_form():
    for d in (128, 256):
        H = hadamard(d)
        assert np.array_equal(H @ H, d * np.eye(d))


@pytest.mark.parametrize("d", [128, 256])
def test_key_on_codebook_round_trips_exactly(d):
    """x built so that its rotated, normalised image sits exactly on signed codebook levels:
    the codes come back unchanged and the decoded key equals x up to the fp16 rounding of g."""
    rng = np.random.default_rng(d)
    C, _ = oracle.codebook()
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    H = hadamard(d)
    for trial in range(20):
        # magnitudes drawn with the Gaussian cell probabilities, so that the mean square of c is
        # close to 1 and the encoder's normalisation (w / |x| = c * sqrt(d) / |c|) keeps every
        # coordinate well inside its own decision cell
        mag = rng.choice(4, size=d, p=[0.3833, 0.3230, 0.2132, 0.0805])
        r = math.sqrt(d) / np.linalg.norm(C[mag].astype(np.float64))
        assert 0.85 < r < 1.25      # cells stay intact for 0.82 < r < 1.29
        sgn = rng.integers(0, 2, d)
        c = np.where(sgn == 1, -1.0, 1.0) * C[mag].astype(np.float64)
        x64 = sigma * (H @ c) / d                       # then H(sigma*x) = c  exactly in exact arithmetic
        x = x64.astype(np.float32)
        # keep the construction away from decision thresholds: fp32 rounding of x perturbs w by ~1e-6
        code, g = oracle.tq3_encode_key(x, sigma)
        assert np.array_equal(code & 3, mag.astype(np.uint8))
        assert np.array_equal(code >> 2, sgn.astype(np.uint8))
        xhat = oracle.tq3_decode_key(code, g, sigma)
        gg = oracle.f16_to_f32(g)
        # |x| / |c| = 1/sqrt(d) here
        assert abs(gg * math.sqrt(d) - 1.0) < 2.0 ** -10
        assert np.abs(xhat - x64).max() <= (2.0 ** -10) * np.abs(x64).max() + 1e-7


@pytest.mark.parametrize("d", [128, 256])
def test_key_norm_is_preserved_and_distortion_matches_quantiser_theory(d):
    rng = np.random.default_rng(7 + d)
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    gold = read_golden("lloyd_max_gaussian_8.txt")
    D = gold["mse"]
    rel = []
    for trial in range(300):
        x = rng.standard_normal(d).astype(np.float32) * np.float32(10.0 ** rng.uniform(-2, 2))
        code, g = oracle.tq3_encode_key(x, sigma)
        xhat = oracle.tq3_decode_key(code, g, sigma)
        nx = np.linalg.norm(x.astype(np.float64))
        # norm correction: |k^| = |x| up to fp16 rounding of g (relative 2^-11) and fp32 noise
        assert abs(np.linalg.norm(xhat) / nx - 1.0) < 2.0 ** -11 + 1e-5
        rel.append(np.sum((xhat - x) ** 2) / nx ** 2)
    # a norm-corrected decoder has relative squared error 2(1 - sqrt(1 - D)) for quantiser MSE D
    expect = 2 * (1 - math.sqrt(1 - D))
    assert abs(np.mean(rel) - expect) < 0.0015, (np.mean(rel), expect)


def test_key_degenerate_and_tie_cases():
    d = 128
    sigma = np.ones(d, np.int8)
    code, g = oracle.tq3_encode_key(np.zeros(d, np.float32), sigma)
    assert g == 0 and not code.any()
    assert np.array_equal(oracle.tq3_decode_key(code, g, sigma), np.zeros(d))
    # a single non-zero entry: every rotated coordinate has |w| = |x_0|, i.e. w/|x| = +-1 -> level 1
    x = np.zeros(d, np.float32)
    x[0] = -3.0
    code, g = oracle.tq3_encode_key(x, sigma)
    assert np.all((code & 3) == 1) and np.all((code >> 2) == 1)
    xhat = oracle.tq3_decode_key(code, g, sigma)
    assert abs(xhat[0] + 3.0) < 3.0 * 2.0 ** -10 and np.abs(xhat[1:]).max() < 1e-12


def test_rotation_signs_enter_the_decoder():
    d = 128
    rng = np.random.default_rng(3)
    x = rng.standard_normal(d).astype(np.float32)
    s1 = np.ones(d, np.int8)
    s2 = s1.copy()
    s2[5] = -1
    c1, g1 = oracle.tq3_encode_key(x, s1)
    x2 = x.copy()
    x2[5] = -x2[5]
    c2, g2 = oracle.tq3_encode_key(x2, s2)          # sigma*x identical -> identical codes
    assert np.array_equal(c1, c2) and g1 == g2
    k1 = oracle.tq3_decode_key(c1, g1, s1)
    k2 = oracle.tq3_decode_key(c2, g2, s2)
    assert k1[5] == -k2[5] and np.array_equal(np.delete(k1, 5), np.delete(k2, 5))


@pytest.mark.parametrize("d", [128, 256])
def test_value_quantiser_bounds_and_extremes(d):
    rng = np.random.default_rng(11 + d)
    v = rng.standard_normal((16, d)).astype(np.float32)
    v[:, 3] *= 8
    v[:, 7] = 1.25            # constant channel
    v[:, 9] = 0.0
    code, sc, zp = oracle.tq3_encode_value_page(v)
    assert code.max() <= 7
    for c in range(d):
        s, z = oracle.f16_to_f32(int(sc[c])), oracle.f16_to_f32(int(zp[c]))
        col = v[:, c].astype(np.float64)
        if c in (7, 9):
            assert s == 0.0 and not code[:, c].any() and z == float(np.float16(col[0]))
            continue
        assert code[np.argmin(col), c] == 0 and code[np.argmax(col), c] == 7
        rec = np.array([oracle.tq3_decode_value(int(code[t, c]), int(sc[c]), int(zp[c])) for t in range(16)])
        rng_c = col.max() - col.min()
        # |v^ - v| <= s/2 (rounding) + 7*|s - range/7| (fp16 scale) + |z - min| (fp16 zero)
        bound = s / 2 + 7 * abs(s - rng_c / 7) + abs(z - col.min()) + 1e-6
        assert np.abs(rec - col).max() <= bound
        assert abs(s - rng_c / 7) <= (rng_c / 7) * 2.0 ** -11 + 1e-12
    # decode definition: scale*code + zero
    assert oracle.tq3_decode_value(5, int(np.float16(0.5).view(np.uint16)), int(np.float16(-2).view(np.uint16))) == 0.5


def test_value_rounding_is_half_to_even():
    d = 128
    v = np.zeros((16, d), np.float32)
    v[:, 0] = np.float32([0, 7, 0.5, 1.5, 2.5, 3.5, 4.5, 5.5, 6.5, 1, 2, 3, 4, 5, 6, 7])   # scale exactly 1
    code, sc, zp = oracle.tq3_encode_value_page(v)
    assert oracle.f16_to_f32(int(sc[0])) == 1.0 and oracle.f16_to_f32(int(zp[0])) == 0.0
    assert code[:, 0].tolist() == [0, 7, 0, 2, 2, 4, 4, 6, 6, 1, 2, 3, 4, 5, 6, 7]


@pytest.mark.parametrize("d", [128, 256])
def test_packed_record_is_a_bijection_of_its_fields(d):
    """Every field bit lands on its own record bit, every record bit is used, sizes follow
    16d + 32, and unpack inverts pack."""
    nbytes = oracle.tq3_record_bytes(d)
    assert nbytes == 16 * d + 32 and oracle.fp8_record_bytes(d) == 32 * d
    rng = np.random.default_rng(d)
    kc = rng.integers(0, 8, (16, d)).astype(np.uint8)
    vc = rng.integers(0, 8, (16, d)).astype(np.uint8)
    g = rng.integers(0, 65536, 16).astype(np.uint16)
    sc = rng.integers(0, 65536, d).astype(np.uint16)
    zp = rng.integers(0, 65536, d).astype(np.uint16)
    rec = oracle.tq3_pack_record(kc, g, vc, sc, zp)
    out = oracle.tq3_unpack_record(rec, d)
    for a, b in zip(out, (kc, g, vc, sc, zp)):
        assert np.array_equal(a, b)
    # all-ones fields fill every bit of the record
    full = oracle.tq3_pack_record(np.full((16, d), 7, np.uint8), np.full(16, 0xFFFF, np.uint16),
                                  np.full((16, d), 7, np.uint8), np.full(d, 0xFFFF, np.uint16),
                                  np.full(d, 0xFFFF, np.uint16))
    assert np.all(full == 0xFF)
    # single-bit probes: each lands on exactly one bit and no two coincide
    seen = np.zeros(nbytes * 8, bool)
    z16, zd = np.zeros(16, np.uint16), np.zeros(d, np.uint16)
    for which in range(2):
        for t in range(16):
            for i in range(0, d, 5):
                for bit in range(3):
                    a = np.zeros((16, d), np.uint8)
                    a[t, i] = 1 << bit
                    r = oracle.tq3_pack_record(a if which == 0 else 0 * a, z16, a if which == 1 else 0 * a, zd, zd)
                    bits = np.unpackbits(r, bitorder="little")
                    assert bits.sum() == 1
                    pos = int(np.argmax(bits))
                    assert not seen[pos]
                    seen[pos] = True
                    # code sections: K in [0, 6d), V in [6d, 12d)
                    assert (pos // 8) // (6 * d) == which
    # section offsets are multiples of 16 bytes
    for off in (0, 6 * d, 12 * d, 12 * d + 32):
        assert off % 16 == 0


def test_fp8_record_layout_token_major_keys_channel_major_values():
    d = 128
    k = np.zeros((16, d), np.float32)
    v = np.zeros((16, d), np.float32)
    k[3, 5] = 1.0
    v[3, 5] = -2.0
    rec = oracle.fp8_pack_record(k, v)
    nz = np.nonzero(rec)[0].tolist()
    assert nz == [3 * d + 5, 16 * d + 5 * 16 + 3]
    assert rec[3 * d + 5] == 0x38 and rec[16 * d + 5 * 16 + 3] == 0xC0
    k2, v2 = oracle.fp8_unpack_record_f32(rec, d)
    assert np.array_equal(k2, k) and np.array_equal(v2, v)
    # tokens beyond n_valid stay zero bytes
    rec = oracle.fp8_pack_record(np.ones((16, d), np.float32), np.ones((16, d), np.float32), n_valid=5)
    kk, vv = oracle.fp8_unpack_record_f32(rec, d)
    assert kk[:5].all() and not kk[5:].any() and vv[:5].all() and not vv[5:].any()


def test_demote_equals_encoding_the_dequantised_fp8_page():
    d = 128
    rng = np.random.default_rng(5)
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    k = rng.standard_normal((16, d)).astype(np.float32)
    v = rng.standard_normal((16, d)).astype(np.float32)
    rec8 = oracle.fp8_pack_record(k, v)
    kq, vq = oracle.fp8_unpack_record_f32(rec8, d)
    assert np.array_equal(oracle.demote_record(rec8, d, sigma), oracle.tq3_record_from_f32(kq, vq, sigma))
    # FP8 scales (stored = x / scale): power-of-two scales change bytes but not dequantised values
    rec8s = oracle.fp8_pack_record(k, v, 16, 0.5, 2.0)
    ks, vs = oracle.fp8_unpack_record_f32(rec8s, d, 0.5, 2.0)
    assert np.abs(ks - k).max() <= np.abs(k).max() * 2.0 ** -4 and np.abs(vs - v).max() <= np.abs(v).max() * 2.0 ** -4


@pytest.mark.parametrize("d", [128, 256])
def test_promote_reconstructs_the_decoded_page_up_to_fp8_rounding(d):
    """Promote (Algorithm 1 step 3): the FP8 page written from a TQ3 record dequantises to the fp64
    decode of that record within half an e4m3 step, and values that are e4m3-exact come back exactly."""
    rng = np.random.default_rng(31 + d)
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    k = rng.standard_normal((16, d)).astype(np.float32)
    v = rng.standard_normal((16, d)).astype(np.float32)
    v[:, 3] = 2.5                                         # constant channel: zero = 2.5, scale = 0
    v[:, 4] = np.float32([0, 7] * 8) * 0.5                # codes 0 / 7 with scale 0.5: values 0 and 3.5
    rec3 = oracle.tq3_record_from_f32(k, v, sigma)
    rec8 = oracle.promote_record(rec3, d, sigma)
    kq, vq = oracle.fp8_unpack_record_f32(rec8, d)
    kc, g, vc, sc, zp = oracle.tq3_unpack_record(rec3, d)
    for t in range(16):
        ref = oracle.tq3_decode_key(kc[t], int(g[t]), sigma)
        # e4m3 keeps 4 significant bits: relative half-step 2^-4, absolute 2^-10 in the subnormal range
        assert np.all(np.abs(kq[t] - ref) <= np.maximum(np.abs(ref) * 2.0 ** -4, 2.0 ** -10) + 1e-6)
    for c in range(d):
        ref = np.array([oracle.tq3_decode_value(int(vc[t, c]), int(sc[c]), int(zp[c])) for t in range(16)])
        assert np.all(np.abs(vq[:, c] - ref) <= np.maximum(np.abs(ref) * 2.0 ** -4, 2.0 ** -10) + 1e-6)
    assert np.all(vq[:, 3] == 2.5) and np.array_equal(vq[:, 4], np.float32([0, 3.5] * 8))
    # scales move the stored bytes, not the dequantised values
    rec8s = oracle.promote_record(rec3, d, sigma, 0.5, 2.0)
    ks, vs = oracle.fp8_unpack_record_f32(rec8s, d, 0.5, 2.0)
    assert np.abs(ks - kq).max() <= np.abs(kq).max() * 2.0 ** -3 and np.all(vs[:, 3] == 2.5)
