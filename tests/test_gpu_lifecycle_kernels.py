"""Bit-exact parity of the packing kernels with the oracle: Append (bf16 -> e4m3 records) and
Demote (FP8 record -> TQ3 record), through the C ABI, compared by raw page read-back."""
import numpy as np
import pytest
import torch

import mkv_workloads as W
import oracle
import paper_2608_23834_b200 as M
from _gpu_util import bf16_tensor

pytestmark = pytest.mark.gpu


def special_bf16(rng, shape):
    """N(0,1) with outliers plus values that exercise rounding ties, saturation, subnormals and zeros."""
    x = rng.standard_normal(shape).astype(np.float32)
    flat = x.reshape(-1)
    specials = np.float32([0.0, -0.0, 448.0, 449.0, 464.0, 480.0, 1e4, -1e4, 2.0 ** -10, 3 * 2.0 ** -10, 2.0 ** -9,
                           -2.0 ** -9, 17.0, 19.0, 0.0009765625, 1e-8, -1e-8, 0.28125, 0.296875, 240.0, 232.0])
    idx = rng.choice(flat.size, size=4 * len(specials), replace=False)
    flat[idx] = np.tile(specials, 4)
    return W.f32_to_bf16_bits(x)


@pytest.mark.parametrize("d,hkv,k_scale,v_scale", [(128, 2, 1.0, 1.0), (256, 4, 1.0, 1.0), (128, 1, 0.5, 2.0)])
def test_append_is_bit_exact(d, hkv, k_scale, v_scale):
    rng = np.random.default_rng(d + hkv)
    n_pages = 7
    pool = M.Pool(d, hkv, hkv * 4, n_pages, 1, np.ones(d, np.int8), k_scale, v_scale)
    n_tok = 16 * 5 + 3
    k_bits, v_bits = special_bf16(rng, (n_tok, hkv, d)), special_bf16(rng, (n_tok, hkv, d))
    # tokens land on shuffled pages, in order inside each page; two tokens are skipped (-1)
    page_of = rng.permutation(n_pages)[:6]
    slots = np.array([page_of[t // 16] * 16 + t % 16 for t in range(n_tok)], np.int32)
    skipped = [5, 40]
    slots[skipped] = -1
    # append in two calls to cover repeated launches
    for lo, hi in ((0, 30), (30, n_tok)):
        pool.append(bf16_tensor(k_bits[lo:hi]), bf16_tensor(v_bits[lo:hi]), torch.from_numpy(slots[lo:hi]).cuda())
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    kf, vf = oracle.bf16_bits_to_f32(k_bits), oracle.bf16_bits_to_f32(v_bits)
    for lp in range(6):
        got = pool.page_read_raw(M.FMT_FP8, int(page_of[lp])).reshape(hkv, 32 * d)
        for h in range(hkv):
            kk = np.zeros((16, d), np.float32)
            vv = np.zeros((16, d), np.float32)
            n = min(16, n_tok - 16 * lp)
            kk[:n], vv[:n] = kf[16 * lp:16 * lp + n, h], vf[16 * lp:16 * lp + n, h]
            ref = oracle.fp8_pack_record(kk, vv, n, k_scale, v_scale).copy()
            for t in skipped:                       # skipped tokens leave the zero-filled slot untouched
                if t // 16 == lp:
                    ref[:16 * d].reshape(16, d)[t % 16] = 0
                    ref[16 * d:].reshape(d, 16)[:, t % 16] = 0
            assert np.array_equal(got[h], ref), (lp, h)
    # the untouched page is still zero
    assert not pool.page_read_raw(M.FMT_FP8, int(np.setdiff1d(np.arange(n_pages), page_of)[0])).any()


@pytest.mark.parametrize("d,hkv,k_scale,v_scale", [(128, 2, 1.0, 1.0), (256, 4, 0.5, 2.0)])
def test_prefill_sized_append_is_bit_exact(d, hkv, k_scale, v_scale):
    """One call of many tokens: groups of 16 input tokens that fill a page front to back take the
    transposing path, every other group (a skipped token, a run that starts inside a page, a page that
    does not exist, the ragged tail) the per-token path; both must write the same bytes."""
    rng = np.random.default_rng(7 * d + hkv)
    n_pages = 12
    pool = M.Pool(d, hkv, hkv * 2, n_pages, 1, np.ones(d, np.int8), k_scale, v_scale)
    page_of = rng.permutation(n_pages)
    plan = []                                            # (page, first slot, tokens) per input group, in input order
    plan += [(int(page_of[i]), 0, 16) for i in range(4)]             # whole pages
    plan += [(int(page_of[4]), 0, 16)]                               # whole page with one skipped token (below)
    plan += [(int(page_of[5]), 0, 16)]                               # whole page, slots permuted (below)
    plan += [(n_pages + 3, 0, 16)]                                   # a page beyond the arena: flagged, not written
    plan += [(int(page_of[6]), 8, 8), (int(page_of[7]), 0, 8)]       # one input group over two half pages
    plan += [(int(page_of[8]), 0, 16)]                               # aligned again
    plan += [(int(page_of[9]), 0, 5)]                                # ragged tail
    slots = np.concatenate([p * 16 + s0 + np.arange(n) for p, s0, n in plan]).astype(np.int32)
    skipped = 4 * 16 + 9
    slots[skipped] = -1
    perm = 5 * 16 + rng.permutation(16)
    slots[5 * 16:6 * 16] = slots[perm]
    n_tok = len(slots)
    k_bits, v_bits = special_bf16(rng, (n_tok, hkv, d)), special_bf16(rng, (n_tok, hkv, d))
    pool.append(bf16_tensor(k_bits), bf16_tensor(v_bits), torch.from_numpy(slots).cuda())
    torch.cuda.synchronize()
    assert pool.status() == M.E_BOUNDS and pool.status() == M.OK
    kf, vf = oracle.bf16_bits_to_f32(k_bits), oracle.bf16_bits_to_f32(v_bits)
    want = {}                                            # page -> (k [16][d], v [16][d], filled slots) per head
    for t, sm in enumerate(slots):
        if sm < 0 or sm // 16 >= n_pages:
            continue
        kk, vv, used = want.setdefault(int(sm) // 16, (np.zeros((hkv, 16, d), np.float32), np.zeros((hkv, 16, d), np.float32), set()))
        kk[:, sm % 16], vv[:, sm % 16] = kf[t], vf[t]
        used.add(int(sm) % 16)
    assert len(want) == 10
    for page in range(n_pages):
        got = pool.page_read_raw(M.FMT_FP8, page).reshape(hkv, 32 * d)
        if page not in want:
            assert not got.any()
            continue
        kk, vv, used = want[page]
        for h in range(hkv):
            ref = oracle.fp8_pack_record(kk[h], vv[h], 16, k_scale, v_scale).copy()
            for s in set(range(16)) - used:              # slots never written stay zero
                ref[:16 * d].reshape(16, d)[s] = 0
                ref[16 * d:].reshape(d, 16)[:, s] = 0
            assert np.array_equal(got[h], ref), (page, h)


@pytest.mark.parametrize("d,hkv,k_scale,v_scale", [(128, 2, 1.0, 1.0), (256, 4, 1.0, 1.0), (256, 1, 0.25, 4.0)])
def test_demote_is_bit_exact_and_publishes_after_the_copy(d, hkv, k_scale, v_scale):
    rng = np.random.default_rng(100 + d + hkv)
    n = 9
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    pool = M.Pool(d, hkv, hkv, n, n + 2, sigma, k_scale, v_scale)
    recs = np.zeros((n, hkv, 32 * d), np.uint8)
    for p in range(n):
        for h in range(hkv):
            k = rng.standard_normal((16, d)).astype(np.float32)
            v = rng.standard_normal((16, d)).astype(np.float32)
            k[:, rng.integers(0, d, 3)] *= 8
            v[:, rng.integers(0, d, 3)] *= 8
            if p == 1:
                k[3] = 0.0                   # zero key vector -> codes 0, g = 0
                v[:, 5] = 1.5                # constant channel -> scale 0
                v[:, 6] = 0.0
            if p == 2:
                v[:, 7] = np.float32([0, 7, 0.5, 1.5, 2.5, 3.5, 4.5, 5.5, 6.5, 1, 2, 3, 4, 5, 6, 7])   # rounding ties
                v[::2, 9], v[1::2, 9] = 0.0, -0.0
            recs[p, h] = oracle.fp8_pack_record(k, v, 16, k_scale, v_scale)
        pool.page_write_raw(M.FMT_FP8, p, recs[p])
    src = torch.from_numpy(rng.permutation(n).astype(np.int32)).cuda()
    dst = torch.from_numpy((rng.permutation(n + 2)[:n]).astype(np.int32)).cuda()
    bt = torch.full((3, 8), -1, dtype=torch.int32, device="cuda:0")
    tags = torch.zeros((3, 8), dtype=torch.uint8, device="cuda:0")
    entry = torch.arange(n, dtype=torch.int64, device="cuda:0") * 2
    entry[4] = -1                                       # one page is encoded but not published
    pool.demote(src, dst, bt, tags, entry)
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    s, t = src.cpu().numpy(), dst.cpu().numpy()
    for i in range(n):
        got = pool.page_read_raw(M.FMT_TQ3, int(t[i])).reshape(hkv, 16 * d + 32)
        for h in range(hkv):
            ref = oracle.demote_record(recs[s[i], h], d, sigma, k_scale, v_scale)
            assert np.array_equal(got[h], ref), (i, h, np.nonzero(got[h] != ref)[0][:8])
        # the source page is untouched
        assert np.array_equal(pool.page_read_raw(M.FMT_FP8, int(s[i])).reshape(hkv, 32 * d), recs[s[i]])
    btc, tc = bt.cpu().numpy().reshape(-1), tags.cpu().numpy().reshape(-1)
    for i in range(n):
        if i == 4:
            continue
        assert btc[2 * i] == t[i] and tc[2 * i] == M.TAG_STALE
    assert (btc[1::2] == -1).all() and (tc[1::2] == 0).all() and btc[8] == -1 and tc[8] == 0


@pytest.mark.parametrize("fmt", [1, 2])
@pytest.mark.parametrize("d,hkv,k_scale,v_scale", [(256, 2, 1.0, 1.0), (128, 3, 1.0, 0.37), (256, 1, 3.0, 3.0),
                                                    (128, 2, 2.0 ** -24, 2.0 ** -24), (128, 2, 1.0e7, 1.0e7)])
def test_demote_of_arbitrary_byte_patterns_is_bit_exact(d, hkv, k_scale, v_scale, fmt):
    """FP8 records filled with random bytes (every finite e4m3 value, subnormals, both zeros, +-448): value
    channels whose range is 7 * 2^k or 7 * 3 * 2^k put many quotients exactly on a half-integer, large and tiny
    values in one channel stress the quotient's rounding, and scales outside 2^-20 .. 2^20 take the encoder's
    other division path.  The record bytes must equal the oracle's in every case."""
    with oracle.record_format(fmt):
        rng = np.random.default_rng(7 * d + hkv + fmt)
        n = 12
        sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
        pool = M.Pool(d, hkv, hkv, n, n, sigma, k_scale, v_scale, tq3_format=fmt)
        recs = rng.integers(0, 256, (n, hkv, 32 * d), dtype=np.uint8)
        recs[(recs & 0x7F) == 0x7F] = 0x38                       # no NaN bytes
        # a few pages with small magnitudes only (|x| < 2: ranges on the e4m3 grid, many exact ties)
        small = recs[:4]
        small &= 0xBF
        for p in range(n):
            pool.page_write_raw(M.FMT_FP8, p, recs[p])
        ids = torch.arange(n, dtype=torch.int32, device="cuda:0")
        pool.demote(ids, ids)
        torch.cuda.synchronize()
        assert pool.status() == M.OK
        for p in range(n):
            got = pool.page_read_raw(M.FMT_TQ3, p).reshape(hkv, 16 * d + 32)
            for h in range(hkv):
                ref = oracle.demote_record(recs[p, h], d, sigma, k_scale, v_scale)
                assert np.array_equal(got[h], ref), (p, h, np.nonzero(got[h] != ref)[0][:8])


@pytest.mark.parametrize("fmt", [1, 2])
@pytest.mark.parametrize("d,hkv,k_scale,v_scale", [(256, 2, 1.0, 1.0), (128, 3, 1.0, 1.0), (256, 1, 0.5, 4.0), (128, 2, 3.0, 0.37)])
def test_promote_of_arbitrary_records_is_bit_exact(d, hkv, k_scale, v_scale, fmt):
    """TQ3 records filled with random bytes: every code pattern in every position, norm corrections, scales and
    zeros anywhere in the finite fp16 range below 2.  The rebuilt FP8 pages must equal the oracle's byte for byte
    (format 2 rebuilds the keys by an integer matrix product, format 1 by butterflies)."""
    with oracle.record_format(fmt):
        rng = np.random.default_rng(31 * d + hkv + fmt)
        n = 10
        sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
        pool = M.Pool(d, hkv, hkv, n, n, sigma, k_scale, v_scale, tq3_format=fmt)
        recs = rng.integers(0, 256, (n, hkv, 16 * d + 32), dtype=np.uint8)
        meta = recs[:, :, 12 * d:].view(np.uint16)
        meta &= 0xBFFF                                        # clear the top exponent bit: finite, |x| < 2
        recs[0, :, 12 * d:12 * d + 32] = 0                    # a page whose norm corrections are all zero
        for p in range(n):
            pool.page_write_raw(M.FMT_TQ3, p, recs[p])
        ids = torch.arange(n, dtype=torch.int32, device="cuda:0")
        pool.promote(ids, ids)
        torch.cuda.synchronize()
        assert pool.status() == M.OK
        for p in range(n):
            got = pool.page_read_raw(M.FMT_FP8, p).reshape(hkv, 32 * d)
            for h in range(hkv):
                ref = oracle.promote_record(recs[p, h], d, sigma, k_scale, v_scale)
                assert np.array_equal(got[h], ref), (p, h, np.nonzero(got[h] != ref)[0][:8])


def test_out_of_range_ids_are_flagged_not_dereferenced():
    d, hkv = 128, 1
    pool = M.Pool(d, hkv, 4, 4, 4, np.ones(d, np.int8))
    k = torch.zeros((2, hkv, d), dtype=torch.bfloat16, device="cuda:0")
    pool.append(k, k, torch.tensor([4 * 16, 16], dtype=torch.int32, device="cuda:0"))     # page 4 does not exist
    assert pool.status() == M.E_BOUNDS and pool.status() == M.OK
    pool.demote(torch.tensor([0, 9], dtype=torch.int32, device="cuda:0"), torch.tensor([0, 1], dtype=torch.int32, device="cuda:0"))
    assert pool.status() == M.E_BOUNDS
    pool.demote(torch.tensor([0], dtype=torch.int32, device="cuda:0"), torch.tensor([-3], dtype=torch.int32, device="cuda:0"))
    assert pool.status() == M.E_BOUNDS


def test_an_entry_index_beyond_the_tables_is_flagged_and_nothing_is_published():
    d, hkv, n = 128, 2, 3
    pool = M.Pool(d, hkv, hkv, 2 * n, 2 * n, np.ones(d, np.int8))
    k = torch.randn((16 * n, hkv, d), device="cuda:0").to(torch.bfloat16)
    pool.append(k, k, torch.arange(16 * n, dtype=torch.int32, device="cuda:0"))
    ids = torch.arange(n, dtype=torch.int32, device="cuda:0")
    buf_bt = torch.full((8 + 16,), -7, dtype=torch.int32, device="cuda:0")       # the tables are the first 8 entries
    buf_tg = torch.full((8 + 16,), 9, dtype=torch.uint8, device="cuda:0")
    bt, tags = buf_bt[:8], buf_tg[:8]
    entry = torch.tensor([2, 8, 10 ** 9], dtype=torch.int64, device="cuda:0")     # one good, two beyond the tables
    pool.demote(ids, ids, bt, tags, entry)
    torch.cuda.synchronize()
    assert pool.status() == M.E_BOUNDS
    assert buf_bt.cpu().tolist() == [-7, -7, 0] + [-7] * 21 and buf_tg.cpu().tolist() == [9, 9, M.TAG_STALE] + [9] * 21
    pool.promote(ids, (ids + n).contiguous(), bt, tags, entry)
    torch.cuda.synchronize()
    assert pool.status() == M.E_BOUNDS
    assert buf_bt.cpu().tolist() == [-7, -7, n] + [-7] * 21 and buf_tg.cpu().tolist() == [9, 9, M.TAG_ANCHOR] + [9] * 21
    with pytest.raises(M.MkvError) as e:
        pool.set_anchor(tags, 8, True)
    assert e.value.code == M.E_BOUNDS


def test_set_anchor_flips_fp8_tags_and_refuses_stale():
    pool = M.Pool(128, 1, 4, 4, 4, np.ones(128, np.int8))
    tags = torch.tensor([[0, 0, 2, 1]], dtype=torch.uint8, device="cuda:0")
    pool.set_anchor(tags, 1, True)
    pool.set_anchor(tags, 3, False)
    assert pool.status() == M.OK
    assert tags.cpu().numpy().tolist() == [[0, 1, 2, 0]]
    pool.set_anchor(tags, 2, True)            # Stale must be promoted first
    assert pool.status() == M.E_STATE
    assert tags.cpu().numpy().tolist() == [[0, 1, 2, 0]]


@pytest.mark.parametrize("d,hkv,k_scale,v_scale", [(128, 2, 1.0, 1.0), (256, 4, 1.0, 1.0), (128, 1, 0.5, 2.0)])
def test_promote_is_bit_exact_and_publishes_anchor(d, hkv, k_scale, v_scale):
    rng = np.random.default_rng(200 + d + hkv)
    n = 6
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    pool = M.Pool(d, hkv, hkv, n + 2, n, sigma, k_scale, v_scale)
    recs = np.zeros((n, hkv, 16 * d + 32), np.uint8)
    for p in range(n):
        for h in range(hkv):
            k = rng.standard_normal((16, d)).astype(np.float32)
            v = rng.standard_normal((16, d)).astype(np.float32)
            k[:, rng.integers(0, d, 3)] *= 8
            v[:, rng.integers(0, d, 3)] *= 8
            if p == 0:
                k[2] = 0.0
                v[:, 1] = -0.75
            recs[p, h] = oracle.tq3_record_from_f32(k, v, sigma)
        pool.page_write_raw(M.FMT_TQ3, p, recs[p])
    src = torch.from_numpy(rng.permutation(n).astype(np.int32)).cuda()
    dst = torch.from_numpy(rng.permutation(n + 2)[:n].astype(np.int32)).cuda()
    bt = torch.full((2, 8), -1, dtype=torch.int32, device="cuda:0")
    tags = torch.full((2, 8), 2, dtype=torch.uint8, device="cuda:0")
    entry = torch.arange(n, dtype=torch.int64, device="cuda:0") * 2 + 1
    pool.promote(src, dst, bt, tags, entry)
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    s, t = src.cpu().numpy(), dst.cpu().numpy()
    for i in range(n):
        got = pool.page_read_raw(M.FMT_FP8, int(t[i])).reshape(hkv, 32 * d)
        for h in range(hkv):
            ref = oracle.promote_record(recs[s[i], h], d, sigma, k_scale, v_scale)
            assert np.array_equal(got[h], ref), (i, h, np.nonzero(got[h] != ref)[0][:8])
        assert np.array_equal(pool.page_read_raw(M.FMT_TQ3, int(s[i])).reshape(hkv, -1), recs[s[i]])   # source untouched
    btc, tc = bt.cpu().numpy().reshape(-1), tags.cpu().numpy().reshape(-1)
    for i in range(n):
        assert btc[2 * i + 1] == t[i] and tc[2 * i + 1] == M.TAG_ANCHOR
    assert (btc[0::2] == -1).all() and (tc[0::2] == 2).all()
    pool.promote(torch.tensor([99], dtype=torch.int32, device="cuda:0"), torch.tensor([0], dtype=torch.int32, device="cuda:0"))
    assert pool.status() == M.E_BOUNDS


@pytest.mark.parametrize("d,hkv", [(128, 1), (128, 3), (256, 6), (128, 12), (256, 16)])
def test_demote_then_promote_for_every_head_split(d, hkv):
    """The blocks of a page's cluster share out the KV heads (1, 3, 6 blocks of one head; 6 blocks of two;
    8 blocks of two): every head's record is bit-exact both ways and both calls publish once."""
    rng = np.random.default_rng(300 + d + hkv)
    n = 5
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    pool = M.Pool(d, hkv, hkv, 2 * n, n, sigma)
    recs = np.zeros((n, hkv, 32 * d), np.uint8)
    for p in range(n):
        for h in range(hkv):
            k = rng.standard_normal((16, d)).astype(np.float32) * (1 + h)
            v = rng.standard_normal((16, d)).astype(np.float32)
            v[:, rng.integers(0, d, 2)] *= 8
            recs[p, h] = oracle.fp8_pack_record(k, v, 16, 1.0, 1.0)
        pool.page_write_raw(M.FMT_FP8, p, recs[p])
    ids = torch.arange(n, dtype=torch.int32, device="cuda:0")
    bt = torch.full((1, n), -1, dtype=torch.int32, device="cuda:0")
    tags = torch.zeros((1, n), dtype=torch.uint8, device="cuda:0")
    entry = torch.arange(n, dtype=torch.int64, device="cuda:0")
    pool.demote(ids, ids.flip(0).contiguous(), bt, tags, entry)
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    assert bt.cpu().numpy().tolist() == [list(range(n - 1, -1, -1))] and (tags.cpu().numpy() == M.TAG_STALE).all()
    stale = np.zeros((n, hkv, 16 * d + 32), np.uint8)
    for p in range(n):
        stale[p] = pool.page_read_raw(M.FMT_TQ3, n - 1 - p).reshape(hkv, -1)
        for h in range(hkv):
            assert np.array_equal(stale[p, h], oracle.demote_record(recs[p, h], d, sigma, 1.0, 1.0)), (p, h)
    pool.promote(ids.flip(0).contiguous(), ids + n, bt, tags, entry)
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    assert bt.cpu().numpy().tolist() == [list(range(n, 2 * n))] and (tags.cpu().numpy() == M.TAG_ANCHOR).all()
    for p in range(n):
        got = pool.page_read_raw(M.FMT_FP8, n + p).reshape(hkv, 32 * d)
        for h in range(hkv):
            assert np.array_equal(got[h], oracle.promote_record(stale[p, h], d, sigma, 1.0, 1.0)), (p, h)


@pytest.mark.parametrize("d,hkv", [(128, 8), (256, 4)])
def test_bulk_calls_write_the_same_bytes_as_small_calls(d, hkv):
    """A call of hundreds of pages keeps a page's heads in one block, a call of a few pages spreads them
    over a cluster: both layouts of the work must produce identical arenas (and match the oracle)."""
    rng = np.random.default_rng(400 + d)
    n = 320
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    pool = M.Pool(d, hkv, hkv, 2 * n, 2 * n, sigma)
    k, v = bf16_tensor(special_bf16(rng, (16 * n, hkv, d))), bf16_tensor(special_bf16(rng, (16 * n, hkv, d)))
    pool.append(k, v, torch.arange(16 * n, dtype=torch.int32, device="cuda:0"))
    ids = torch.arange(n, dtype=torch.int32, device="cuda:0")
    pool.demote(ids, ids)                                   # one bulk call -> TQ3 pages 0 .. n-1
    for lo in range(0, n, 8):                               # small calls -> TQ3 pages n .. 2n-1
        pool.demote(ids[lo:lo + 8], (ids[lo:lo + 8] + n).contiguous())
    pool.promote(ids, (ids + n).contiguous())               # bulk -> FP8 pages n .. 2n-1
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    rec3 = hkv * (16 * d + 32)
    tq3 = pool.tq3_arena[:2 * n * rec3].view(2, n * rec3)
    assert torch.equal(tq3[0], tq3[1])
    rec8 = hkv * 32 * d
    bulk_fp8 = pool.fp8_arena[n * rec8:2 * n * rec8].clone()
    for lo in range(0, n, 8):                               # small promote calls over the same target pages
        pool.promote((ids[lo:lo + 8] + n).contiguous(), (ids[lo:lo + 8] + n).contiguous())
    torch.cuda.synchronize()
    assert torch.equal(bulk_fp8, pool.fp8_arena[n * rec8:2 * n * rec8])
    for p in (0, 157, n - 1):
        src = pool.page_read_raw(M.FMT_FP8, p).reshape(hkv, 32 * d)
        got = pool.page_read_raw(M.FMT_TQ3, p).reshape(hkv, -1)
        for h in range(hkv):
            assert np.array_equal(got[h], oracle.demote_record(src[h], d, sigma, 1.0, 1.0)), (p, h)
