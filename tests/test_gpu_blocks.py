"""Pages of 16 M tokens (the paper's blocks of 1,792 / 832 tokens) through the C ABI: Append, Demote and
Promote byte for byte against the oracle, decode attention within the attention tolerance."""
import numpy as np
import pytest
import torch

import mkv_workloads as W
import oracle
import paper_2608_23834_b200 as M
from _gpu_util import Case, bf16_tensor, check_case, check_close

pytestmark = pytest.mark.gpu


def _kv_bits(rng, n_tok, hkv, d):
    k = rng.standard_normal((n_tok, hkv, d)).astype(np.float32)
    v = rng.standard_normal((n_tok, hkv, d)).astype(np.float32)
    k[:, :, rng.integers(0, d, 3)] *= 8
    v[:, :, rng.integers(0, d, 3)] *= 8
    return W.f32_to_bf16_bits(k), W.f32_to_bf16_bits(v)


@pytest.mark.parametrize("d,hkv,page_tokens", [(128, 2, 48), (256, 4, 832), (128, 3, 1792)])
def test_append_demote_promote_of_big_pages_are_bit_exact(d, hkv, page_tokens):
    rng = np.random.default_rng(d + page_tokens)
    Mt = page_tokens // 16
    n_pages = 3
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    pool = M.Pool(d, hkv, hkv, 2 * n_pages + 1, n_pages + 1, sigma, page_tokens=page_tokens)
    assert pool.fp8_rec == oracle.fp8_block_bytes(d, Mt) and pool.tq3_rec == oracle.tq3_block_bytes(d, Mt)
    n_tok = n_pages * page_tokens
    k_bits, v_bits = _kv_bits(rng, n_tok, hkv, d)
    # channels whose extremes are zeros of both signs (the sign of the earliest one goes into the record), a
    # constant channel, and an all-zero key vector
    v_bits[:, :, 9] = np.where(np.arange(n_tok) % 5 == 1, 0x8000, 0x0000).astype(np.uint16)[:, None]
    v_bits[:, :, 10] = np.where(np.arange(n_tok) % 7 == 0, 0x0000, 0x8000).astype(np.uint16)[:, None]
    v_bits[:, :, 11] = W.f32_to_bf16_bits(np.float32([1.5]))[0]
    v_bits[:, :, 12] = np.where(np.arange(n_tok) % 3 == 2, 0x8000, W.f32_to_bf16_bits(np.float32([-2.0]))[0]).astype(np.uint16)[:, None]
    k_bits[page_tokens + 3] = 0
    page_of = rng.permutation(2 * n_pages + 1)[:n_pages]
    slots = np.concatenate([p * page_tokens + np.arange(page_tokens) for p in page_of]).astype(np.int32)
    # one prefill-sized call for most tokens, the last 20 tokens one decode-sized call each way
    cut = n_tok - 20
    pool.append(bf16_tensor(k_bits[:cut]), bf16_tensor(v_bits[:cut]), torch.from_numpy(slots[:cut]).cuda())
    pool.append(bf16_tensor(k_bits[cut:]), bf16_tensor(v_bits[cut:]), torch.from_numpy(slots[cut:]).cuda())
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    kf, vf = oracle.bf16_bits_to_f32(k_bits), oracle.bf16_bits_to_f32(v_bits)
    fp8_pages = np.zeros((n_pages, hkv, pool.fp8_rec), np.uint8)
    for i, p in enumerate(page_of):
        got = pool.page_read_raw(M.FMT_FP8, int(p)).reshape(hkv, -1)
        for h in range(hkv):
            fp8_pages[i, h] = oracle.fp8_pack_block(kf[i * page_tokens:(i + 1) * page_tokens, h],
                                                    vf[i * page_tokens:(i + 1) * page_tokens, h])
            assert np.array_equal(got[h], fp8_pages[i, h]), ("append", i, h)
    # Demote: page scale/zero over all tokens, tiles, publication
    src = torch.from_numpy(page_of.astype(np.int32)).cuda()
    dst_ids = rng.permutation(n_pages + 1)[:n_pages].astype(np.int32)
    dst = torch.from_numpy(dst_ids).cuda()
    bt = torch.full((1, 2 * n_pages), -1, dtype=torch.int32, device="cuda:0")
    tags = torch.zeros((1, 2 * n_pages), dtype=torch.uint8, device="cuda:0")
    entry = torch.arange(n_pages, dtype=torch.int64, device="cuda:0") * 2
    entry[1] = -1
    pool.demote(src, dst, bt, tags, entry)
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    tq3_pages = np.zeros((n_pages, hkv, pool.tq3_rec), np.uint8)
    for i in range(n_pages):
        got = pool.page_read_raw(M.FMT_TQ3, int(dst_ids[i])).reshape(hkv, -1)
        for h in range(hkv):
            tq3_pages[i, h] = oracle.demote_block(fp8_pages[i, h], d, Mt, sigma)
            bad = np.nonzero(got[h] != tq3_pages[i, h])[0]
            assert bad.size == 0, ("demote", i, h, bad[:8], bad.size)
    btc, tc = bt.cpu().numpy()[0], tags.cpu().numpy()[0]
    assert btc[0] == dst_ids[0] and tc[0] == M.TAG_STALE and btc[2] == -1 and tc[2] == 0 and btc[4] == dst_ids[2]
    # Promote into other FP8 pages
    free_fp8 = np.setdiff1d(np.arange(2 * n_pages + 1), page_of)[:n_pages].astype(np.int32)
    entry2 = torch.arange(n_pages, dtype=torch.int64, device="cuda:0") * 2 + 1
    pool.promote(dst, torch.from_numpy(free_fp8).cuda(), bt, tags, entry2)
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    for i in range(n_pages):
        got = pool.page_read_raw(M.FMT_FP8, int(free_fp8[i])).reshape(hkv, -1)
        for h in range(hkv):
            assert np.array_equal(got[h], oracle.promote_block(tq3_pages[i, h], d, Mt, sigma)), ("promote", i, h)
    assert (bt.cpu().numpy()[0, 1::2] == free_fp8).all() and (tags.cpu().numpy()[0, 1::2] == M.TAG_ANCHOR).all()
    # ids out of range are flagged, not dereferenced
    pool.demote(torch.tensor([99], dtype=torch.int32, device="cuda:0"), torch.tensor([0], dtype=torch.int32, device="cuda:0"))
    assert pool.status() == M.E_BOUNDS
    pool.promote(torch.tensor([0], dtype=torch.int32, device="cuda:0"), torch.tensor([-1], dtype=torch.int32, device="cuda:0"))
    assert pool.status() == M.E_BOUNDS


@pytest.mark.parametrize("d,hkv,group,page_tokens,lens", [
    (128, 2, 4, 48, (5 * 48 + 37, 2 * 48, 0, 17)),
    (256, 2, 6, 832, (7 * 832 + 400, 3 * 832 + 1)),
    (128, 1, 8, 1792, (9 * 1792 + 5,)),
])
def test_decode_over_big_pages_matches_the_oracle(d, hkv, group, page_tokens, lens):
    spec = W.config(0, seq_lens=lens, head_dim=d, n_kv_heads=hkv, group=group, anchor_prefix=page_tokens, anchor_spans=1,
                    anchor_span_tokens=page_tokens, recent_tokens=page_tokens + 5, page_tokens=page_tokens, seed=21 + d)
    case = Case(spec, extra_fp8=2, extra_tq3=3)
    assert (case.tab.tier_tag[0, :spec.n_pages(0)] == W.TAG_STALE).sum() >= 2
    out, lse = case.run()
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)
    # the CUDA-core kernel, a second implementation of the page layout, agrees
    out_s, lse_s = case.run(M.DECODE_SCALAR)
    check_case(case, out_s, lse_s, ref, ref_lse)
    # the tcgen05 kernel has no support for several tiles per page and refuses the call
    case.pool.set_decode_variant(M.DECODE_TMEM)
    with pytest.raises(M.MkvError):
        case.pool.decode_attention(case.q, case.bt, case.tags, case.lens, spec.scale)
    case.pool.set_decode_variant(M.DECODE_TENSOR)
    # the refusals launched nothing and left the pool usable
    out2, _ = case.run()
    assert np.array_equal(out, out2)


def test_canary_shape_with_1792_token_pages_full_size():
    """2 x 59,008 tokens, d = 256, 4 KV x 6 query heads, 33 pages of 1,792 tokens per request (10 FP8 + 23 TQ3):
    the whole layer through the benchmark's launch shape, one KV head of one request against the oracle."""
    spec = W.config(5)
    case = Case(spec)
    out, lse = case.run()
    ref, ref_lse = case.reference(only_b=1, only_h=2)
    g = spec.group
    for hq in range(2 * g, 3 * g):
        check_close(out[1, hq], ref[1, hq], f"cfg5 b=1 hq={hq}")
        assert abs(lse[1, hq] - ref_lse[1, hq]) < 2e-3
    assert np.isfinite(out).all() and out.any()
    # physical bytes of the layer: 20 FP8 + 46 TQ3 pages of 4 heads
    assert case.pool.fp8_rec * 4 * 20 + case.pool.tq3_rec * 4 * 46 == 4 * (20 * 917_504 + 46 * 348_672)


def test_runs_longer_than_a_round_park_and_fold_across_rounds():
    """8 x 32,256 tokens, d = 128, 8 KV heads, pages of 1,792 tokens, half of them Stale: every warp scans more than
    64 tiles, so its page lists are rebuilt and the parked accumulators carried from round to round."""
    spec = W.config(4, batch=8, ctx=18 * 1792, stale_fraction=0.5, page_tokens=1792)
    case = Case(spec, requests=[3])
    n_units = sum((n + 15) // 16 for n in spec.seq_lens) * spec.n_kv_heads
    assert n_units / (148 * 12) > 64
    out, lse = case.run()
    ref, ref_lse = case.reference(only_b=3, only_h=5)
    g = spec.group
    for hq in range(5 * g, 6 * g):
        check_close(out[3, hq], ref[3, hq], f"b=3 hq={hq}")
        assert abs(lse[3, hq] - ref_lse[3, hq]) < 2e-3
    assert np.isfinite(out).all()


@pytest.mark.parametrize("seed", range(6))
def test_random_page_sizes_lengths_and_tier_mixes(seed):
    """Drawn shapes: page size, head geometry, ragged lengths (empty, shorter than a tile, partial last pages), tier
    mix; the tensor-core kernel and the CUDA-core kernel against the oracle, plus the page mass."""
    rng = np.random.default_rng(1000 + seed)
    page_tokens = int(rng.choice([32, 48, 80, 160, 256, 1024]))
    d = int(rng.choice([128, 256]))
    hkv = int(rng.choice([1, 2, 3]))
    group = int(rng.choice([1, 4, 6, 8]))
    batch = int(rng.integers(1, 5))
    lens = [int(rng.choice([0, 5, page_tokens, int(rng.integers(1, 9 * page_tokens))])) for _ in range(batch)]
    lens[0] = int(rng.integers(3 * page_tokens, 12 * page_tokens))
    spec = W.config(0, seq_lens=lens, head_dim=d, n_kv_heads=hkv, group=group, anchor_prefix=page_tokens * int(rng.integers(0, 2)),
                    anchor_spans=int(rng.integers(0, 3)), anchor_span_tokens=page_tokens,
                    recent_tokens=int(rng.integers(1, 3 * page_tokens)), page_tokens=page_tokens, seed=50 + seed)
    case = Case(spec, extra_fp8=1, extra_tq3=1)
    out, lse = case.run()
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)
    out_s, lse_s = case.run(M.DECODE_SCALAR)
    check_case(case, out_s, lse_s, ref, ref_lse)
    case.pool.set_decode_variant(M.DECODE_TENSOR)
    _, _, mass = case.pool.decode_attention_scored(case.q, case.bt, case.tags, case.lens, spec.scale)
    torch.cuda.synchronize()
    assert case.pool.status() == M.OK
    want = oracle.page_mass(case.L.fp8_arena, case.L.tq3_arena, d, hkv, group, case.L.sigma, case.L.q_bits, case.tab.block_table,
                            case.tab.tier_tag, case.tab.seq_lens, spec.scale, page_tokens=page_tokens)
    got = mass.cpu().numpy().astype(np.float64)
    assert (np.abs(got - want) <= 1e-6 + 1e-4 * want).all(), np.abs(got - want).max()


def test_publication_of_big_pages_in_small_and_large_calls():
    """Pages of several tiles are written by many blocks; the table entry of a page may appear only after all of
    them.  Small calls publish from inside the tile kernel (the cluster that draws the page's last ticket), large
    calls with a kernel of their own.  Both must publish every page exactly as asked, the ticket counters must be
    back at zero (a second small call works), and the records must be the oracle's."""
    d, hkv, page_tokens = 128, 2, 48
    Mt = page_tokens // 16
    rng = np.random.default_rng(11)
    n_big, n_small = 60, 5
    n_pages = n_big + 2 * n_small
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    pool = M.Pool(d, hkv, hkv, n_pages, n_pages, sigma, page_tokens=page_tokens)
    k_bits, v_bits = _kv_bits(rng, n_pages * page_tokens, hkv, d)
    slots = torch.arange(n_pages * page_tokens, dtype=torch.int32, device="cuda:0")
    pool.append(bf16_tensor(k_bits), bf16_tensor(v_bits), slots)
    kf, vf = oracle.bf16_bits_to_f32(k_bits), oracle.bf16_bits_to_f32(v_bits)
    bt = torch.full((1, n_pages), -1, dtype=torch.int32, device="cuda:0")
    tags = torch.zeros((1, n_pages), dtype=torch.uint8, device="cuda:0")
    calls = [(0, n_big), (n_big, n_big + n_small), (n_big + n_small, n_pages)]      # large, small, small again
    for lo, hi in calls:
        ids = torch.arange(lo, hi, dtype=torch.int32, device="cuda:0")
        dst = torch.arange(hi - 1, lo - 1, -1, dtype=torch.int32, device="cuda:0")     # reversed inside the call
        entry = torch.arange(lo, hi, dtype=torch.int64, device="cuda:0")
        if hi - lo == n_small:
            entry[2] = -1                                                              # encoded, not published
        pool.demote(ids, dst, bt, tags, entry)
        torch.cuda.synchronize()
        assert pool.status() == M.OK
        btc, tc = bt.cpu().numpy()[0], tags.cpu().numpy()[0]
        for i in range(lo, hi):
            if hi - lo == n_small and i == lo + 2:
                assert btc[i] == -1 and tc[i] == 0
            else:
                assert btc[i] == lo + hi - 1 - i and tc[i] == M.TAG_STALE, (lo, hi, i)
    for page in (3, n_big + 1, n_pages - 1):
        lo, hi = next(c for c in calls if c[0] <= page < c[1])
        got = pool.page_read_raw(M.FMT_TQ3, lo + hi - 1 - page).reshape(hkv, -1)
        for h in range(hkv):
            fp8 = oracle.fp8_pack_block(kf[page * page_tokens:(page + 1) * page_tokens, h],
                                        vf[page * page_tokens:(page + 1) * page_tokens, h])
            assert np.array_equal(got[h], oracle.demote_block(fp8, d, Mt, sigma)), (page, h)
    # and back: a large and a small Promote call
    for lo, hi in ((0, n_big), (n_big, n_big + n_small)):
        src = torch.arange(hi - 1, lo - 1, -1, dtype=torch.int32, device="cuda:0")
        dst = torch.arange(lo, hi, dtype=torch.int32, device="cuda:0")
        pool.promote(src, dst, bt, tags, torch.arange(lo, hi, dtype=torch.int64, device="cuda:0"))
        torch.cuda.synchronize()
        assert pool.status() == M.OK
        assert (bt.cpu().numpy()[0, lo:hi] == np.arange(lo, hi)).all() and (tags.cpu().numpy()[0, lo:hi] == M.TAG_ANCHOR).all()
