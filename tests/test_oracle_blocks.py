"""Pins of the oracle for pages of 16 M tokens (the paper's blocks of 1,792 / 832 tokens): sizes against
the byte counters the paper prints, the M = 1 case against the 16-token records, the shared value
scale/zero against its invariants, and the attention over such pages against an independent dense
evaluation of the unpacked values."""
import numpy as np
import pytest

import mkv_workloads as W
import oracle
from oracle.harness import build_layer


def test_block_sizes_reproduce_the_papers_byte_counters():
    # Section 5.4 (measured canary, one layer, both requests): 18 FP8 + 47 TQ3 blocks of 1,792 tokens,
    # 4 KV heads, d = 256 occupy 131,610,624 bytes; the same 65 blocks in BF16 477,102,080 bytes; 3.6251x.
    d, M, hkv = 256, 1792 // 16, 4
    mixed = hkv * (18 * oracle.fp8_block_bytes(d, M) + 47 * oracle.tq3_block_bytes(d, M))
    dense = 65 * oracle.page_bytes_dense(1792, d, hkv, 2)
    assert mixed == 131_610_624
    assert dense == 477_102_080
    assert round(dense / mixed, 4) == 3.6251
    # the closed form of the physical TQ3 rate (Eq. effective-bits, b_S): 3 + 8/d + 1/M bits per scalar
    assert oracle.tq3_block_bytes(d, M) * 8 / (2 * 1792 * d) == pytest.approx(3 + 8 / d + 1 / M, abs=1e-12)
    assert oracle.tq3_block_bytes(d, M) == oracle.page_bytes_tq3(1792, d, 1)
    assert oracle.tq3_block_bytes(128, 52) == oracle.page_bytes_tq3(832, 128, 1)


@pytest.mark.parametrize("d", [128, 256])
def test_one_tile_blocks_are_the_16_token_records(d):
    rng = np.random.default_rng(d)
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    k = rng.standard_normal((16, d)).astype(np.float32)
    v = rng.standard_normal((16, d)).astype(np.float32)
    assert oracle.tq3_block_bytes(d, 1) == oracle.tq3_record_bytes(d) and oracle.fp8_block_bytes(d, 1) == oracle.fp8_record_bytes(d)
    rec = oracle.tq3_record_from_f32(k, v, sigma)
    assert np.array_equal(oracle.tq3_block_from_f32(k, v, sigma), rec)
    f8 = oracle.fp8_pack_record(k, v)
    assert np.array_equal(oracle.fp8_pack_block(k, v), f8)
    assert np.array_equal(oracle.demote_block(f8, d, 1, sigma), oracle.demote_record(f8, d, sigma))
    assert np.array_equal(oracle.promote_block(rec, d, 1, sigma), oracle.promote_record(rec, d, sigma))


def test_value_scale_and_zero_are_shared_by_all_tokens_of_the_page():
    rng = np.random.default_rng(3)
    d, M = 128, 7
    v = rng.standard_normal((16 * M, d)).astype(np.float32)
    v[:, 5] *= 8
    v[:, 9] = 0.25                                         # constant channel
    code, sc, zp = oracle.tq3_encode_value_block(v)
    scf = np.array([oracle.f16_to_f32(int(x)) for x in sc], np.float64)
    zpf = np.array([oracle.f16_to_f32(int(x)) for x in zp], np.float64)
    # invariants: the channel minimum takes code 0 and the maximum code 7, over the WHOLE page
    for c in (0, 5, 17, 100):
        assert code[np.argmin(v[:, c]), c] == 0 and code[np.argmax(v[:, c]), c] == 7
        assert code[:, c].min() == 0 and code[:, c].max() == 7
    assert sc[9] == 0 and (code[:, 9] == 0).all() and zpf[9] == 0.25
    # reconstruction error: half a step plus the fp16 rounding of scale (7 steps) and zero
    err = np.abs(scf[None, :] * code + zpf[None, :] - v)
    bound = scf / 2 + 7 * scf * 2.0 ** -11 + np.abs(zpf) * 2.0 ** -11 + 1e-7
    assert (err <= bound[None, :]).all()
    # a tile taken alone would choose a different (finer) scale: the sharing is real
    _, sc_tile, _ = oracle.tq3_encode_value_page(v[:16])
    assert (sc_tile[:8] != sc[:8]).any()


def test_tiles_hold_per_token_key_codes_and_the_pages_value_metadata():
    rng = np.random.default_rng(4)
    d, M = 128, 5
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    k = rng.standard_normal((16 * M, d)).astype(np.float32)
    v = rng.standard_normal((16 * M, d)).astype(np.float32)
    blk = oracle.tq3_block_from_f32(k, v, sigma)
    tile = 12 * d + 32
    assert blk.size == M * tile + 4 * d
    kc, g, vc, sc, zp = oracle.tq3_unpack_block(blk, d, M)
    code, sc2, zp2 = oracle.tq3_encode_value_block(v)
    assert np.array_equal(vc, code) and np.array_equal(sc, sc2) and np.array_equal(zp, zp2)
    for m in range(M):
        # keys are coded per token: the key bytes and g of tile m equal those of the 16-token record of its tokens
        rec = oracle.tq3_record_from_f32(k[16 * m:16 * m + 16], v[16 * m:16 * m + 16], sigma)
        assert np.array_equal(blk[m * tile:m * tile + 6 * d], rec[:6 * d])
        assert np.array_equal(blk[m * tile + 12 * d:(m + 1) * tile], rec[12 * d:12 * d + 32])
        for t in range(16):
            c1, g1 = oracle.tq3_encode_key(k[16 * m + t], sigma)
            assert np.array_equal(kc[16 * m + t], c1) and g[16 * m + t] == g1
    # round trip of the packer
    assert np.array_equal(oracle.tq3_pack_block(kc, g, vc, sc, zp), blk)
    # demote = dequantise the FP8 page exactly, then encode; promote rebuilds tile by tile with the page's metadata
    f8 = oracle.fp8_pack_block(k, v)
    kq, vq = oracle.fp8_unpack_block_f32(f8, d, M)
    assert np.array_equal(oracle.demote_block(f8, d, M, sigma), oracle.tq3_block_from_f32(kq, vq, sigma))
    back = oracle.promote_block(blk, d, M, sigma)
    kb, vb = oracle.fp8_unpack_block_f32(back, d, M)
    scf = np.array([oracle.f16_to_f32(int(x)) for x in sc], np.float32)
    zpf = np.array([oracle.f16_to_f32(int(x)) for x in zp], np.float32)
    want_v = (scf[None, :] * vc.astype(np.float32) + zpf[None, :]).astype(np.float32)
    assert np.abs(vb - want_v).max() <= np.abs(want_v).max() * 2.0 ** -4      # e4m3 rounding of the rebuilt values


def _dense_reference(spec, tab, L, b, hq):
    """Independent evaluation: unpack every page with the block readers, softmax in numpy fp64."""
    d, hkv, M = spec.head_dim, spec.n_kv_heads, spec.tiles_per_page
    h = hq // spec.group
    ln = spec.seq_lens[b]
    K = np.zeros((spec.n_pages(b) * spec.page_tokens, d))
    V = np.zeros_like(K)
    for pg in range(spec.n_pages(b)):
        pid, tag = tab.block_table[b, pg], tab.tier_tag[b, pg]
        lo = pg * spec.page_tokens
        if tag == W.TAG_STALE:
            kc, g, vc, sc, zp = oracle.tq3_unpack_block(L.tq3_arena[pid, h], d, M)
            for t in range(spec.page_tokens):
                K[lo + t] = oracle.tq3_decode_key(kc[t], int(g[t]), L.sigma)
            scf = np.array([oracle.f16_to_f32(int(x)) for x in sc], np.float64)
            zpf = np.array([oracle.f16_to_f32(int(x)) for x in zp], np.float64)
            V[lo:lo + spec.page_tokens] = scf[None, :] * vc + zpf[None, :]
        else:
            kk, vv = oracle.fp8_unpack_block_f32(L.fp8_arena[pid, h], d, M)
            K[lo:lo + spec.page_tokens], V[lo:lo + spec.page_tokens] = kk, vv
    q = oracle.bf16_bits_to_f32(L.q_bits[b, hq]).astype(np.float64)
    s = (K[:ln] @ q) * spec.scale
    w = np.exp(s - s.max())
    return (w[:, None] * V[:ln]).sum(0) / w.sum(), s.max() + np.log(w.sum())


@pytest.mark.parametrize("page_tokens", [48, 832])
def test_attention_over_blocks_equals_dense_attention_on_the_unpacked_values(page_tokens):
    spec = W.config(0, seq_lens=(5 * page_tokens + 3 * 16 + 5, 2 * page_tokens), head_dim=128, n_kv_heads=2, group=2,
                    anchor_prefix=page_tokens, anchor_spans=0, recent_tokens=page_tokens, page_tokens=page_tokens, seed=11)
    tab = W.tables(spec)
    assert (tab.tier_tag[0, :spec.n_pages(0)] == W.TAG_STALE).sum() >= 2
    L = build_layer(spec, tab)
    out, lse = oracle.decode_attention(L.fp8_arena, L.tq3_arena, spec.head_dim, spec.n_kv_heads, spec.group, L.sigma,
                                       L.q_bits, tab.block_table, tab.tier_tag, tab.seq_lens, spec.scale,
                                       page_tokens=page_tokens)
    for b, hq in ((0, 0), (0, 3), (1, 2)):
        ref, ref_lse = _dense_reference(spec, tab, L, b, hq)
        assert np.abs(out[b, hq] - ref).max() < 1e-12
        assert abs(lse[b, hq] - ref_lse) < 1e-12
    # Eq. (softmax-merge) over the two format partitions and over contiguous ranges gives the same result
    for mode in (1, 5):
        o2, l2 = oracle.decode_attention(L.fp8_arena, L.tq3_arena, spec.head_dim, spec.n_kv_heads, spec.group, L.sigma,
                                         L.q_bits, tab.block_table, tab.tier_tag, tab.seq_lens, spec.scale, mode=mode,
                                         page_tokens=page_tokens)
        assert np.abs(o2 - out).max() < 1e-12 and np.abs(l2 - lse).max() < 1e-12


def test_all_fp8_blocks_and_16_token_pages_hold_the_same_cache():
    """With every page FP8 the page size changes only where a token's bytes sit: the attention must not move."""
    base = dict(seq_lens=(333,), head_dim=128, n_kv_heads=1, group=4, anchor_prefix=0, anchor_spans=0, recent_tokens=10 ** 6, seed=5)
    outs = []
    for pt in (16, 64, 208):
        spec = W.config(0, page_tokens=pt, **base)
        tab = W.tables(spec)
        assert (tab.tier_tag[0, :spec.n_pages(0)] != W.TAG_STALE).all()
        L = build_layer(spec, tab)
        outs.append(oracle.decode_attention(L.fp8_arena, L.tq3_arena, 128, 1, 4, L.sigma, L.q_bits, tab.block_table,
                                            tab.tier_tag, tab.seq_lens, spec.scale, page_tokens=pt)[0])
    assert np.abs(outs[0] - outs[1]).max() < 1e-13 and np.abs(outs[0] - outs[2]).max() < 1e-13


def test_page_mass_of_blocks_is_the_softmax_probability_summed_over_the_page():
    """Eq. (score-partial) / (score-global-weight) with the two format partitions collapse to: the mass of a page is the
    sum of the global softmax probabilities of its tokens.  Checked against an independent evaluation, and, for an
    all-FP8 cache, against the 16-token page masses of the same cache added up per block."""
    pt = 80
    spec = W.config(0, seq_lens=(6 * pt + 33, 3 * pt), head_dim=128, n_kv_heads=2, group=2, anchor_prefix=pt, anchor_spans=0,
                    recent_tokens=pt + 1, page_tokens=pt, seed=13)
    tab = W.tables(spec)
    L = build_layer(spec, tab)
    mass = oracle.page_mass(L.fp8_arena, L.tq3_arena, 128, 2, 2, L.sigma, L.q_bits, tab.block_table, tab.tier_tag, tab.seq_lens,
                            spec.scale, page_tokens=pt)
    assert mass.shape == (2, 4, tab.block_table.shape[1])
    assert np.abs(mass.sum(-1) - 1).max() < 1e-12
    for b, hq in ((0, 1), (1, 3)):
        d, M = 128, pt // 16
        h, ln = hq // spec.group, spec.seq_lens[b]
        K = np.zeros((spec.n_pages(b) * pt, d))
        for pg in range(spec.n_pages(b)):
            pid = tab.block_table[b, pg]
            if tab.tier_tag[b, pg] == W.TAG_STALE:
                kc, g, _, _, _ = oracle.tq3_unpack_block(L.tq3_arena[pid, h], d, M)
                for t in range(pt):
                    K[pg * pt + t] = oracle.tq3_decode_key(kc[t], int(g[t]), L.sigma)
            else:
                K[pg * pt:(pg + 1) * pt] = oracle.fp8_unpack_block_f32(L.fp8_arena[pid, h], d, M)[0]
        q = oracle.bf16_bits_to_f32(L.q_bits[b, hq]).astype(np.float64)
        s = (K[:ln] @ q) * spec.scale
        p = np.exp(s - s.max())
        p /= p.sum()
        want = np.array([p[pg * pt:(pg + 1) * pt].sum() for pg in range(spec.n_pages(b))])
        assert np.abs(mass[b, hq, :spec.n_pages(b)] - want).max() < 1e-13
        assert not mass[b, hq, spec.n_pages(b):].any()
    # Eq. (attention-score) over blocks: pages are counted in units of the page size
    prev = np.full((2, mass.shape[2]), 0.25)
    got = oracle.page_score_update(mass, tab.seq_lens, 0b0101, 0.5, prev, page_tokens=pt)
    n0 = spec.n_pages(0)
    assert np.abs(got[0, :n0] - (0.125 + 0.5 * (mass[0, 0, :n0] + mass[0, 2, :n0]) / 2)).max() < 1e-15
    assert np.array_equal(got[0, n0:], prev[0, n0:])
    # all-FP8: the same cache in 16-token pages; block masses are sums of page masses
    base = dict(seq_lens=(5 * pt + 7,), head_dim=128, n_kv_heads=1, group=4, anchor_prefix=0, anchor_spans=0, recent_tokens=10 ** 6, seed=5)
    sb, s16 = W.config(0, page_tokens=pt, **base), W.config(0, **base)
    tb, t16 = W.tables(sb), W.tables(s16)
    Lb, L16 = build_layer(sb, tb), build_layer(s16, t16)
    mb = oracle.page_mass(Lb.fp8_arena, Lb.tq3_arena, 128, 1, 4, Lb.sigma, Lb.q_bits, tb.block_table, tb.tier_tag, tb.seq_lens,
                          sb.scale, page_tokens=pt)
    m16 = oracle.page_mass(L16.fp8_arena, L16.tq3_arena, 128, 1, 4, L16.sigma, L16.q_bits, t16.block_table, t16.tier_tag,
                           t16.seq_lens, s16.scale)
    for pg in range(sb.n_pages(0)):
        assert np.abs(mb[0, :, pg] - m16[0, :, pg * 5:(pg + 1) * 5].sum(-1)).max() < 1e-13
