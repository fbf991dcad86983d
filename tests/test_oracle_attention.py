"""Pins for the oracle's dequantise-then-attend (Section 3.3, Eq. softmax-merge)."""
import math

import numpy as np
import pytest
import torch

import mkv_workloads as W
import oracle
from oracle.harness import build_layer
from _util import errs


def dense_attention(q, K, V, scale):
    """numpy fp64 softmax attention of one query over [n][d] keys/values."""
    s = (K @ q) * scale
    w = np.exp(s - s.max())
    return (w[:, None] * V).sum(0) / w.sum(), s.max() + math.log(w.sum())


def e4m3_to_f64(bytes_):
    return torch.from_numpy(np.ascontiguousarray(bytes_)).view(torch.float8_e4m3fn).to(torch.float64).numpy()


def hadamard(d):
    H = np.array([[1.0]])
    while H.shape[0] < d:
        H = np.block([[H, H], [H, -H]])
    return H


def small_spec(cfg, lens, **kw):
    return W.config(cfg, seq_lens=lens, **kw)


def test_all_fp8_assignment_equals_dense_attention_on_dequantised_fp8():
    spec = small_spec(1, (333, 64, 1, 200), recent_tokens=10 ** 9, anchor_spans=0)   # every page Recent/Anchor
    tab = W.tables(spec)
    assert not (tab.tier_tag == W.TAG_STALE).any()
    L = build_layer(spec, tab)
    out, lse = oracle.decode_attention(L.fp8_arena, L.tq3_arena, spec.head_dim, spec.n_kv_heads, spec.group,
                                       L.sigma, L.q_bits, tab.block_table, tab.tier_tag, tab.seq_lens, spec.scale)
    d, G = spec.head_dim, spec.group
    q = oracle.bf16_bits_to_f32(L.q_bits).astype(np.float64)
    for b in range(spec.batch):
        ln = spec.seq_lens[b]
        for h in range(spec.n_kv_heads):
            # dense dequantised tensors through torch's float8 type, gathered by the block table
            K = np.zeros((ln, d)); V = np.zeros((ln, d))
            for pg in range(spec.n_pages(b)):
                rec = L.fp8_arena[tab.block_table[b, pg], h]
                n = min(16, ln - 16 * pg)
                K[16 * pg:16 * pg + n] = e4m3_to_f64(rec[:16 * d]).reshape(16, d)[:n]
                V[16 * pg:16 * pg + n] = e4m3_to_f64(rec[16 * d:]).reshape(d, 16).T[:n]
            for g in range(G):
                ref, ref_lse = dense_attention(q[b, h * G + g], K, V, spec.scale)
                assert np.abs(out[b, h * G + g] - ref).max() < 1e-12
                assert abs(lse[b, h * G + g] - ref_lse) < 1e-12


def test_brute_force_softmax_on_tiny_inputs():
    for n in (1, 2, 5, 8):
        spec = small_spec(0, (n,), recent_tokens=10 ** 9, group=2)
        tab = W.tables(spec)
        L = build_layer(spec, tab)
        out, lse = oracle.decode_attention(L.fp8_arena, L.tq3_arena, spec.head_dim, 1, 2, L.sigma, L.q_bits,
                                           tab.block_table, tab.tier_tag, tab.seq_lens, spec.scale)
        d = spec.head_dim
        rec = L.fp8_arena[tab.block_table[0, 0], 0]
        for g in range(2):
            q = [float(x) for x in oracle.bf16_bits_to_f32(L.q_bits[0, g])]
            s = []
            for t in range(n):
                acc = 0.0
                for i in range(d):
                    acc += q[i] * oracle.e4m3_decode(int(rec[t * d + i]))
                s.append(acc * spec.scale)
            mx = max(s)
            w = [math.exp(x - mx) for x in s]
            for c in range(0, d, 9):
                ref = sum(w[t] * oracle.e4m3_decode(int(rec[16 * d + c * 16 + t])) for t in range(n)) / sum(w)
                assert abs(out[0, g, c] - ref) < 1e-13
            assert abs(lse[0, g] - (mx + math.log(sum(w)))) < 1e-13
            if n == 1:   # a single token: the output is that token's value
                v0 = np.array([oracle.e4m3_decode(int(rec[16 * d + c * 16])) for c in range(d)])
                assert np.array_equal(out[0, g], v0)


@pytest.fixture(params=[1, 2])
def record_format(request):
    with oracle.record_format(request.param):
        yield request.param


def test_tq3_pages_match_numpy_dense_attention_on_decoded_codes(record_format):
    """Stale pages: decode the packed codes with an explicit Hadamard matrix (k^ = g d^-1/2 sigma.(H c),
    v^ = scale*code + zero) and attend densely in numpy; in both record formats."""
    spec = small_spec(0, (16 * 9 + 5,), anchor_prefix=16, recent_tokens=40)
    tab = W.tables(spec)
    assert (tab.tier_tag[0, :spec.n_pages(0)] == W.TAG_STALE).sum() >= 5
    L = build_layer(spec, tab)
    d, G = spec.head_dim, spec.group
    out, lse = oracle.decode_attention(L.fp8_arena, L.tq3_arena, d, 1, G, L.sigma, L.q_bits, tab.block_table,
                                       tab.tier_tag, tab.seq_lens, spec.scale)
    C, _ = oracle.codebook()
    H = hadamard(d)
    ln = spec.seq_lens[0]
    K = np.zeros((ln, d)); V = np.zeros((ln, d))
    f16 = lambda bits: np.asarray(bits, np.uint16).view(np.float16).astype(np.float64)
    for pg in range(spec.n_pages(0)):
        n = min(16, ln - 16 * pg)
        pid = tab.block_table[0, pg]
        if tab.tier_tag[0, pg] == W.TAG_STALE:
            kc, g, vc, sc, zp = oracle.tq3_unpack_record(L.tq3_arena[pid, 0], d)
            c = np.where(kc >> 2 == 1, -1.0, 1.0) * C[kc & 3].astype(np.float64)
            K[16 * pg:16 * pg + 16] = f16(g)[:, None] * L.sigma[None, :] * (c @ H) / math.sqrt(d)
            V[16 * pg:16 * pg + 16] = vc * f16(sc)[None, :] + f16(zp)[None, :]
        else:
            rec = L.fp8_arena[pid, 0]
            K[16 * pg:16 * pg + n] = e4m3_to_f64(rec[:16 * d]).reshape(16, d)[:n]
            V[16 * pg:16 * pg + n] = e4m3_to_f64(rec[16 * d:]).reshape(d, 16).T[:n]
    q = oracle.bf16_bits_to_f32(L.q_bits).astype(np.float64)
    for g in range(G):
        ref, ref_lse = dense_attention(q[0, g], K, V, spec.scale)
        assert np.abs(out[0, g] - ref).max() < 1e-11
        assert abs(lse[0, g] - ref_lse) < 1e-11
    # and the quantised cache is a faithful version of the bf16 originals (codec error only)
    k_bits, v_bits = W.kv(spec, 0, 0)
    K0 = oracle.bf16_bits_to_f32(k_bits)[:, 0].astype(np.float64)
    assert 0.10 < np.linalg.norm(K - K0) / np.linalg.norm(K0) < 0.25


def test_softmax_merge_is_invariant_to_the_partition():
    """Eq. (softmax-merge): merging per-partition (m_j, l_j, O_j) equals attention over the
    concatenated cache -- by format, and by any number of contiguous ranges."""
    spec = small_spec(1, (700, 16 * 30, 90), anchor_span_tokens=64, recent_tokens=100)
    tab = W.tables(spec)
    L = build_layer(spec, tab)
    args = (L.fp8_arena, L.tq3_arena, spec.head_dim, spec.n_kv_heads, spec.group, L.sigma, L.q_bits,
            tab.block_table, tab.tier_tag, tab.seq_lens, spec.scale)
    ref, ref_lse = oracle.decode_attention(*args, mode=0)
    for mode in (1, 2, 3, 7, 50):
        got, got_lse = oracle.decode_attention(*args, mode=mode)
        assert np.abs(got - ref).max() < 1e-12 and np.abs(got_lse - ref_lse).max() < 1e-12, mode


def test_page_table_indexing_gqa_mapping_and_length_mask():
    """K = 0 gives uniform weights, so the output is the mean of the values read; values are chosen
    per (kv head, logical page) so that any wrong page id, arena, head or slot shows up."""
    d, hkv, G = 128, 2, 3
    lens = (16 * 6 + 3, 16 * 4)
    spec = small_spec(0, lens, n_kv_heads=hkv, group=G, anchor_prefix=16, recent_tokens=20)
    tab = W.tables(spec, extra_fp8=3, extra_tq3=3)
    rng = np.random.default_rng(0)
    fp8 = rng.integers(0, 0x78, (tab.fp8_pages, hkv, 32 * d)).astype(np.uint8)    # garbage everywhere
    tq3 = rng.integers(0, 256, (tab.tq3_pages, hkv, 16 * d + 32)).astype(np.uint8)
    sigma = W.rotation_signs(spec)
    expect = np.zeros((len(lens), hkv, d))
    for b, ln in enumerate(lens):
        for pg in range(spec.n_pages(b)):
            n = min(16, ln - 16 * pg)
            for h in range(hkv):
                val = np.zeros((16, d), np.float32)
                val[:, :] = (8 + pg % 8) * 2.0 ** (h - 3 + 2 * b)     # four significant bits: fp16- and e4m3-exact
                val[:, pg] = 0.0                                       # a page-specific channel
                k = np.zeros((16, d), np.float32)
                pid = tab.block_table[b, pg]
                if tab.tier_tag[b, pg] == W.TAG_STALE:
                    tq3[pid, h] = oracle.tq3_record_from_f32(k, val, sigma)
                else:
                    rec = oracle.fp8_pack_record(k, val, 16)
                    if n < 16:   # slots beyond the sequence length hold garbage that must be masked
                        rec = rec.copy()
                        kk = rec[:16 * d].reshape(16, d); kk[n:] = 0x77
                        vv = rec[16 * d:].reshape(d, 16); vv[:, n:] = 0x7E
                    fp8[pid, h] = rec
                expect[b, h] += n * val[0].astype(np.float64)
        expect[b] /= ln
    q = W.query(spec)
    out, lse = oracle.decode_attention(fp8, tq3, d, hkv, G, sigma, q, tab.block_table, tab.tier_tag,
                                       tab.seq_lens, spec.scale)
    for b in range(len(lens)):
        for hq in range(hkv * G):
            assert np.abs(out[b, hq] - expect[b, hq // G]).max() < 1e-12     # head hq reads KV head hq // G
            assert abs(lse[b, hq] - math.log(lens[b])) < 1e-12


def test_empty_request_and_invalid_entries():
    spec = small_spec(0, (0, 40), recent_tokens=10 ** 9)
    tab = W.tables(spec)
    L = build_layer(spec, tab)
    out, lse = oracle.decode_attention(L.fp8_arena, L.tq3_arena, spec.head_dim, 1, spec.group, L.sigma, L.q_bits,
                                       tab.block_table, tab.tier_tag, tab.seq_lens, spec.scale)
    assert not out[0].any() and np.all(np.isneginf(lse[0])) and out[1].any()
    bad = tab.block_table.copy()
    bad[1, 0] = 10 ** 6
    with pytest.raises(ValueError):
        oracle.decode_attention(L.fp8_arena, L.tq3_arena, spec.head_dim, 1, spec.group, L.sigma, L.q_bits,
                                bad, tab.tier_tag, tab.seq_lens, spec.scale)


def test_workload_generator_shapes_match_the_configurations():
    expect_bytes = {0: 572800, 1: 74866688, 2: 126474240}
    for i, nbytes in expect_bytes.items():
        s = W.config(i)
        t = W.tables(s)
        assert W.kv_bytes(s, t) == nbytes
    s = W.config(2)
    t = W.tables(s)
    tags = t.tier_tag[0]
    assert (tags == W.TAG_ANCHOR).sum() == 16 and (tags == W.TAG_RECENT).sum() == 128 and (tags == W.TAG_STALE).sum() == 3544
    s3 = W.config(3)
    assert s3.batch == 64 and min(s3.seq_lens) >= 1024 and max(s3.seq_lens) < 131072
    t3 = W.tables(s3)
    for b in range(64):
        n = s3.n_pages(b)
        ids = t3.block_table[b, :n]
        assert (ids >= 0).all() and (t3.block_table[b, n:] == -1).all()
        if s3.seq_lens[b] % 16:
            assert t3.tier_tag[b, n - 1] != W.TAG_STALE
    # ids are unique inside each arena
    st = t3.tier_tag == W.TAG_STALE
    used = t3.block_table >= 0
    assert len(np.unique(t3.block_table[used & st])) == (used & st).sum()
    assert len(np.unique(t3.block_table[used & ~st])) == (used & ~st).sum()
    k, v = W.kv(W.config(0), 0, 0)
    assert k.shape == (4096, 1, 128) and k.dtype == np.uint16
    kf = W.bf16_bits_to_f32(k)
    ch = W.outlier_channels(W.config(0), 0, 0)
    assert len(ch) == 4 and 6 < kf[:, 0, ch].std() < 10 and 0.9 < np.delete(kf[:, 0], ch, axis=1).std() < 1.1
