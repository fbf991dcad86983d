"""Pins for the oracle's globally normalised page mass (Section 3.1, Eq. score-partial,
Eq. score-global-weight, Eq. attention-score)."""
import numpy as np
import torch

import mkv_workloads as W
import oracle
from oracle.harness import build_layer


def e4m3_to_f64(bytes_):
    return torch.from_numpy(np.ascontiguousarray(bytes_)).view(torch.float8_e4m3fn).to(torch.float64).numpy()


def keys_of_row(spec, tab, L, b, h):
    """Dequantised keys [len][d] of one (request, KV head): FP8 pages through torch's float8 type, Stale
    pages through the record unpacker and the key decoder (both pinned in their own tests)."""
    d, ln = spec.head_dim, spec.seq_lens[b]
    K = np.zeros((ln, d))
    for pg in range(spec.n_pages(b)):
        n = min(16, ln - 16 * pg)
        if tab.tier_tag[b, pg] == W.TAG_STALE:
            kcode, g, _, _, _ = oracle.tq3_unpack_record(L.tq3_arena[tab.block_table[b, pg], h], d)
            for t in range(n):
                K[16 * pg + t] = oracle.tq3_decode_key(kcode[t], int(g[t]), L.sigma)
        else:
            rec = L.fp8_arena[tab.block_table[b, pg], h]
            K[16 * pg:16 * pg + n] = e4m3_to_f64(rec[:16 * d]).reshape(16, d)[:n]
    return K


def plain_page_mass(q, K, scale, n_pages):
    """Textbook definition: softmax over all tokens, summed per 16-token page."""
    s = (K @ q) * scale
    w = np.exp(s - s.max())
    w /= w.sum()
    out = np.zeros(n_pages)
    for pg in range(n_pages):
        out[pg] = w[16 * pg:16 * pg + 16].sum()
    return out


def run_mass(spec, tab, L):
    return oracle.page_mass(L.fp8_arena, L.tq3_arena, spec.head_dim, spec.n_kv_heads, spec.group, L.sigma, L.q_bits,
                            tab.block_table, tab.tier_tag, tab.seq_lens, spec.scale)


def test_two_level_formula_equals_the_plain_softmax_mass_all_fp8_and_mixed():
    for spec in (W.config(1, seq_lens=(333, 64, 1, 200), recent_tokens=10 ** 9, anchor_spans=0),     # all FP8
                 W.config(1, seq_lens=(613, 400, 96, 1024), recent_tokens=80, anchor_span_tokens=32),   # mixed
                 W.config(4, batch=2, ctx=512, stale_fraction=0.95)):
        tab = W.tables(spec)
        L = build_layer(spec, tab)
        mass = run_mass(spec, tab, L)
        q = oracle.bf16_bits_to_f32(L.q_bits).astype(np.float64)
        G = spec.group
        for b in range(spec.batch):
            npg = spec.n_pages(b)
            for h in range(spec.n_kv_heads):
                K = keys_of_row(spec, tab, L, b, h)
                for g in range(G):
                    ref = plain_page_mass(q[b, h * G + g], K, spec.scale, npg)
                    got = mass[b, h * G + g]
                    assert np.abs(got[:npg] - ref).max() < 1e-12, (spec.name, b, h, g)
                    assert abs(got[:npg].sum() - 1.0) < 1e-12
                    assert not got[npg:].any()                      # pages beyond the length carry no mass


def test_mass_follows_a_planted_key():
    """A key equal to a large multiple of the query direction takes almost all of the mass of its page."""
    spec = W.config(0, seq_lens=(640,), recent_tokens=10 ** 9)                 # all FP8: keys are e4m3 of what we plant
    tab = W.tables(spec)
    d = spec.head_dim
    rng = np.random.default_rng(5)
    k = rng.standard_normal((640, spec.n_kv_heads, d)).astype(np.float32) * 0.25      # [len][hkv][d]
    v = rng.standard_normal((640, spec.n_kv_heads, d)).astype(np.float32)
    qv = np.zeros((1, spec.n_q_heads, d), np.float32)
    qv[..., :8] = 2.0
    k[16 * 23 + 5, 0, :8] = 8.0                                            # score 8*2*8/sqrt(128) = 11.3 above the rest
    fp8 = np.zeros((tab.fp8_pages, spec.n_kv_heads, 32 * d), np.uint8)
    tq3 = np.zeros((max(tab.tq3_pages, 1), spec.n_kv_heads, 16 * d + 32), np.uint8)
    sigma = W.rotation_signs(spec, 0)
    oracle.encode_request(W.f32_to_bf16_bits(k), W.f32_to_bf16_bits(v), tab.block_table[0, :40], tab.tier_tag[0, :40], sigma, fp8, tq3)
    mass = oracle.page_mass(fp8, tq3, d, spec.n_kv_heads, spec.group, sigma, W.f32_to_bf16_bits(qv), tab.block_table,
                            tab.tier_tag, tab.seq_lens, spec.scale)
    assert mass[0, :, 23].min() > 0.95
    assert (np.argmax(mass[0], axis=1) == 23).all()


def test_score_update_is_the_head_mean_and_an_ewma():
    rng = np.random.default_rng(11)
    B, Hq, P = 2, 6, 9
    mass = rng.random((B, Hq, P))
    lens = np.array([9 * 16 - 3, 4 * 16], np.int32)                           # 9 and 4 pages
    prev = rng.random((B, P))
    mask = 0b101001                                                            # heads 0, 3, 5
    got = oracle.page_score_update(mass, lens, mask, 0.75, prev)
    r = (mass[:, 0] + mass[:, 3] + mass[:, 5]) / 3.0
    ref = prev.copy()
    ref[0, :9] = 0.75 * prev[0, :9] + 0.25 * r[0, :9]
    ref[1, :4] = 0.75 * prev[1, :4] + 0.25 * r[1, :4]
    assert np.abs(got - ref).max() < 1e-15
    assert np.array_equal(got[1, 4:], prev[1, 4:])                             # beyond the length: untouched
    assert np.abs(oracle.page_score_update(mass, lens, (1 << Hq) - 1, 0.0, prev)[0] - mass[0].mean(0)).max() < 1e-15
    assert np.array_equal(oracle.page_score_update(mass, lens, 1, 1.0, prev), prev)
