"""Parity of mkv_decode_attention (through the C ABI) with the fp64 oracle on identical quantised
pages: scaled-down versions of the five configurations, edge cases, and both kernels."""
import numpy as np
import pytest
import torch

import mkv_workloads as W
import oracle
import paper_2608_23834_b200 as M
from _gpu_util import Case, check_case, check_close

pytestmark = pytest.mark.gpu

VARIANTS = [pytest.param(M.DECODE_TENSOR, id="tensor"), pytest.param(M.DECODE_SCALAR, id="scalar"),
            pytest.param(M.DECODE_TMEM, id="tmem")]     # tmem: tcgen05 kernel at d = 256, the tensor kernel at d = 128

SCALED = {
    "cfg0": lambda: W.config(0),                                                        # 4,096 tokens as specified
    "cfg1": lambda: W.config(1, seq_lens=(2048 + 16 * i for i in range(8)), recent_tokens=256, anchor_span_tokens=64),
    "cfg2": lambda: W.config(2, seq_lens=(5008, 4432), recent_tokens=512, n_layers=1),
    "cfg3": lambda: W.config(3, seq_lens=[int(1024 * 8 ** u) for u in np.random.default_rng(3).random(12)], recent_tokens=200),
    "cfg4_f0": lambda: W.config(4, batch=3, ctx=1024, stale_fraction=0.0),
    "cfg4_f50": lambda: W.config(4, batch=3, ctx=1024, stale_fraction=0.5),
    "cfg4_f95": lambda: W.config(4, batch=3, ctx=1024, stale_fraction=0.95),
}


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("name", list(SCALED))
def test_decode_matches_oracle_on_scaled_configs(name, variant):
    case = Case(SCALED[name](), extra_fp8=5, extra_tq3=7)
    out, lse = case.run(variant)
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("d,hkv,group", [(128, 2, 4), (256, 1, 6), (128, 1, 1), (256, 2, 8), (128, 3, 5)])
def test_decode_edge_lengths(d, hkv, group, variant):
    """Empty, single-token, one-short-of-a-page, exactly-a-page, one-over, and ragged lengths in one batch."""
    lens = (0, 1, 15, 16, 17, 33, 16 * 20, 16 * 20 + 9, 300)
    spec = W.config(0, seq_lens=lens, head_dim=d, n_kv_heads=hkv, group=group, anchor_prefix=16, recent_tokens=40,
                    n_outlier=3)
    case = Case(spec, extra_fp8=2, extra_tq3=2)
    out, lse = case.run(variant)
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)
    # without an lse buffer the output is unchanged
    out2, _ = case.run(variant, want_lse=False)
    assert np.array_equal(out, out2)


@pytest.mark.parametrize("variant", VARIANTS)
def test_decode_all_fp8_and_all_stale_tiers(variant):
    for kw in (dict(recent_tokens=10 ** 9), dict(anchor_prefix=0, recent_tokens=0)):
        spec = W.config(1, seq_lens=(640, 1600, 16), **kw, anchor_spans=0)
        case = Case(spec)
        out, lse = case.run(variant)
        ref, ref_lse = case.reference()
        check_case(case, out, lse, ref, ref_lse)


@pytest.mark.parametrize("variant", VARIANTS)
def test_decode_with_fp8_scales(variant):
    spec = W.config(0, seq_lens=(700,), recent_tokens=300)
    case = Case.__new__(Case)
    # pages encoded with non-unit power-of-two FP8 scales
    tab = W.tables(spec)
    import oracle.harness as H
    d, hkv = spec.head_dim, spec.n_kv_heads
    fp8 = np.zeros((tab.fp8_pages, hkv, 32 * d), np.uint8)
    tq3 = np.zeros((tab.tq3_pages, hkv, 16 * d + 32), np.uint8)
    sigma = W.rotation_signs(spec)
    kb, vb = W.kv(spec, 0, 0)
    oracle.encode_request(kb, vb, tab.block_table[0, :spec.n_pages(0)], tab.tier_tag[0, :spec.n_pages(0)], sigma, fp8, tq3, 0.5, 4.0)
    pool = M.Pool(d, hkv, spec.n_q_heads, tab.fp8_pages, tab.tq3_pages, sigma, 0.5, 4.0, max_batch=1)
    pool.upload_arenas(fp8, tq3)
    pool.set_decode_variant(variant)
    from _gpu_util import bf16_tensor
    q_bits = W.query(spec)
    out = pool.decode_attention(bf16_tensor(q_bits), torch.from_numpy(tab.block_table).cuda(), torch.from_numpy(tab.tier_tag).cuda(),
                                torch.from_numpy(tab.seq_lens).cuda(), spec.scale).cpu().numpy()
    ref, _ = oracle.decode_attention(fp8, tq3, d, hkv, spec.group, sigma, q_bits, tab.block_table, tab.tier_tag, tab.seq_lens,
                                     spec.scale, 0.5, 4.0)
    check_close(out, ref, "fp8 scales")


@pytest.mark.parametrize("variant", VARIANTS)
def test_decode_reads_exactly_the_pages_the_table_names(variant):
    """K = 0 gives uniform weights, so the output is the mean of the values read: any wrong page id,
    arena, KV head or slot, or a read beyond seq_len, changes it."""
    d, hkv, G = 128, 2, 3
    lens = (16 * 6 + 3, 16 * 4)
    spec = W.config(0, seq_lens=lens, n_kv_heads=hkv, group=G, anchor_prefix=16, recent_tokens=20)
    tab = W.tables(spec, extra_fp8=3, extra_tq3=3)
    rng = np.random.default_rng(0)
    fp8 = rng.integers(0, 0x78, (tab.fp8_pages, hkv, 32 * d)).astype(np.uint8)       # finite garbage everywhere
    tq3 = np.zeros((tab.tq3_pages, hkv, 16 * d + 32), np.uint8)
    sigma = W.rotation_signs(spec)
    for b, ln in enumerate(lens):
        for pg in range(spec.n_pages(b)):
            n = min(16, ln - 16 * pg)
            for h in range(hkv):
                val = np.full((16, d), (8 + pg % 8) * 2.0 ** (h - 3 + 2 * b), np.float32)
                val[:, pg] = 0.0
                k = np.zeros((16, d), np.float32)
                pid = tab.block_table[b, pg]
                if tab.tier_tag[b, pg] == W.TAG_STALE:
                    tq3[pid, h] = oracle.tq3_record_from_f32(k, val, sigma)
                else:
                    rec = oracle.fp8_pack_record(k, val, 16).copy()
                    if n < 16:
                        rec[:16 * d].reshape(16, d)[n:] = 0x77
                        rec[16 * d:].reshape(d, 16)[:, n:] = 0x7E
                    fp8[pid, h] = rec
    pool = M.Pool(d, hkv, hkv * G, tab.fp8_pages, tab.tq3_pages, sigma, max_batch=2)
    pool.upload_arenas(fp8, tq3)
    pool.set_decode_variant(variant)
    from _gpu_util import bf16_tensor
    q_bits = W.query(spec)
    lse = torch.zeros((2, hkv * G), dtype=torch.float32, device="cuda:0")
    out = pool.decode_attention(bf16_tensor(q_bits), torch.from_numpy(tab.block_table).cuda(), torch.from_numpy(tab.tier_tag).cuda(),
                                torch.from_numpy(tab.seq_lens).cuda(), spec.scale, lse=lse).cpu().numpy()
    ref, ref_lse = oracle.decode_attention(fp8, tq3, d, hkv, G, sigma, q_bits, tab.block_table, tab.tier_tag, tab.seq_lens, spec.scale)
    assert np.abs(out - ref).max() < 1e-4 * np.abs(ref).max()
    assert np.abs(lse.cpu().numpy() - ref_lse).max() < 1e-4


@pytest.mark.parametrize("variant", VARIANTS)
def test_decode_flags_bad_table_entries_without_faulting(variant):
    spec = W.config(0, seq_lens=(200,), recent_tokens=60)
    case = Case(spec)
    case.pool.set_decode_variant(variant)
    bad = case.bt.clone()
    bad[0, 3] = 10 ** 6
    case.pool.decode_attention(case.q, bad, case.tags, case.lens, spec.scale)
    torch.cuda.synchronize()
    assert case.pool.status() == M.E_BOUNDS
    bad_tag = case.tags.clone()
    bad_tag[0, 2] = 7
    case.pool.decode_attention(case.q, case.bt, bad_tag, case.lens, spec.scale)
    torch.cuda.synchronize()
    assert case.pool.status() == M.E_BOUNDS
    out, lse = case.run(variant)                  # the pool and workspace are still usable
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)


def test_host_side_argument_checks():
    spec = W.config(0, seq_lens=(64,))
    case = Case(spec)
    L = M.lib()
    import ctypes as C
    small = torch.empty(256, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(M.MkvError) as e:
        case.pool.decode_attention(case.q, case.bt, case.tags, case.lens, spec.scale, workspace=small)
    assert e.value.code == M.E_INVALID
    with pytest.raises(M.MkvError):
        M.Pool(96, 1, 1, 1, 1, np.ones(96, np.int8))              # unsupported head_dim
    with pytest.raises(M.MkvError):
        M.Pool(128, 1, 9, 1, 1, np.ones(128, np.int8))             # more than 8 query heads per KV head
    with pytest.raises(M.MkvError) as e:
        case.pool.page_read_raw(M.FMT_TQ3, 10 ** 6)
    assert e.value.code == M.E_BOUNDS


def test_append_and_decode_replay_from_a_cuda_graph():
    """The step's device calls take only stream-ordered actions, so they can be captured once and
    replayed (Section 4.1 runs the decode path from a CUDA graph).  The replayed result must equal
    the directly launched one bit for bit, for split rows too, and new lengths must be picked up from
    the captured buffers."""
    spec = SCALED["cfg2"]()                     # 8 rows over all blocks: every row is split and merged by ticket
    case = Case(spec, extra_fp8=4)
    pool = case.pool
    pool.set_decode_variant(M.DECODE_TENSOR)
    out_direct = pool.decode_attention(case.q, case.bt, case.tags, case.lens, spec.scale).clone()
    lens2 = case.lens.clone()
    lens2[1] -= 16 * 3 + 5                      # a shorter second request (its last page becomes partial)
    out_direct2 = pool.decode_attention(case.q, case.bt, case.tags, lens2, spec.scale).clone()
    torch.cuda.synchronize()

    cur_lens = case.lens.clone()
    out_graph = torch.zeros_like(out_direct)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        pool.decode_attention(case.q, case.bt, case.tags, cur_lens, spec.scale, out=out_graph)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out_graph, out_direct)
    cur_lens.copy_(lens2)
    g.replay()
    g.replay()                                   # tickets are left clear: a second replay gives the same
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    assert torch.equal(out_graph, out_direct2)
    check_close(out_graph.cpu().numpy(),
                oracle.decode_attention(case.L.fp8_arena, case.L.tq3_arena, spec.head_dim, spec.n_kv_heads, spec.group,
                                        case.L.sigma, case.L.q_bits, case.tab.block_table, case.tab.tier_tag,
                                        lens2.cpu().numpy(), spec.scale)[0], "graph replay")


def test_decode_maximum_batch_of_short_requests():
    """1,024 requests (the largest batch a call accepts) of 0 to 70 tokens: every block walks many
    (request, KV head) rows, most of them whole, some split at a block boundary."""
    rng = np.random.default_rng(17)
    lens = [int(x) for x in rng.integers(0, 71, size=1024)]
    lens[0], lens[1], lens[-1] = 0, 70, 1
    spec = W.config(0, seq_lens=lens, head_dim=128, n_kv_heads=2, group=3, anchor_prefix=16, recent_tokens=20, n_outlier=2)
    case = Case(spec)
    out, lse = case.run(M.DECODE_TENSOR)
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)
    # one request more than the maximum is refused before anything is launched
    q2 = torch.zeros((1025, spec.n_q_heads, 128), dtype=torch.bfloat16, device="cuda:0")
    bt2 = torch.zeros((1025, case.bt.shape[1]), dtype=torch.int32, device="cuda:0")
    tg2 = torch.zeros((1025, case.bt.shape[1]), dtype=torch.uint8, device="cuda:0")
    ln2 = torch.zeros(1025, dtype=torch.int32, device="cuda:0")
    big = M.Pool(128, 2, 6, 4, 4, case.L.sigma, max_batch=1025)
    with pytest.raises(M.MkvError) as e:
        big.decode_attention(q2, bt2, tg2, ln2, spec.scale)
    assert e.value.code == M.E_INVALID


def test_decode_one_long_row_and_the_page_limit():
    """One request of 12,000 pages on a single KV head: 148 blocks share one row (the longest split the
    tests see), with Anchor spans in the middle.  A table wider than 65,535 pages is refused."""
    spec = W.config(0, seq_lens=(16 * 12000 - 5,), head_dim=128, n_kv_heads=1, group=2, anchor_prefix=64, anchor_spans=3,
                    anchor_span_tokens=160, recent_tokens=1000, n_outlier=2)
    case = Case(spec)
    out, lse = case.run(M.DECODE_TENSOR)
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)
    wide_bt = torch.zeros((1, 65536), dtype=torch.int32, device="cuda:0")
    wide_tg = torch.zeros((1, 65536), dtype=torch.uint8, device="cuda:0")
    with pytest.raises(M.MkvError) as e:
        case.pool.decode_attention(case.q, wide_bt, wide_tg, case.lens, spec.scale)
    assert e.value.code == M.E_INVALID
    assert b"65535" in M.lib().mkv_last_cuda_error()
