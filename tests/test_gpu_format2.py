"""Record format 2 (e4m3-exact key codebook, FP8 key products) through the C ABI: Demote and Promote bit-exact
with the oracle, decode attention within the tolerance of format 1, on the same cases."""
import numpy as np
import pytest
import torch

import mkv_workloads as W
import oracle
import paper_2608_23834_b200 as M
from _gpu_util import Case, check_case, check_close
from test_gpu_decode import SCALED

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def format2():
    with oracle.record_format(2):
        yield


VARIANTS = [pytest.param(M.DECODE_TENSOR, id="tensor"), pytest.param(M.DECODE_SCALAR, id="scalar")]

# eight e4m3-exact entries (rest zero, rotation signs +1) whose squares sum to N^2 and that sum to threshold j * N
TIES = [(16, 8, 0, [1, -8, 4, -4, 10, -3, 7, 1]), (32, 34, 1, [2, 11, 11, 0, -18, -2, 15, 15]),
        (32, 58, 2, [9, -4, 14, -6, 9, 3, 22, 11])]


@pytest.mark.parametrize("d,hkv,k_scale,v_scale", [(128, 2, 1.0, 1.0), (256, 4, 1.0, 1.0), (256, 1, 0.25, 4.0)])
def test_demote_and_promote_are_bit_exact_in_format2(d, hkv, k_scale, v_scale):
    rng = np.random.default_rng(500 + d + hkv)
    n = 7
    sigma = (rng.integers(0, 2, d) * 2 - 1).astype(np.int8)
    pool = M.Pool(d, hkv, hkv, 2 * n, n, sigma, k_scale, v_scale, tq3_format=2)
    recs = np.zeros((n, hkv, 32 * d), np.uint8)
    for p in range(n):
        for h in range(hkv):
            k = rng.standard_normal((16, d)).astype(np.float32)
            v = rng.standard_normal((16, d)).astype(np.float32)
            k[:, rng.integers(0, d, 3)] *= 8
            v[:, rng.integers(0, d, 3)] *= 8
            if p == 1:
                k[3] = 0.0
                v[:, 5] = 1.5
            recs[p, h] = oracle.fp8_pack_record(k, v, 16, k_scale, v_scale)
        pool.page_write_raw(M.FMT_FP8, p, recs[p])
    ids = torch.arange(n, dtype=torch.int32, device="cuda:0")
    dst = torch.from_numpy(rng.permutation(n).astype(np.int32)).cuda()
    pool.demote(ids, dst)
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    t = dst.cpu().numpy()
    stale = np.zeros((n, hkv, 16 * d + 32), np.uint8)
    with oracle.record_format(1):
        other = oracle.demote_record(recs[0, 0], d, sigma, k_scale, v_scale)
    for i in range(n):
        stale[i] = pool.page_read_raw(M.FMT_TQ3, int(t[i])).reshape(hkv, -1)
        for h in range(hkv):
            ref = oracle.demote_record(recs[i, h], d, sigma, k_scale, v_scale)
            assert np.array_equal(stale[i, h], ref), (i, h, np.nonzero(stale[i, h] != ref)[0][:8])
    assert not np.array_equal(stale[0, 0], other)            # and it is not the format-1 record
    pool.promote(dst, (ids + n).contiguous())
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    for i in range(n):
        got = pool.page_read_raw(M.FMT_FP8, n + i).reshape(hkv, 32 * d)
        for h in range(hkv):
            assert np.array_equal(got[h], oracle.promote_record(stale[i, h], d, sigma, k_scale, v_scale)), (i, h)


@pytest.mark.parametrize("d", [128, 256])
def test_demote_keeps_the_lower_magnitude_on_a_threshold(d):
    """Keys whose rotated coordinate equals threshold j times the norm (both signs): the strict comparison of
    the tie rule gives magnitude j; the kernel must write the bytes the oracle writes."""
    k = np.zeros((16, d), np.float32)
    want = {}
    for r, (N, on, j, head) in enumerate(TIES):
        k[2 * r, :8] = head
        k[2 * r + 1, :8] = [-x for x in head]
        want[2 * r], want[2 * r + 1] = (j, 0), (j, 1)
    v = np.zeros((16, d), np.float32)
    sigma = np.ones(d, np.int8)
    rec8 = oracle.fp8_pack_record(k, v)
    kq, _ = oracle.fp8_unpack_record_f32(rec8, d)
    assert np.array_equal(kq, k)                               # every entry is e4m3-exact
    pool = M.Pool(d, 1, 1, 2, 2, sigma, tq3_format=2)
    pool.page_write_raw(M.FMT_FP8, 0, rec8)
    one = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    pool.demote(one, one)
    torch.cuda.synchronize()
    got = pool.page_read_raw(M.FMT_TQ3, 0)
    assert np.array_equal(got, oracle.demote_record(rec8, d, sigma))
    kc = oracle.tq3_unpack_record(got, d)[0]
    for t, (j, sgn) in want.items():
        assert np.all((kc[t, ::8] & 3) == j) and np.all((kc[t, ::8] >> 2) == sgn), t


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("name", list(SCALED))
def test_decode_matches_oracle_on_scaled_configs_in_format2(name, variant):
    case = Case(SCALED[name](), extra_fp8=5, extra_tq3=7)
    out, lse = case.run(variant)
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("d,hkv,group", [(128, 2, 4), (256, 1, 6), (128, 1, 1), (256, 2, 8), (128, 3, 5)])
def test_decode_edge_lengths_in_format2(d, hkv, group, variant):
    lens = (0, 1, 15, 16, 17, 33, 16 * 20, 16 * 20 + 9, 300)
    spec = W.config(0, seq_lens=lens, head_dim=d, n_kv_heads=hkv, group=group, anchor_prefix=16, recent_tokens=40, n_outlier=3)
    case = Case(spec, extra_fp8=2, extra_tq3=2)
    out, lse = case.run(variant)
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)


def test_all_stale_tier_and_the_layers_call_in_format2():
    spec_fn = lambda: W.config(2, seq_lens=(5008, 4432), recent_tokens=512, n_layers=3)
    cases = [Case(spec_fn(), layer=i, extra_fp8=4) for i in range(3)]
    spec = cases[0].spec
    outs = [torch.zeros((spec.batch, spec.n_q_heads, spec.head_dim), dtype=torch.float32, device="cuda:0") for _ in cases]
    lses = [torch.zeros((spec.batch, spec.n_q_heads), dtype=torch.float32, device="cuda:0") for _ in cases]
    M.decode_attention_layers([c.pool for c in cases], [c.q for c in cases], [c.bt for c in cases], [c.tags for c in cases],
                              cases[0].lens, spec.scale, outs, lses)
    torch.cuda.synchronize()
    for i, c in enumerate(cases):
        assert c.pool.status() == M.OK
        single = c.pool.decode_attention(c.q, c.bt, c.tags, c.lens, spec.scale)
        assert torch.equal(single, outs[i])
        ref, ref_lse = c.reference()
        check_case(c, outs[i].cpu().numpy(), lses[i].cpu().numpy(), ref, ref_lse)
    allst = Case(W.config(1, seq_lens=(640, 1600, 16), anchor_prefix=0, recent_tokens=0, anchor_spans=0))
    out, lse = allst.run(M.DECODE_TENSOR)
    ref, ref_lse = allst.reference()
    check_case(allst, out, lse, ref, ref_lse)
    # pools of different formats do not go into one launch
    with oracle.record_format(1):
        old = Case(spec_fn(), layer=0, extra_fp8=4)
    with pytest.raises(M.MkvError) as e:
        M.decode_attention_layers([cases[0].pool, old.pool], [cases[0].q, old.q], [cases[0].bt, old.bt],
                                  [cases[0].tags, old.tags], cases[0].lens, spec.scale, outs[:2])
    assert e.value.code == M.E_INVALID


def test_page_mass_and_pages_of_several_tiles_in_format2():
    spec = W.config(0, seq_lens=(16 * 40 + 7, 16 * 13), head_dim=128, n_kv_heads=2, group=4, anchor_prefix=32, recent_tokens=64)
    case = Case(spec)
    out, lse, mass = case.pool.decode_attention_scored(case.q, case.bt, case.tags, case.lens, spec.scale)
    torch.cuda.synchronize()
    assert case.pool.status() == M.OK
    ref, ref_lse = case.reference()
    check_case(case, out.cpu().numpy(), lse.cpu().numpy(), ref, ref_lse)
    ref_mass = oracle.page_mass(case.L.fp8_arena, case.L.tq3_arena, spec.head_dim, spec.n_kv_heads, spec.group, case.L.sigma,
                                case.L.q_bits, case.tab.block_table, case.tab.tier_tag, case.tab.seq_lens, spec.scale)
    got = mass.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref_mass) <= 1e-6 + 1e-4 * np.abs(ref_mass))
    # pages of 4 tiles (64 tokens): the tiled scan reads format-2 key sections too
    spec4 = W.config(0, seq_lens=(64 * 9 + 5, 64 * 4), head_dim=256, n_kv_heads=2, group=3, anchor_prefix=64, recent_tokens=128,
                     page_tokens=64)
    c4 = Case(spec4)
    for variant in (M.DECODE_TENSOR, M.DECODE_SCALAR):
        out, lse = c4.run(variant)
        ref, ref_lse = c4.reference()
        check_case(c4, out, lse, ref, ref_lse)


def test_the_tensor_memory_variant_refuses_format2():
    case = Case(W.config(0, seq_lens=(200,), head_dim=256, recent_tokens=60))
    case.pool.set_decode_variant(M.DECODE_TMEM)
    with pytest.raises(M.MkvError) as e:
        case.pool.decode_attention(case.q, case.bt, case.tags, case.lens, case.spec.scale)
    assert e.value.code == M.E_INVALID and b"format 2" in M.lib().mkv_last_cuda_error()
    with pytest.raises(M.MkvError):
        M.Pool(128, 1, 1, 1, 1, np.ones(128, np.int8), tq3_format=3)


@pytest.mark.parametrize("variant", VARIANTS)
def test_queries_with_outlier_dims_a_zero_head_and_mixed_scales(variant):
    """The tensor-core scan carries the rotated query of format 2 as three base-128 digits per head, scaled to the
    head's largest component.  Heads whose query is zero, has a few components 20 times the rest, or is small as a
    whole must come out within the same tolerance."""
    spec = W.config(2, seq_lens=(3008, 1000), recent_tokens=256, n_layers=1)
    case = Case(spec, extra_fp8=2, extra_tq3=2)
    q = oracle.bf16_bits_to_f32(case.L.q_bits).copy()                 # [B][Hq][d]
    q[:, 0] = 0.0                                                      # a zero head: uniform attention
    q[:, 1, 7] *= 20.0                                                 # outlier components
    q[:, 1, 130] *= -20.0
    q[:, 2] *= 1e-3                                                    # a small head
    q[:, 3] *= 6.0                                                     # a large head (peaked attention)
    q[1, 4, :] = q[1, 4, 0]                                            # constant over the dims
    case.L.q_bits[:] = W.f32_to_bf16_bits(q)
    from _gpu_util import bf16_tensor
    case.q = bf16_tensor(case.L.q_bits)
    out, lse = case.run(variant)
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("k_scale,v_scale", [(0.5, 2.0), (3.0, 0.37)])
def test_decode_with_fp8_scales_other_than_one(k_scale, v_scale, variant):
    """Pool-level FP8 scales: a Recent/Anchor byte means e4m3 x scale (the Stale records carry their own norms,
    scales and zeros and are not rescaled).  The same pages read under other scales must match the oracle reading
    them under the same scales."""
    spec = W.config(1, seq_lens=(1500, 700, 16, 333), recent_tokens=400, anchor_span_tokens=64)
    case = Case(spec, extra_fp8=2, extra_tq3=2, k_scale=k_scale, v_scale=v_scale)
    out, lse = case.run(variant)
    s = spec
    ref, ref_lse = oracle.decode_attention(case.L.fp8_arena, case.L.tq3_arena, s.head_dim, s.n_kv_heads, s.group, case.L.sigma,
                                           case.L.q_bits, case.tab.block_table, case.tab.tier_tag, case.tab.seq_lens, s.scale,
                                           k_scale=k_scale, v_scale=v_scale)
    check_case(case, out, lse, ref, ref_lse)
    # and the scales matter: the result differs from the one under unit scales
    ref1, _ = case.reference()
    assert np.abs(ref - ref1).max() > 1e-2
