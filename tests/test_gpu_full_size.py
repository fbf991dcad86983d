"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: one full layer of
config 2 (every output), config 1 as specified, and the ragged 64-request config 3 with the oracle
computing a sample of requests (the pages of the other requests are zero records, which are valid
input)."""
import numpy as np
import pytest
import torch

import mkv_workloads as W
import oracle
import paper_2608_23834_b200 as M
from _gpu_util import Case, bf16_tensor, check_case, check_close

pytestmark = pytest.mark.gpu


def test_config2_one_full_layer_every_output():
    spec = W.config(2, n_layers=1)
    assert spec.seq_lens == (59008, 59008) and spec.head_dim == 256
    case = Case(spec, layer=3)
    out, lse = case.run(M.DECODE_TENSOR)
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)
    out_tm, lse_tm = case.run(M.DECODE_TMEM)                 # the tcgen05 kernel on the same layer
    check_case(case, out_tm, lse_tm, ref, ref_lse)
    case.pool.set_decode_variant(M.DECODE_TENSOR)
    # the scored call on the same layer: same output bit for bit, page mass against the oracle
    out_s, _, mass = case.pool.decode_attention_scored(case.q, case.bt, case.tags, case.lens, spec.scale)
    torch.cuda.synchronize()
    assert np.array_equal(out_s.cpu().numpy(), out)
    ref_mass = oracle.page_mass(case.L.fp8_arena, case.L.tq3_arena, spec.head_dim, spec.n_kv_heads, spec.group, case.L.sigma,
                                case.L.q_bits, case.tab.block_table, case.tab.tier_tag, case.tab.seq_lens, spec.scale)
    got = mass.cpu().numpy().astype(np.float64)
    assert (np.abs(got - ref_mass) <= 1e-6 + 1e-4 * ref_mass).all(), np.abs(got - ref_mass).max()


def test_config1_as_specified():
    case = Case(W.config(1))
    out, lse = case.run(M.DECODE_TENSOR)
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)


def test_config3_ragged_batch_sampled_requests():
    spec = W.config(3)
    tab = W.tables(spec)
    d, hkv = spec.head_dim, spec.n_kv_heads
    order = np.argsort(spec.seq_lens)
    sample = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2]), int(order[5]), 7})
    from oracle.harness import build_layer
    L = build_layer(spec, tab, requests=sample)          # other requests keep zero pages
    pool = M.Pool(d, hkv, spec.n_q_heads, tab.fp8_pages, tab.tq3_pages, L.sigma, max_batch=spec.batch)
    pool.upload_arenas(L.fp8_arena, L.tq3_arena)
    out = pool.decode_attention(bf16_tensor(L.q_bits), torch.from_numpy(tab.block_table).cuda(),
                                torch.from_numpy(tab.tier_tag).cuda(), torch.from_numpy(tab.seq_lens).cuda(), spec.scale)
    torch.cuda.synchronize()
    assert pool.status() == M.OK
    out = out.cpu().numpy()
    assert np.isfinite(out).all()
    for b in sample:
        ref, _ = oracle.decode_attention(L.fp8_arena, L.tq3_arena, d, hkv, spec.group, L.sigma, L.q_bits, tab.block_table,
                                         tab.tier_tag, tab.seq_lens, spec.scale, only_b=b)
        check_close(out[b], ref[b], f"config 3 request {b} len {spec.seq_lens[b]}")
    # a request whose pages are all zero records attends uniformly to zeros
    other = [b for b in range(spec.batch) if b not in sample][0]
    assert not out[other].any()


def test_long_rows_many_rounds_kernels_agree():
    """Rows long enough that every block lists its pages in several rounds (thousands of pages per block and
    row): the two tensor-core kernels must agree with each other (2.8 M token-heads),
    and a sampled (request, KV head) row is checked against the oracle on its own."""
    spec = W.config(2, seq_lens=(16 * 24000 - 3, 16 * 20000), n_layers=1, recent_tokens=4096, anchor_prefix=512,
                    anchor_spans=3, anchor_span_tokens=640)
    tab = W.tables(spec)
    d, hkv = spec.head_dim, spec.n_kv_heads
    # pages: random valid records (any byte pattern is a valid record for the kernels except NaN bytes 0x7F/0xFF
    # in FP8 records and fp16 specials in the TQ3 metadata, which the generator below avoids)
    g = torch.Generator(device="cuda").manual_seed(7)
    pool = M.Pool(d, hkv, spec.n_q_heads, tab.fp8_pages, tab.tq3_pages, W.rotation_signs(spec, 0), max_batch=spec.batch)
    fp8 = torch.randint(0, 0x48, (tab.fp8_pages, hkv, 32 * d), generator=g, device="cuda", dtype=torch.uint8)      # |x| < 4
    fp8 |= (torch.randint(0, 2, fp8.shape, generator=g, device="cuda", dtype=torch.uint8) << 7)
    tq3 = torch.randint(0, 256, (tab.tq3_pages, hkv, 16 * d + 32), generator=g, device="cuda", dtype=torch.uint8)
    meta16 = tq3[:, :, 12 * d:].view(torch.int16)              # key norms, value scales and zeros: fp16 in (-2, 2)
    meta16 &= -16385                                             # clear the top exponent bit (0x4000): |x| < 2, never inf/nan
    pool.fp8_arena.view(torch.uint8)[:fp8.numel()].copy_(fp8.reshape(-1))
    pool.tq3_arena.view(torch.uint8)[:tq3.numel()].copy_(tq3.reshape(-1))
    q = bf16_tensor(W.query(spec, 0))
    bt = torch.from_numpy(tab.block_table).cuda()
    tg = torch.from_numpy(tab.tier_tag).cuda()
    ln = torch.from_numpy(tab.seq_lens).cuda()
    outs = {}
    for name, variant in (("tensor", M.DECODE_TENSOR), ("tmem", M.DECODE_TMEM)):
        pool.set_decode_variant(variant)
        lse = torch.empty((spec.batch, spec.n_q_heads), dtype=torch.float32, device="cuda")
        outs[name] = (pool.decode_attention(q, bt, tg, ln, spec.scale, lse=lse).cpu().numpy(), lse.cpu().numpy())
        torch.cuda.synchronize()
        assert pool.status() == M.OK
    a, b = outs["tensor"], outs["tmem"]
    assert np.isfinite(a[0]).all() and np.isfinite(b[0]).all()
    assert np.abs(a[0] - b[0]).max() <= 2e-4 * max(1.0, np.abs(a[0]).max())
    assert np.abs(a[1] - b[1]).max() <= 1e-4
    # one row against the oracle, which gets the same arenas
    ref, ref_lse = oracle.decode_attention(fp8.cpu().numpy(), tq3.cpu().numpy(), d, hkv, spec.group, W.rotation_signs(spec, 0),
                                           W.query(spec, 0), tab.block_table, tab.tier_tag, tab.seq_lens, spec.scale,
                                           only_b=1, only_h=2)
    G = spec.group
    check_close(a[0][1, 2 * G:3 * G], ref[1, 2 * G:3 * G], "long row, request 1, KV head 2")


def _layers_call(cases, lse=True):
    """The call bench.py times: all layers in one launch (mkv_decode_attention_layers)."""
    spec = cases[0].spec
    outs = [torch.full((spec.batch, spec.n_q_heads, spec.head_dim), 7.0, dtype=torch.float32, device="cuda:0") for _ in cases]
    lses = [torch.full((spec.batch, spec.n_q_heads), 7.0, dtype=torch.float32, device="cuda:0") for _ in cases] if lse else None
    M.decode_attention_layers([c.pool for c in cases], [c.q for c in cases], [c.bt for c in cases],
                              [c.tags for c in cases], cases[0].lens, spec.scale, outs, lses)
    torch.cuda.synchronize()
    for c in cases:
        assert c.pool.status() == M.OK
    return [o.cpu().numpy() for o in outs], ([l.cpu().numpy() for l in lses] if lse else None)


def test_config2_record_format2_two_full_layers_in_one_launch_every_output():
    """The benchmark's default: pools of record format 2, the layers of the step in one launch.  Two full
    layers of config 2 (different pages, tables' ids and queries per layer), every output of both."""
    with oracle.record_format(2):
        spec = W.config(2, n_layers=2)
        cases = [Case(spec, layer=i) for i in range(2)]
        outs, lses = _layers_call(cases)
        for i, c in enumerate(cases):
            ref, ref_lse = c.reference()
            check_case(c, outs[i], lses[i], ref, ref_lse)


def test_config3_one_request_per_length_decile():
    """Config 3 as specified (64 ragged requests, 1,024 .. 131,072 tokens), record format 2, through the call the
    benchmark times; the oracle computes the shortest, the longest and one request per decile of the length order
    (the test above covers record format 1 and the single-layer call on a smaller sample)."""
    with oracle.record_format(2):
        spec = W.config(3)
        order = np.argsort(spec.seq_lens)
        sample = sorted({int(order[min(63, round(6.3 * k))]) for k in range(11)})
        assert len(sample) == 11 and int(order[0]) in sample and int(order[-1]) in sample
        case = Case(spec, requests=sample)
        (out,), (lse,) = _layers_call([case])
        assert np.isfinite(out).all()
        for b in sample:
            ref, ref_lse = case.reference(only_b=b)
            check_close(out[b], ref[b], f"config 3 request {b} len {spec.seq_lens[b]}")
            assert np.abs(lse[b] - ref_lse[b]).max() < 2e-3
        other = [b for b in range(spec.batch) if b not in sample][0]
        assert not out[other].any()


CORNERS = [(b, c, f) for b in (1, 32) for c in (4096, 131072) for f in (0.0, 0.95)]


@pytest.mark.parametrize("batch,ctx,frac", CORNERS)
def test_config4_corner_cells_at_full_size(batch, ctx, frac):
    """The eight corners of the config-4 sweep (batch x context x Stale fraction) at their full sizes, record
    format 2, through the call the benchmark times.  The oracle computes every request of the small cells and
    two sampled requests of the large 32-request cells (the pages of the others are zero records)."""
    with oracle.record_format(2):
        spec = W.config(4, batch=batch, ctx=ctx, stale_fraction=frac)
        sample = list(range(batch)) if batch * ctx <= 262144 else [5, 31] if ctx <= 4096 * 8 else [3, 17]
        case = Case(spec, requests=sample)
        (out,), (lse,) = _layers_call([case])
        assert np.isfinite(out).all()
        for b in sample:
            ref, ref_lse = case.reference(only_b=b)
            check_close(out[b], ref[b], f"{spec.name} request {b}")
            assert np.abs(lse[b] - ref_lse[b]).max() < 2e-3
