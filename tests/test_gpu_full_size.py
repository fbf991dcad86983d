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
