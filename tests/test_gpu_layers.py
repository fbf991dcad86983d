"""mkv_decode_attention_layers / mkv_append_layers (several layers in one launch), the length clamp and the
bounded wait of the decode scan, all through the C ABI."""
import numpy as np
import pytest
import torch

import mkv_workloads as W
import oracle
import paper_2608_23834_b200 as M
from _gpu_util import Case, check_case, check_close

pytestmark = pytest.mark.gpu


def _layer_cases(n_layers, spec_fn):
    return [Case(spec_fn(), layer=i, extra_fp8=4) for i in range(n_layers)]


@pytest.mark.parametrize("name", ["cfg2", "cfg1", "edge", "pages_of_832", "pages_of_48_d128"])
def test_layers_call_equals_per_layer_calls(name):
    """Section 4.1: the decode step of all layers runs as one unit.  One launch over three pools must give,
    bit for bit, what three calls give (the per-layer arithmetic is the same code), and match the oracle."""
    fn = {"cfg2": lambda: W.config(2, seq_lens=(5008, 4432), recent_tokens=512, n_layers=3),
          "cfg1": lambda: W.config(1, seq_lens=(2048 + 16 * i for i in range(8)), recent_tokens=256, anchor_span_tokens=64),
          "pages_of_832": lambda: W.config(2, seq_lens=(9 * 832 + 100, 7 * 832), anchor_prefix=832, recent_tokens=900,
                                           n_layers=3, page_tokens=832),
          "pages_of_48_d128": lambda: W.config(1, seq_lens=(48 * 21 + 5, 48 * 30, 47, 48 * 9 + 47), anchor_prefix=48,
                                               recent_tokens=100, anchor_span_tokens=96, page_tokens=48),
          "edge": lambda: W.config(0, seq_lens=(0, 1, 15, 16, 17, 33, 16 * 20 + 9, 300), head_dim=128, n_kv_heads=2, group=4,
                                   anchor_prefix=16, recent_tokens=40, n_outlier=3)}[name]
    cases = _layer_cases(3, fn)
    spec = cases[0].spec
    singles = []
    for c in cases:
        lse = torch.zeros((spec.batch, spec.n_q_heads), dtype=torch.float32, device="cuda:0")
        singles.append((c.pool.decode_attention(c.q, c.bt, c.tags, c.lens, spec.scale, lse=lse).clone(), lse))
    outs = [torch.full_like(singles[0][0], 7.0) for _ in cases]
    lses = [torch.full_like(singles[0][1], 7.0) for _ in cases]
    M.decode_attention_layers([c.pool for c in cases], [c.q for c in cases], [c.bt for c in cases],
                              [c.tags for c in cases], cases[0].lens, spec.scale, outs, lses)
    torch.cuda.synchronize()
    for i, c in enumerate(cases):
        assert c.pool.status() == M.OK
        assert torch.equal(outs[i], singles[i][0]) and torch.equal(lses[i], singles[i][1]), i
        ref, ref_lse = c.reference()
        check_case(c, outs[i].cpu().numpy(), lses[i].cpu().numpy(), ref, ref_lse)
    # captured once, replayed twice (the tickets of every layer's workspace return to zero)
    g = torch.cuda.CUDAGraph()
    outs2 = [torch.zeros_like(o) for o in outs]
    with torch.cuda.graph(g):
        M.decode_attention_layers([c.pool for c in cases], [c.q for c in cases], [c.bt for c in cases],
                                  [c.tags for c in cases], cases[0].lens, spec.scale, outs2)
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    for i in range(3):
        assert torch.equal(outs2[i], outs[i])


def test_layers_call_argument_checks():
    a = Case(W.config(0, seq_lens=(64,)))
    b = Case(W.config(0, seq_lens=(64,), head_dim=256))
    out = torch.zeros((1, a.spec.n_q_heads, 128), dtype=torch.float32, device="cuda:0")
    with pytest.raises(M.MkvError) as e:                         # same workspace twice
        M.decode_attention_layers([a.pool, a.pool], [a.q, a.q], [a.bt, a.bt], [a.tags, a.tags], a.lens, a.spec.scale, [out, out])
    assert e.value.code == M.E_INVALID and b"workspace" in M.lib().mkv_last_cuda_error()
    out_b = torch.zeros((1, b.spec.n_q_heads, 256), dtype=torch.float32, device="cuda:0")
    with pytest.raises(M.MkvError) as e:                         # different geometry
        M.decode_attention_layers([a.pool, b.pool], [a.q, b.q], [a.bt, a.bt], [a.tags, a.tags], a.lens, a.spec.scale, [out, out_b])
    assert e.value.code == M.E_INVALID


def test_append_layers_is_bit_exact_with_per_layer_append():
    d, hkv, n = 256, 4, 5
    sig = np.ones(d, np.int8)
    rng = np.random.default_rng(5)
    pools_a = [M.Pool(d, hkv, hkv, 8, 1, sig, max_batch=1) for _ in range(3)]
    pools_b = [M.Pool(d, hkv, hkv, 8, 1, sig, max_batch=1) for _ in range(3)]
    ks = [torch.from_numpy(rng.standard_normal((n, hkv, d)).astype(np.float32) * 40).cuda().to(torch.bfloat16) for _ in range(3)]
    vs = [torch.from_numpy(rng.standard_normal((n, hkv, d)).astype(np.float32) * 40).cuda().to(torch.bfloat16) for _ in range(3)]
    slots = torch.tensor([3, 16 * 2 + 15, -1, 16 * 7, 16 * 9 + 1], dtype=torch.int32, device="cuda:0")   # one skipped, one beyond the arena
    for p, k, v in zip(pools_a, ks, vs):
        p.append(k, v, slots)
    M.append_layers(pools_b, ks, vs, slots)
    torch.cuda.synchronize()
    for pa, pb in zip(pools_a, pools_b):
        assert pa.status() == M.E_BOUNDS and pb.status() == M.E_BOUNDS
        for pid in range(8):
            assert np.array_equal(pa.page_read_raw(M.FMT_FP8, pid), pb.page_read_raw(M.FMT_FP8, pid))


@pytest.mark.parametrize("variant", [M.DECODE_TENSOR, M.DECODE_SCALAR, M.DECODE_TMEM])
@pytest.mark.parametrize("d", [128, 256])
def test_sequence_length_beyond_the_table_is_cut_and_flagged(d, variant):
    """A seq_len larger than the table row can hold must not make the scan read past the row: the length
    is cut to max_pages * 16, the status word says MKV_E_BOUNDS, and the output equals that of the cut length."""
    spec = W.config(0, seq_lens=(16 * 9, 16 * 12), head_dim=d, n_kv_heads=2, group=3, anchor_prefix=16, recent_tokens=48)
    case = Case(spec)
    case.pool.set_decode_variant(variant)
    max_pages = case.bt.shape[1]
    assert max_pages == 12
    good = case.pool.decode_attention(case.q, case.bt, case.tags, case.lens, spec.scale).clone()
    torch.cuda.synchronize()
    assert case.pool.status() == M.OK
    long_lens = case.lens.clone()
    long_lens[1] = 16 * 12 + 16 * 100000                        # far beyond the row (and beyond the arena)
    out = case.pool.decode_attention(case.q, case.bt, case.tags, long_lens, spec.scale)
    torch.cuda.synchronize()
    assert case.pool.status() == M.E_BOUNDS
    assert torch.isfinite(out).all()
    assert torch.equal(out, good)                                 # request 1 is full to the last entry: same pages read
    out2 = case.pool.decode_attention(case.q, case.bt, case.tags, case.lens, spec.scale)     # still usable
    torch.cuda.synchronize()
    assert case.pool.status() == M.OK and torch.equal(out2, good)


def test_scored_call_with_a_length_beyond_the_table_writes_inside_its_buffers():
    spec = W.config(0, seq_lens=(16 * 9, 16 * 12), head_dim=128, n_kv_heads=2, group=3, anchor_prefix=16, recent_tokens=48)
    case = Case(spec)
    B, hq, mp = 2, spec.n_q_heads, case.bt.shape[1]
    guard = torch.full((B * hq * mp + 64,), 12345.0, dtype=torch.float32, device="cuda:0")
    mass = guard[:B * hq * mp].view(B, hq, mp)
    score_buf = torch.full((B * mp + 64,), 0.5, dtype=torch.float32, device="cuda:0")
    score = score_buf[:B * mp].view(B, mp)
    long_lens = case.lens.clone()
    long_lens[1] = 10 ** 7
    out, lse, _ = case.pool.decode_attention_scored(case.q, case.bt, case.tags, long_lens, spec.scale, page_mass=mass)
    M.page_score_update(mass, long_lens, 0b111, 0.5, score)
    torch.cuda.synchronize()
    assert case.pool.status() == M.E_BOUNDS
    assert torch.isfinite(out).all() and torch.isfinite(mass).all()
    assert bool((guard[B * hq * mp:] == 12345.0).all()) and bool((score_buf[B * mp:] == 0.5).all())
    assert abs(float(mass[1].sum()) - hq) < 1e-3                  # still a distribution over the row's pages


def test_a_wait_that_runs_out_is_reported_and_the_pool_stays_usable():
    """Section 4.1 ("fails closed"): with the diagnostic wait limit of zero the scan's first look at a copy
    that is still in flight counts as a time-out.  The blocks then wait for what they have in flight, finish
    and take their tickets; the status word says MKV_E_TIMEOUT; the next call with the normal limit is correct."""
    spec = W.config(2, seq_lens=(5008, 4432), recent_tokens=512, n_layers=1)
    case = Case(spec)
    out, lse = case.run(M.DECODE_TENSOR)
    ref, ref_lse = case.reference()
    check_case(case, out, lse, ref, ref_lse)
    case.pool.set_wait_limit_ns(0)
    case.pool.decode_attention(case.q, case.bt, case.tags, case.lens, spec.scale)
    torch.cuda.synchronize()
    assert case.pool.status() == M.E_TIMEOUT
    case.pool.set_wait_limit_ns(20_000_000)
    for _ in range(2):                                            # tickets were left at zero: split rows merge as usual
        out2, lse2 = case.run(M.DECODE_TENSOR)
        assert np.array_equal(out2, out) and np.array_equal(lse2, lse)
