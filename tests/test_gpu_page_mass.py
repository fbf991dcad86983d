"""Parity of mkv_decode_attention_scored / mkv_page_score_update with the fp64 oracle (Section 3.1:
Eq. score-partial, Eq. score-global-weight, Eq. attention-score) on identical quantised pages."""
import numpy as np
import pytest
import torch

import mkv_workloads as W
import oracle
import paper_2608_23834_b200 as M
from _gpu_util import Case, check_case

pytestmark = pytest.mark.gpu

# q~ lies in [0, 1]; the kernel takes it from fp32 page sums (fp16 hi + lo probabilities), one lg2 and one
# ex2 approximation: a few 1e-7 relative.  Bound used: 1e-6 absolute plus 1e-4 relative.
MASS_ABS, MASS_REL = 1e-6, 1e-4

CASES = {
    "cfg0": lambda: W.config(0),
    "cfg1": lambda: W.config(1, seq_lens=(2048 + 16 * i for i in range(8)), recent_tokens=256, anchor_span_tokens=64),
    "cfg2": lambda: W.config(2, seq_lens=(5008, 4432), recent_tokens=512, n_layers=1),
    "cfg3": lambda: W.config(3, seq_lens=[int(1024 * 8 ** u) for u in np.random.default_rng(3).random(12)], recent_tokens=200),
    "cfg4_f95": lambda: W.config(4, batch=3, ctx=1024, stale_fraction=0.95),
    "ragged": lambda: W.config(1, seq_lens=(1, 17, 0, 1000, 16, 333), recent_tokens=40, anchor_spans=0),
    # pages of several 16-token tiles: a page's mass is gathered from the warps and blocks that scan its tiles
    "pages_of_48": lambda: W.config(0, seq_lens=(21 * 48 + 37, 4 * 48, 0, 17), head_dim=128, n_kv_heads=2, group=4,
                                    anchor_prefix=48, anchor_spans=2, anchor_span_tokens=96, recent_tokens=150, page_tokens=48,
                                    seed=31),
    "pages_of_832_d256": lambda: W.config(2, seq_lens=(11 * 832 + 500, 9 * 832), anchor_prefix=832, recent_tokens=1700,
                                          n_layers=1, page_tokens=832),
}


def oracle_mass(case):
    s = case.spec
    return oracle.page_mass(case.L.fp8_arena, case.L.tq3_arena, s.head_dim, s.n_kv_heads, s.group, case.L.sigma,
                            case.L.q_bits, case.tab.block_table, case.tab.tier_tag, case.tab.seq_lens, s.scale,
                            page_tokens=s.page_tokens)


@pytest.mark.parametrize("name", list(CASES))
def test_page_mass_matches_oracle(name):
    case = Case(CASES[name](), extra_fp8=3, extra_tq3=2)
    spec = case.spec
    mass = torch.full((spec.batch, spec.n_q_heads, case.bt.shape[1]), 7.0, dtype=torch.float32, device="cuda:0")
    out, lse, mass = case.pool.decode_attention_scored(case.q, case.bt, case.tags, case.lens, spec.scale, page_mass=mass)
    torch.cuda.synchronize()
    assert case.pool.status() == M.OK
    ref_out, ref_lse = case.reference()
    check_case(case, out.cpu().numpy(), lse.cpu().numpy(), ref_out, ref_lse)      # the output is unchanged by scoring
    got, ref = mass.cpu().numpy().astype(np.float64), oracle_mass(case)
    assert np.isfinite(got).all()
    assert (np.abs(got - ref) <= MASS_ABS + MASS_REL * ref).all(), np.abs(got - ref).max()
    for b in range(spec.batch):
        npg = spec.n_pages(b)
        assert not got[b, :, npg:].any()                                          # beyond the length: zero
        if npg:
            assert np.abs(got[b, :, :npg].sum(1) - 1.0).max() < 1e-5
    # the unscored call gives the same output bit for bit
    out2 = case.pool.decode_attention(case.q, case.bt, case.tags, case.lens, spec.scale)
    assert torch.equal(out, out2)


@pytest.mark.parametrize("name", ["cfg2", "pages_of_832_d256"])
def test_score_update_matches_oracle_over_two_steps(name):
    case = Case(CASES[name]())
    spec = case.spec
    _, _, mass = case.pool.decode_attention_scored(case.q, case.bt, case.tags, case.lens, spec.scale)
    P = case.bt.shape[1]
    score = torch.zeros((spec.batch, P), dtype=torch.float32, device="cuda:0")
    score[:, ::3] = 0.5
    ref = score.cpu().numpy().astype(np.float64)
    mask = 0b100100100100100100100101                                              # a sampled head set
    ref_mass = oracle_mass(case)
    for beta in (0.9, 0.5):
        M.page_score_update(mass, case.lens, mask, beta, score, page_tokens=spec.page_tokens)
        ref = oracle.page_score_update(ref_mass, case.tab.seq_lens, mask, beta, ref, page_tokens=spec.page_tokens)
    torch.cuda.synchronize()
    got = score.cpu().numpy().astype(np.float64)
    assert np.abs(got - ref).max() <= 2e-6
    npg = spec.n_pages(1)
    assert np.array_equal(got[1, npg:], np.where(np.arange(npg, P) % 3 == 0, 0.5, 0.0).astype(np.float64))


def test_scored_call_validates_its_arguments():
    case = Case(W.config(0, seq_lens=(256,)))
    spec = case.spec
    L = M.lib()
    mass = torch.empty((1, spec.n_q_heads, case.bt.shape[1]), dtype=torch.float32, device="cuda:0")
    out = torch.empty((1, spec.n_q_heads, spec.head_dim), dtype=torch.float32, device="cuda:0")
    ws = case.pool.workspace
    args = lambda lse, pm: (case.pool.handle, M._ptr(case.q), M._ptr(case.bt), M._ptr(case.tags), M._ptr(case.lens), 1,
                            case.bt.shape[1], spec.scale, M._ptr(out), lse, pm, M._ptr(ws), ws.numel(), None)
    assert L.mkv_decode_attention_scored(*args(None, M._ptr(mass))) == M.E_INVALID     # lse is required
    lse = torch.empty((1, spec.n_q_heads), dtype=torch.float32, device="cuda:0")
    assert L.mkv_decode_attention_scored(*args(M._ptr(lse), None)) == M.E_INVALID
    assert L.mkv_page_score_update(M._ptr(mass), M._ptr(case.lens), 1, spec.n_q_heads, case.bt.shape[1], 0, 0.5,
                                   M._ptr(mass), None) == M.E_INVALID                  # empty head set
    assert L.mkv_page_score_update(M._ptr(mass), M._ptr(case.lens), 1, spec.n_q_heads, case.bt.shape[1], 1, 1.5,
                                   M._ptr(mass), None) == M.E_INVALID                  # beta outside [0, 1]
