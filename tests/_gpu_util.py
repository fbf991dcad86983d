"""Helpers shared by the GPU tests: build a pool from a seeded workload whose pages were encoded by
the oracle, run the CUDA decode through the C ABI, and compare with the oracle."""
import numpy as np
import torch

import mkv_workloads as W
import oracle
import paper_2608_23834_b200 as M
from oracle.harness import build_layer

MAX_ABS, REL_L2 = 2e-3, 1e-3     # attention tolerance against the fp64 oracle on identical pages


def bf16_tensor(bits: np.ndarray, device="cuda:0") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


class Case:
    def __init__(self, spec, layer=0, extra_fp8=0, extra_tq3=0, k_scale=1.0, v_scale=1.0, requests=None):
        """requests: encode only these requests' pages (the others stay zero-filled records: valid input,
        compared nowhere) to keep the oracle's share of a full-size case short."""
        self.spec = spec
        self.tab = W.tables(spec, extra_fp8, extra_tq3)
        self.L = build_layer(spec, self.tab, layer, requests=requests)
        # the pool reads its Stale pages in the record format the oracle wrote them in
        self.fmt = oracle.get_format()
        self.pool = M.Pool(spec.head_dim, spec.n_kv_heads, spec.n_q_heads, max(self.tab.fp8_pages, 1),
                           max(self.tab.tq3_pages, 1), self.L.sigma, k_scale, v_scale, max_batch=spec.batch,
                           page_tokens=spec.page_tokens, tq3_format=self.fmt)
        self.pool.upload_arenas(self.L.fp8_arena, self.L.tq3_arena)
        self.q = bf16_tensor(self.L.q_bits)
        self.bt = torch.from_numpy(self.tab.block_table).cuda()
        self.tags = torch.from_numpy(self.tab.tier_tag).cuda()
        self.lens = torch.from_numpy(self.tab.seq_lens).cuda()

    def run(self, variant=M.DECODE_TENSOR, want_lse=True):
        self.pool.set_decode_variant(variant)
        lse = torch.full((self.spec.batch, self.spec.n_q_heads), 123.0, dtype=torch.float32, device="cuda:0") if want_lse else None
        out = self.pool.decode_attention(self.q, self.bt, self.tags, self.lens, self.spec.scale, lse=lse)
        torch.cuda.synchronize()
        assert self.pool.status() == M.OK
        return out.cpu().numpy(), (lse.cpu().numpy() if want_lse else None)

    def reference(self, only_b=-1, only_h=-1):
        s = self.spec
        assert oracle.get_format() == self.fmt
        return oracle.decode_attention(self.L.fp8_arena, self.L.tq3_arena, s.head_dim, s.n_kv_heads, s.group,
                                       self.L.sigma, self.L.q_bits, self.tab.block_table, self.tab.tier_tag,
                                       self.tab.seq_lens, s.scale, only_b=only_b, only_h=only_h,
                                       page_tokens=s.page_tokens)


def check_close(got, ref, what=""):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    assert np.isfinite(got).all(), what
    max_abs = np.abs(got - ref).max()
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    assert max_abs <= MAX_ABS and rel <= REL_L2, f"{what}: max-abs {max_abs:.3e} rel-L2 {rel:.3e}"
    return max_abs, rel


def check_case(case, out, lse, ref, ref_lse):
    """Whole output, plus the worst (request, head) row."""
    check_close(out, ref, case.spec.name)
    for b in range(case.spec.batch):
        if case.spec.seq_lens[b] == 0:
            assert not out[b].any() and np.all(np.isneginf(lse[b]))
            continue
        for h in range(case.spec.n_q_heads):
            check_close(out[b, h], ref[b, h], f"{case.spec.name} b={b} h={h}")
        if lse is not None:
            assert np.abs(lse[b] - ref_lse[b]).max() < 2e-3, (b, lse[b], ref_lse[b])
