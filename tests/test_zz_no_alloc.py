"""mkv_decode_attention_static: the decode entry point for callers that must not allocate device
memory (its split partials live in a fixed array inside the library instead of a caller workspace).

Collected last on purpose: a run that stops at the first failure has then already run every other
test.  Checks, through the C ABI, that two calls in a row give what mkv_decode_attention gives on
the same inputs, and that sizes beyond the documented maximum are refused."""
import numpy as np
import pytest
import torch

import mkv_workloads as W
import paper_2608_23834_b200 as M
from _gpu_util import Case, MAX_ABS, REL_L2, bf16_tensor

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg", ["d256", "d128", "d256_pages_of_832"])
def test_static_scratch_entry_matches_the_workspace_entry_twice_in_a_row(cfg):
    if cfg == "d256":
        spec = W.config(2, seq_lens=(9008, 7600), recent_tokens=512, n_layers=1)
    elif cfg == "d256_pages_of_832":
        spec = W.config(2, seq_lens=(9 * 832 + 100, 7 * 832), anchor_prefix=832, recent_tokens=900, n_layers=1,
                        page_tokens=832)
    else:
        spec = W.config(1, seq_lens=(3000, 1500, 4100, 16), recent_tokens=256, anchor_span_tokens=64)
    case = Case(spec, extra_fp8=3, extra_tq3=3)
    case.pool.set_decode_variant(M.DECODE_TENSOR)
    # set-up call: the first call on a device resolves the scratch array's address (the CUDA runtime may load the
    # library's image on that occasion); a caller makes it at start-up, before its memory budget is frozen
    M.decode_attention_static(case.pool, case.q, case.bt, case.tags, case.lens, spec.scale)
    torch.cuda.synchronize()
    for call in range(2):
        # a different query on the second call: the shared scratch still holds the first call's partials
        q = bf16_tensor(W.query(spec, layer=call))
        lse_ref = torch.empty((spec.batch, spec.n_q_heads), dtype=torch.float32, device="cuda:0")
        lse_got = torch.empty_like(lse_ref)
        ref = case.pool.decode_attention(q, case.bt, case.tags, case.lens, spec.scale, lse=lse_ref)
        out_got = torch.empty_like(ref)                 # the caller's output buffer exists before the call
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        torch_before = torch.cuda.memory_allocated()
        got = M.decode_attention_static(case.pool, q, case.bt, case.tags, case.lens, spec.scale, out=out_got, lse=lse_got)
        torch.cuda.synchronize()
        # the property in the entry point's name: the device has exactly as much free memory as before the call
        # (the first call on the device resolves the scratch array's address, which allocates nothing either)
        assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == torch_before
        assert got.data_ptr() == out_got.data_ptr()
        assert case.pool.status() == M.OK
        ref, got = ref.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert np.abs(got - ref).max() <= MAX_ABS
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= REL_L2
        assert np.abs(lse_got.cpu().numpy() - lse_ref.cpu().numpy()).max() <= 2e-3
    # and against the CPU oracle on the last query, like every other decode test
    import oracle
    s = spec
    ref64, _ = oracle.decode_attention(case.L.fp8_arena, case.L.tq3_arena, s.head_dim, s.n_kv_heads, s.group, case.L.sigma,
                                       W.query(spec, layer=1), case.tab.block_table, case.tab.tier_tag, case.tab.seq_lens,
                                       s.scale, page_tokens=s.page_tokens)
    assert np.abs(got - ref64).max() <= MAX_ABS and np.linalg.norm(got - ref64) / np.linalg.norm(ref64) <= REL_L2


def test_static_scratch_entry_refuses_sizes_beyond_its_maximum():
    spec = W.config(0, seq_lens=(64,))
    case = Case(spec)
    B = 1025                                   # MKV_STATIC_MAX_BATCH is 1024
    q = torch.zeros((B, spec.n_q_heads, spec.head_dim), dtype=torch.bfloat16, device="cuda:0")
    bt = torch.zeros((B, 4), dtype=torch.int32, device="cuda:0")
    tags = torch.zeros((B, 4), dtype=torch.uint8, device="cuda:0")
    lens = torch.zeros(B, dtype=torch.int32, device="cuda:0")
    with pytest.raises(M.MkvError) as e:
        M.decode_attention_static(case.pool, q, bt, tags, lens, spec.scale)
    assert e.value.code == M.E_INVALID
    assert b"MKV_STATIC_MAX_BATCH" in M.lib().mkv_last_cuda_error()
    # a refusal names its real cause: a table wider than the scan can index, or a pool set to another kernel
    wide_bt = torch.zeros((1, 65536), dtype=torch.int32, device="cuda:0")
    wide_tg = torch.zeros((1, 65536), dtype=torch.uint8, device="cuda:0")
    with pytest.raises(M.MkvError) as e:
        M.decode_attention_static(case.pool, case.q, wide_bt, wide_tg, case.lens, spec.scale)
    assert e.value.code == M.E_INVALID and b"65535" in M.lib().mkv_last_cuda_error()
    case.pool.set_decode_variant(M.DECODE_TMEM)
    with pytest.raises(M.MkvError) as e:
        M.decode_attention_static(case.pool, case.q, case.bt, case.tags, case.lens, spec.scale)
    assert e.value.code == M.E_INVALID and b"tensor-core kernel only" in M.lib().mkv_last_cuda_error()
