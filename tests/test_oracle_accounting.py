"""Byte accounting against the numbers the paper prints (Eq. kv-per-token, Eq. effective-bits,
Section 6.3 counters, Table kv-memory)."""
import math

import oracle
from _util import read_golden

G = read_golden("paper_byte_counters.txt")
GIB = 1024.0 ** 3


def test_kv_bytes_per_token_closed_form():
    assert oracle.kv_bytes_per_token(16, 4, 256, 2) == G["kv_bytes_per_token_bf16"]
    assert oracle.kv_bytes_per_token(16, 4, 256, 1) == G["kv_bytes_per_token_fp8"]
    assert oracle.kv_bytes_per_token(16, 4, 256, 2) * 32768 / GIB == G["bf16_gib_per_32k"]
    assert oracle.kv_bytes_per_token(16, 4, 256, 2) * 131072 / GIB == G["bf16_gib_per_128k"]


def test_active_kv_byte_counters_reconcile_to_the_byte():
    """18 FP8 + 47 TQ3 blocks of 1,792 tokens x 4 KV heads x d = 256 give the compressed counter,
    65 BF16 blocks the full-cache counter, and their ratio the printed 3.6251x."""
    Tp, d, H = int(G["canary_page_tokens"]), int(G["canary_head_dim"]), int(G["canary_kv_heads"])
    fp8 = oracle.page_bytes_dense(Tp, d, H, 1)
    bf16 = oracle.page_bytes_dense(Tp, d, H, 2)
    tq3 = oracle.page_bytes_tq3(Tp, d, H)
    assert (fp8, bf16, tq3) == (3670016, 7340032, 1394688)
    assert 18 * fp8 + 47 * tq3 == G["active_kv_bytes_compressed"]
    assert 65 * bf16 == G["active_kv_bytes_full"]
    assert round(65 * bf16 / (18 * fp8 + 47 * tq3), 4) == G["physical_compression"]
    assert math.ceil(G["canary_prompt_tokens"] / Tp) == G["canary_block_entries_per_row"]


def test_tq3_rate_and_effective_bits():
    # realised TQ3 rate: 3 bits of codes + per-token norm + per-channel-per-page scale/zero
    assert abs(oracle.tq3_bits_per_scalar(1792, 256) - 3.0402) < 1e-4
    assert oracle.tq3_bits_per_scalar(16, 128) == 8 * (16 * 128 + 32) / (2 * 16 * 128) == 4.0625
    assert oracle.tq3_bits_per_scalar(16, 256) == 4.03125
    # the packed record holds exactly the accounted bytes
    for d in (128, 256):
        assert oracle.tq3_record_bytes(d) == oracle.page_bytes_tq3(16, d, 1)
        assert oracle.fp8_record_bytes(d) == oracle.page_bytes_dense(16, d, 1, 1)
    # Eq. (effective-bits) on the canary mix: 18 of 65 blocks FP8, 47 TQ3
    b = oracle.effective_bits(18 / 65, 0.0, 47 / 65, oracle.tq3_bits_per_scalar(1792, 256), 0.0)
    assert abs(16.0 / b - G["physical_compression"]) < 1e-4
    assert oracle.effective_bits(0.5, 0.5, 0.0, 3.0, 0.0) == 8.0
    assert oracle.effective_bits(0.0, 0.0, 1.0, 3.0, 0.25) == 3.25


def test_deployment_aggregate_and_memory_table():
    kib = G["deployment_kib_per_token"]
    bits = kib * 1024 * 8 / (G["kv_bytes_per_token_fp8"])          # scalars per token = 32,768
    assert abs(bits - 4.575) < 1e-9 and abs(bits - G["deployment_bits_per_scalar"]) < 0.006
    assert round(64.0 / kib, 3) == G["deployment_vs_bf16"] and round(32.0 / kib, 3) == G["deployment_vs_fp8"]
    for tokens, key, nd in ((8192, "table_kv_memory_8k_gib", 3), (32768, "table_kv_memory_32k_gib", 3),
                            (131072, "table_kv_memory_128k_gib", 3), (262144, "table_kv_memory_262144_gib", 3),
                            (1000000, "table_kv_memory_1m_gib", 2)):
        assert abs(tokens * kib * 1024 / GIB - G[key]) <= 0.5 * 10 ** -nd + 1e-9
    assert round(1000000 * oracle.kv_bytes_per_token(16, 4, 256, 1) / GIB, 2) == G["table_fp8_1m_gib"]
    assert round(1000000 * oracle.kv_bytes_per_token(16, 4, 256, 2) / GIB, 2) == G["table_bf16_1m_gib"]
