"""Builds the page arenas of a synthetic workload with the oracle's codecs -- TEST INFRASTRUCTURE.

Recent/Anchor pages are bf16 -> e4m3 and Stale pages are TQ3-encoded from the bf16 originals, both
by the C oracle; the resulting byte arrays are what tests upload to the CUDA pool, so that the
oracle and the CUDA path attend over identical quantised pages."""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

import mkv_workloads as W

from . import encode_request, fp8_block_bytes, tq3_block_bytes


@dataclass
class LayerArrays:
    fp8_arena: np.ndarray     # uint8 [fp8_pages][hkv][M * 32d]            (M = tiles of 16 tokens per page)
    tq3_arena: np.ndarray     # uint8 [tq3_pages][hkv][M * (12d + 32) + 4d]  (16d + 32 at M = 1)
    sigma: np.ndarray         # int8 [d]
    q_bits: np.ndarray        # uint16 [B][Hq][d]


def build_layer(spec: W.Spec, tab: W.Tables, layer: int = 0, requests=None) -> LayerArrays:
    d, hkv = spec.head_dim, spec.n_kv_heads
    M = spec.tiles_per_page
    fp8 = np.zeros((max(tab.fp8_pages, 1), hkv, fp8_block_bytes(d, M)), np.uint8)
    tq3 = np.zeros((max(tab.tq3_pages, 1), hkv, tq3_block_bytes(d, M)), np.uint8)
    sigma = W.rotation_signs(spec, layer)
    for b in (range(spec.batch) if requests is None else requests):
        k_bits, v_bits = W.kv(spec, layer, b)
        n = spec.n_pages(b)
        encode_request(k_bits, v_bits, tab.block_table[b, :n], tab.tier_tag[b, :n], sigma, fp8, tq3,
                       page_tokens=spec.page_tokens)
    return LayerArrays(fp8, tq3, sigma, W.query(spec, layer))
