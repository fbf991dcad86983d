"""Seeded synthetic inputs for the mixed-format paged decode-attention path.

This module holds NO arithmetic of the method: it draws random numbers, rounds them to bf16 (a
storage-format conversion), lays out tier tags and block tables, and hands the same arrays to the
CPU oracle and to the CUDA library.  It imports neither of them.

The five workload shapes follow the benchmark configurations: K,V ~ N(0,1) rounded to bf16 with a
few channels scaled x8 as outliers, q ~ N(0,1) bf16, softmax scale 1/sqrt(d), 16-token pages, a
first-tokens Anchor span (attention sinks), optional random Anchor spans, a Recent window at the
end of the context (both FP8) and everything else Stale (TQ3); physical page ids are a random
permutation inside each arena.  They stand in for the paper's 2 x 59,008-token decode canary
(24 query / 4 KV heads, d = 256), whose model, runtime and prompts are not available.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional, Tuple

import numpy as np

T = 16
TAG_RECENT, TAG_ANCHOR, TAG_STALE = 0, 1, 2
GENERATOR = "numpy.random.Generator(PCG64), SeedSequence([seed, stream, a, b])"


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even (storage conversion only)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def _rng(seed: int, stream: int, a: int = 0, b: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, stream, a, b])))


@dataclass
class Spec:
    """Shape of one workload.  All token counts are tokens; spans are page-aligned."""
    name: str
    seed: int
    batch: int
    n_layers: int
    head_dim: int
    n_kv_heads: int
    group: int                      # query heads per KV head
    seq_lens: Tuple[int, ...]       # per request
    anchor_prefix: int              # first tokens kept Anchor
    anchor_spans: int               # fixed number of random Anchor spans per request (-1: draw 1..4)
    anchor_span_tokens: int
    recent_tokens: int              # Recent window at the end of the context
    n_outlier: int                  # channels scaled x8, drawn per layer and per tensor
    stale_fraction: Optional[float] = None   # lifecycle sweep: oldest floor(f*P) pages Stale, rest Recent
    page_tokens: int = T            # tokens per page: 16, or 16 M for the paper-scale blocks (1,792 / 832)

    @property
    def n_q_heads(self) -> int:
        return self.n_kv_heads * self.group

    @property
    def scale(self) -> float:
        return float(1.0 / np.sqrt(np.float64(self.head_dim)))

    def n_pages(self, b: int) -> int:
        return (self.seq_lens[b] + self.page_tokens - 1) // self.page_tokens

    @property
    def tiles_per_page(self) -> int:
        return self.page_tokens // T

    @property
    def max_pages(self) -> int:
        return max(self.n_pages(b) for b in range(self.batch))


def config(idx: int, **over) -> Spec:
    """The five benchmark configurations.  ``over`` replaces fields (tests use scaled-down
    contexts: e.g. ``config(2, seq_lens=(4000, 4000), n_layers=2)``); for config 4 pass
    ``batch``, ``ctx`` and ``stale_fraction`` to pick a cell."""
    if idx == 0:
        s = Spec("cfg0_tiny", 0, 1, 1, 128, 1, 8, (4096,), 64, 0, 0, 256, 4)
    elif idx == 1:
        s = Spec("cfg1_small_batch", 1, 8, 1, 128, 4, 8, (16384,) * 8, 128, 2, 256, 1024, 4)
    elif idx == 2:
        s = Spec("cfg2_canary_59k", 2, 2, 16, 256, 4, 6, (59008,) * 2, 256, 0, 0, 2048, 5)
    elif idx == 3:
        u = _rng(3, 0).random(64)
        lens = tuple(int(np.floor(1024.0 * 128.0 ** x)) for x in u)
        s = Spec("cfg3_ragged", 3, 64, 1, 128, 8, 4, lens, 64, -1, 128, 512, 4)
    elif idx == 4:
        batch = over.pop("batch", 8)
        ctx = over.pop("ctx", 32768)
        frac = over.pop("stale_fraction", 0.5)
        s = Spec(f"cfg4_lifecycle_b{batch}_c{ctx}_f{frac}", 4, batch, 1, 128, 8, 4, (ctx,) * batch,
                 0, 0, 0, 0, 3, stale_fraction=frac)
    elif idx == 5:
        # the canary's shape with pages of 1,792 tokens (the block size its byte counters were taken at):
        # 33 pages per request = 1 first-tokens Anchor + 3 Anchor spans + 6 Recent (FP8) + 23 Stale (TQ3)
        s = Spec("cfg5_canary_blocks_1792", 5, 2, 1, 256, 4, 6, (59008,) * 2, 1792, 3, 1792, 5 * 1792, 5,
                 page_tokens=1792)
    else:
        raise ValueError("config index 0..5")
    if "seq_lens" in over:
        over["seq_lens"] = tuple(int(x) for x in over["seq_lens"])
        over.setdefault("batch", len(over["seq_lens"]))
    return replace(s, **over) if over else s


CFG4_CELLS = [(b, c, f) for b in (1, 8, 32) for c in (4096, 32768, 131072) for f in (0.0, 0.5, 0.95)]


def tier_tags(spec: Spec, b: int) -> np.ndarray:
    """Tier tag (0 Recent, 1 Anchor, 2 Stale) of every logical page of request b."""
    n = spec.n_pages(b)
    ln = spec.seq_lens[b]
    Tp = spec.page_tokens
    tags = np.full(n, TAG_STALE, np.uint8)
    if spec.stale_fraction is not None:
        n_stale = int(np.floor(spec.stale_fraction * n))
        tags[n_stale:] = TAG_RECENT
    else:
        rng = _rng(spec.seed, 1, b)
        n_anchor = min(n, spec.anchor_prefix // Tp)
        tags[:n_anchor] = TAG_ANCHOR
        first_recent = max(0, ln - spec.recent_tokens) // Tp   # pages covering the last tokens
        tags[first_recent:] = TAG_RECENT
        n_spans = spec.anchor_spans if spec.anchor_spans >= 0 else int(rng.integers(1, 5))
        span = spec.anchor_span_tokens // Tp
        placed, tries = 0, 0
        while placed < n_spans and span > 0 and tries < 1000:
            tries += 1
            if first_recent - span <= n_anchor:
                break
            start = int(rng.integers(n_anchor, first_recent - span + 1))
            if np.all(tags[start:start + span] == TAG_STALE):      # re-draw on collision
                tags[start:start + span] = TAG_ANCHOR
                placed += 1
    if ln % Tp != 0 and n and tags[-1] == TAG_STALE:
        tags[-1] = TAG_RECENT        # a partial (still open) page is never Stale
    return tags


@dataclass
class Tables:
    block_table: np.ndarray      # int32 [B][max_pages], -1 = unused
    tier_tag: np.ndarray         # uint8 [B][max_pages]
    seq_lens: np.ndarray         # int32 [B]
    fp8_pages: int               # pages used in the FP8 arena
    tq3_pages: int               # pages used in the TQ3 arena


def tables(spec: Spec, extra_fp8: int = 0, extra_tq3: int = 0) -> Tables:
    """Block table with physical ids drawn as a random permutation inside each arena (pages of all
    requests interleaved in one shared pool)."""
    B, mp = spec.batch, spec.max_pages
    tag = np.zeros((B, mp), np.uint8)
    for b in range(B):
        tag[b, :spec.n_pages(b)] = tier_tags(spec, b)
    used = np.zeros((B, mp), bool)
    for b in range(B):
        used[b, :spec.n_pages(b)] = True
    is_tq3 = used & (tag == TAG_STALE)
    is_fp8 = used & ~is_tq3
    n_fp8, n_tq3 = int(is_fp8.sum()), int(is_tq3.sum())
    rng = _rng(spec.seed, 2)
    bt = np.full((B, mp), -1, np.int32)
    bt[is_fp8] = rng.permutation(n_fp8 + extra_fp8)[:n_fp8].astype(np.int32)
    bt[is_tq3] = rng.permutation(n_tq3 + extra_tq3)[:n_tq3].astype(np.int32)
    return Tables(bt, tag, np.array(spec.seq_lens, np.int32), n_fp8 + extra_fp8, n_tq3 + extra_tq3)


def rotation_signs(spec: Spec, layer: int = 0) -> np.ndarray:
    """The +-1 diagonal of the randomised Hadamard rotation of one layer's pool (int8 [d])."""
    return (_rng(spec.seed, 3, layer).integers(0, 2, spec.head_dim) * 2 - 1).astype(np.int8)


def outlier_channels(spec: Spec, layer: int, tensor: int) -> np.ndarray:
    return np.sort(_rng(spec.seed, 4, layer, tensor).permutation(spec.head_dim)[:spec.n_outlier])


def kv(spec: Spec, layer: int, b: int) -> Tuple[np.ndarray, np.ndarray]:
    """bf16 bit patterns of K and V of request b in one layer: uint16 [len][n_kv_heads][d]."""
    ln = spec.seq_lens[b]
    out = []
    for tensor in (0, 1):
        x = _rng(spec.seed, 5 + tensor, layer, b).standard_normal((ln, spec.n_kv_heads, spec.head_dim),
                                                                   dtype=np.float32)
        x[:, :, outlier_channels(spec, layer, tensor)] *= np.float32(8.0)
        out.append(f32_to_bf16_bits(x))
    return out[0], out[1]


def query(spec: Spec, layer: int = 0) -> np.ndarray:
    """bf16 bit patterns of the decode-step queries: uint16 [B][Hq][d]."""
    x = _rng(spec.seed, 7, layer).standard_normal((spec.batch, spec.n_q_heads, spec.head_dim), dtype=np.float32)
    return f32_to_bf16_bits(x)


def new_token_kv(spec: Spec, layer: int, step: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """K,V of one appended token per request (lifecycle sweep): uint16 [B][n_kv_heads][d] each."""
    out = []
    for tensor in (0, 1):
        x = _rng(spec.seed, 8 + tensor, layer, step).standard_normal(
            (spec.batch, spec.n_kv_heads, spec.head_dim), dtype=np.float32)
        x[:, :, outlier_channels(spec, layer, tensor)] *= np.float32(8.0)
        out.append(f32_to_bf16_bits(x))
    return out[0], out[1]


def kv_bytes(spec: Spec, tab: Tables) -> int:
    """Algorithmic KV bytes one decode step of ONE layer must read: 2*d bytes per valid FP8 token and
    M (12 d + 32) + 4 d bytes per Stale page of 16 M tokens (16 d + 32 at M = 1), per KV head (queries,
    outputs, tables and workspace excluded)."""
    d, total, M = spec.head_dim, 0, spec.tiles_per_page
    for b in range(spec.batch):
        n = spec.n_pages(b)
        stale = int((tab.tier_tag[b, :n] == TAG_STALE).sum())
        fp8_tokens = spec.seq_lens[b] - stale * spec.page_tokens
        total += spec.n_kv_heads * (fp8_tokens * 2 * d + stale * (M * (12 * d + 32) + 4 * d))
    return total
