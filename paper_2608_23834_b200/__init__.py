"""Python binding of libmkv: mixed-format (FP8 + TQ3) paged KV cache and decode attention on B200.

Argument marshalling only: every step of the path (append, demote, tag flips, decode attention
with its split merge) runs in the CUDA kernels of ``libmkv.so``.  PyTorch supplies device memory
and streams.  There is no CPU or PyTorch fallback: if the library is missing, or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmkv.so")
_lib = None

OK, E_INVALID, E_OOM_FP8, E_OOM_TQ3, E_STATE, E_BOUNDS, E_CUDA, E_TIMEOUT = 0, -1, -2, -3, -4, -5, -6, -7
TAG_RECENT, TAG_ANCHOR, TAG_STALE = 0, 1, 2
FMT_FP8, FMT_TQ3 = 0, 1
DECODE_TENSOR, DECODE_SCALAR, DECODE_TMEM = 0, 1, 2
_NAMES = {0: "MKV_OK", -1: "MKV_E_INVALID", -2: "MKV_E_OOM_FP8", -3: "MKV_E_OOM_TQ3", -4: "MKV_E_STATE",
          -5: "MKV_E_BOUNDS", -6: "MKV_E_CUDA", -7: "MKV_E_TIMEOUT"}

EXPORTS = [
    "mkv_pool_query", "mkv_decode_workspace_bytes", "mkv_workspace_init", "mkv_pool_create", "mkv_pool_create_host_only",
    "mkv_pool_destroy",
    "mkv_page_alloc", "mkv_page_free", "mkv_pool_stats", "mkv_pool_status", "mkv_pool_set_decode_variant",
    "mkv_page_read_raw", "mkv_page_write_raw", "mkv_last_cuda_error", "mkv_append", "mkv_demote",
    "mkv_set_anchor", "mkv_decode_attention", "mkv_seq_create", "mkv_seq_finish", "mkv_seq_append",
    "mkv_seq_protect", "mkv_seq_demote", "mkv_seq_age", "mkv_seq_len", "mkv_seq_row",
    "mkv_decode_attention_static", "mkv_promote", "mkv_seq_promote",
    "mkv_decode_attention_scored", "mkv_page_score_update", "mkv_page_score_update_paged",
    "mkv_decode_attention_layers", "mkv_append_layers", "mkv_pool_set_wait_limit_ns", "mkv_seq_release",
]
MAX_LAYERS_PER_CALL = 32


class MkvError(RuntimeError):
    def __init__(self, code: int, where: str):
        detail = ""
        if code == E_CUDA and _lib is not None:
            detail = ": " + _lib.mkv_last_cuda_error().decode()
        super().__init__(f"{where} -> {_NAMES.get(code, code)}{detail}")
        self.code = code


class PoolConfig(C.Structure):
    _fields_ = [("page_size", C.c_int32), ("head_dim", C.c_int32), ("n_kv_heads", C.c_int32),
                ("n_q_heads", C.c_int32), ("fp8_pages", C.c_int32), ("tq3_pages", C.c_int32),
                ("k_scale", C.c_float), ("v_scale", C.c_float), ("k_rot_signs", C.POINTER(C.c_int8)),
                ("tq3_format", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("fp8_pages_total", "fp8_pages_used", "tq3_pages_total", "tq3_pages_used",
                                         "fp8_bytes_used", "tq3_bytes_used", "bf16_bytes_equivalent")]


class LayerCall(C.Structure):
    _fields_ = [("pool", C.c_void_p), ("q_dev", C.c_void_p), ("block_table_dev", C.c_void_p), ("tier_tag_dev", C.c_void_p),
                ("out_dev", C.c_void_p), ("lse_dev", C.c_void_p), ("workspace_dev", C.c_void_p)]


class LayerAppend(C.Structure):
    _fields_ = [("pool", C.c_void_p), ("k_dev", C.c_void_p), ("v_dev", C.c_void_p)]


def lib():
    """Load libmkv.so; fails loudly if it has not been built (python paper_2608_23834_b200/build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2608_23834_b200.build` "
                              "(there is no fallback path)")
        L = C.CDLL(_LIB_PATH)
        vp, i32p, u8p, i64p, f32p = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_uint8), C.POINTER(C.c_int64), C.c_void_p
        cfgp, szp = C.POINTER(PoolConfig), C.POINTER(C.c_size_t)
        sig = {
            "mkv_pool_query": [cfgp, szp, szp],
            "mkv_decode_workspace_bytes": [cfgp, C.c_int32, szp],
            "mkv_workspace_init": [vp, C.c_size_t, vp],
            "mkv_pool_create": [cfgp, vp, vp, vp, C.POINTER(vp)],
            "mkv_pool_create_host_only": [cfgp, C.POINTER(vp)],
            "mkv_pool_destroy": [vp],
            "mkv_page_alloc": [vp, C.c_int32, i32p, C.c_int32],
            "mkv_page_free": [vp, C.c_int32, i32p, C.c_int32],
            "mkv_pool_stats": [vp, C.POINTER(Stats)],
            "mkv_pool_status": [vp, vp],
            "mkv_pool_set_decode_variant": [vp, C.c_int32],
            "mkv_page_read_raw": [vp, C.c_int32, C.c_int32, vp, vp],
            "mkv_page_write_raw": [vp, C.c_int32, C.c_int32, vp, vp],
            "mkv_append": [vp, vp, vp, vp, C.c_int32, vp],
            "mkv_demote": [vp, vp, vp, C.c_int32, vp, vp, vp, C.c_int64, vp],
            "mkv_promote": [vp, vp, vp, C.c_int32, vp, vp, vp, C.c_int64, vp],
            "mkv_seq_promote": [vp, C.c_int32, i32p, i32p],
            "mkv_set_anchor": [vp, vp, C.c_int64, C.c_int64, C.c_int32, vp],
            "mkv_decode_attention": [vp, vp, vp, vp, vp, C.c_int32, C.c_int32, C.c_float, f32p, f32p, vp,
                                     C.c_size_t, vp],
            "mkv_decode_attention_static": [vp, vp, vp, vp, vp, C.c_int32, C.c_int32, C.c_float, f32p, f32p, vp],
            "mkv_decode_attention_scored": [vp, vp, vp, vp, vp, C.c_int32, C.c_int32, C.c_float, f32p, f32p, f32p, vp,
                                            C.c_size_t, vp],
            "mkv_page_score_update": [f32p, vp, C.c_int32, C.c_int32, C.c_int32, C.c_uint64, C.c_float, f32p, vp],
            "mkv_page_score_update_paged": [f32p, vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_uint64, C.c_float,
                                            f32p, vp],
            "mkv_decode_attention_layers": [C.POINTER(LayerCall), C.c_int32, vp, C.c_int32, C.c_int32, C.c_float,
                                            C.c_size_t, vp],
            "mkv_append_layers": [C.POINTER(LayerAppend), C.c_int32, vp, C.c_int32, vp],
            "mkv_pool_set_wait_limit_ns": [vp, C.c_uint64],
            "mkv_seq_create": [vp, C.POINTER(vp)],
            "mkv_seq_finish": [vp],
            "mkv_seq_append": [vp, i32p, i32p, i32p],
            "mkv_seq_protect": [vp, C.c_int32, C.c_int32],
            "mkv_seq_demote": [vp, C.c_int32, i32p, i32p],
            "mkv_seq_age": [vp, C.c_int32, i32p, i32p, i32p, C.c_int32, i32p],
            "mkv_seq_release": [vp, C.c_int32, C.c_int32],
            "mkv_seq_len": [vp, i32p, i32p],
            "mkv_seq_row": [vp, i32p, u8p, C.c_int32],
        }
        for name, args in sig.items():
            fn = getattr(L, name)
            fn.argtypes = args
            fn.restype = C.c_int32
        L.mkv_last_cuda_error.restype = C.c_char_p
        L.mkv_last_cuda_error.argtypes = []
        _lib = L
    return _lib


def _check(rc: int, where: str):
    if rc != OK:
        raise MkvError(rc, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def make_config(head_dim, n_kv_heads, n_q_heads, fp8_pages, tq3_pages, sigma: np.ndarray, k_scale=1.0, v_scale=1.0,
                page_tokens=16, tq3_format=1):
    sig = np.ascontiguousarray(sigma, dtype=np.int8)
    cfg = PoolConfig(page_tokens, head_dim, n_kv_heads, n_q_heads, fp8_pages, tq3_pages, k_scale, v_scale,
                     sig.ctypes.data_as(C.POINTER(C.c_int8)), tq3_format)
    cfg._keepalive = sig
    return cfg


# ------------------------------------------------------------------------------- same-name calls
def mkv_pool_query(cfg: PoolConfig):
    a, b = C.c_size_t(), C.c_size_t()
    _check(lib().mkv_pool_query(C.byref(cfg), C.byref(a), C.byref(b)), "mkv_pool_query")
    return a.value, b.value


def mkv_decode_workspace_bytes(cfg: PoolConfig, max_batch: int) -> int:
    n = C.c_size_t()
    _check(lib().mkv_decode_workspace_bytes(C.byref(cfg), max_batch, C.byref(n)), "mkv_decode_workspace_bytes")
    return n.value


class Pool:
    """One layer's page pool.  Owns the torch buffers handed to the library (arenas, workspace)."""

    def __init__(self, head_dim, n_kv_heads, n_q_heads, fp8_pages, tq3_pages, sigma, k_scale=1.0, v_scale=1.0,
                 max_batch=64, device="cuda:0", page_tokens=16, tq3_format=1):
        L = lib()
        self.tq3_format = tq3_format
        self.device = torch.device(device)
        self.d, self.hkv, self.hq = head_dim, n_kv_heads, n_q_heads
        self.group = n_q_heads // n_kv_heads
        self.cfg = make_config(head_dim, n_kv_heads, n_q_heads, fp8_pages, tq3_pages, sigma, k_scale, v_scale, page_tokens,
                               tq3_format)
        fp8_bytes, tq3_bytes = mkv_pool_query(self.cfg)
        # bytes of one page and KV head: a page is page_tokens / 16 tiles (16 d + 32 bytes of TQ3 at one tile)
        self.page_tokens, self.tiles = page_tokens, page_tokens // 16
        self.fp8_rec = self.tiles * 32 * head_dim
        self.tq3_rec = self.tiles * (12 * head_dim + 32) + 4 * head_dim
        with torch.cuda.device(self.device):
            self.fp8_arena = torch.empty(fp8_bytes, dtype=torch.uint8, device=self.device)
            self.tq3_arena = torch.empty(tq3_bytes, dtype=torch.uint8, device=self.device)
            self.max_batch = max_batch
            self.ws_bytes = mkv_decode_workspace_bytes(self.cfg, max_batch)
            self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=self.device)
            h = C.c_void_p()
            _check(L.mkv_pool_create(C.byref(self.cfg), _ptr(self.fp8_arena), _ptr(self.tq3_arena), _stream(None),
                                     C.byref(h)), "mkv_pool_create")
            self.handle = h
            _check(L.mkv_workspace_init(_ptr(self.workspace), self.ws_bytes, _stream(None)), "mkv_workspace_init")

    def close(self):
        if getattr(self, "handle", None):
            lib().mkv_pool_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- bookkeeping
    def page_alloc(self, fmt: int, n: int) -> np.ndarray:
        ids = np.zeros(n, np.int32)
        _check(lib().mkv_page_alloc(self.handle, fmt, ids.ctypes.data_as(C.POINTER(C.c_int32)), n), "mkv_page_alloc")
        return ids

    def page_free(self, fmt: int, ids) -> None:
        ids = np.ascontiguousarray(ids, np.int32)
        _check(lib().mkv_page_free(self.handle, fmt, ids.ctypes.data_as(C.POINTER(C.c_int32)), len(ids)), "mkv_page_free")

    def stats(self) -> Stats:
        s = Stats()
        _check(lib().mkv_pool_stats(self.handle, C.byref(s)), "mkv_pool_stats")
        return s

    def status(self) -> int:
        """Device status word as an mkv_status code (0 when clean); clears it."""
        return lib().mkv_pool_status(self.handle, _stream(None))

    def set_decode_variant(self, variant: int) -> None:
        _check(lib().mkv_pool_set_decode_variant(self.handle, variant), "mkv_pool_set_decode_variant")

    def set_wait_limit_ns(self, ns: int) -> None:
        _check(lib().mkv_pool_set_wait_limit_ns(self.handle, int(ns)), "mkv_pool_set_wait_limit_ns")

    def page_read_raw(self, fmt: int, pid: int) -> np.ndarray:
        buf = np.zeros(self.hkv * (self.fp8_rec if fmt == FMT_FP8 else self.tq3_rec), np.uint8)
        _check(lib().mkv_page_read_raw(self.handle, fmt, pid, C.c_void_p(buf.ctypes.data), _stream(None)), "mkv_page_read_raw")
        return buf

    def page_write_raw(self, fmt: int, pid: int, data: np.ndarray) -> None:
        data = np.ascontiguousarray(data, np.uint8).reshape(-1)
        assert data.size == self.hkv * (self.fp8_rec if fmt == FMT_FP8 else self.tq3_rec)
        _check(lib().mkv_page_write_raw(self.handle, fmt, pid, C.c_void_p(data.ctypes.data), _stream(None)), "mkv_page_write_raw")

    def upload_arenas(self, fp8: np.ndarray, tq3: np.ndarray) -> None:
        """Install whole arenas encoded elsewhere (test hook; one copy per arena)."""
        f = torch.from_numpy(np.ascontiguousarray(fp8, np.uint8).reshape(-1))
        t = torch.from_numpy(np.ascontiguousarray(tq3, np.uint8).reshape(-1))
        assert f.numel() <= self.fp8_arena.numel() - 256 and t.numel() <= self.tq3_arena.numel()
        self.fp8_arena[:f.numel()].copy_(f)
        self.tq3_arena[:t.numel()].copy_(t)
        torch.cuda.synchronize(self.device)

    # ---- hot path
    def append(self, k: torch.Tensor, v: torch.Tensor, slot_mapping: torch.Tensor, stream=None) -> None:
        assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and slot_mapping.dtype == torch.int32
        assert k.is_contiguous() and v.is_contiguous() and k.shape == v.shape and k.shape[1:] == (self.hkv, self.d)
        _check(lib().mkv_append(self.handle, _ptr(k), _ptr(v), _ptr(slot_mapping), k.shape[0], _stream(stream)), "mkv_append")

    def demote(self, src_ids: torch.Tensor, dst_ids: torch.Tensor, block_table=None, tier_tag=None, entry_index=None,
               stream=None) -> None:
        assert src_ids.dtype == torch.int32 and dst_ids.dtype == torch.int32 and src_ids.numel() == dst_ids.numel()
        if entry_index is not None:
            assert entry_index.dtype == torch.int64 and block_table.dtype == torch.int32 and tier_tag.dtype == torch.uint8
        _check(lib().mkv_demote(self.handle, _ptr(src_ids), _ptr(dst_ids), src_ids.numel(), _ptr(block_table),
                                _ptr(tier_tag), _ptr(entry_index), 0 if tier_tag is None else tier_tag.numel(),
                                _stream(stream)), "mkv_demote")

    def promote(self, src_ids: torch.Tensor, dst_ids: torch.Tensor, block_table=None, tier_tag=None, entry_index=None,
                stream=None) -> None:
        assert src_ids.dtype == torch.int32 and dst_ids.dtype == torch.int32 and src_ids.numel() == dst_ids.numel()
        if entry_index is not None:
            assert entry_index.dtype == torch.int64 and block_table.dtype == torch.int32 and tier_tag.dtype == torch.uint8
        _check(lib().mkv_promote(self.handle, _ptr(src_ids), _ptr(dst_ids), src_ids.numel(), _ptr(block_table),
                                 _ptr(tier_tag), _ptr(entry_index), 0 if tier_tag is None else tier_tag.numel(),
                                 _stream(stream)), "mkv_promote")

    def set_anchor(self, tier_tag: torch.Tensor, entry_index: int, flag: bool, stream=None) -> None:
        _check(lib().mkv_set_anchor(self.handle, _ptr(tier_tag), tier_tag.numel(), int(entry_index), int(bool(flag)),
                                    _stream(stream)), "mkv_set_anchor")

    def decode_attention(self, q, block_table, tier_tag, seq_lens, scale, out=None, lse=None, workspace=None, stream=None):
        B = q.shape[0]
        assert q.dtype == torch.bfloat16 and q.is_contiguous() and q.shape == (B, self.hq, self.d)
        assert block_table.dtype == torch.int32 and block_table.is_contiguous() and block_table.shape[0] == B
        assert tier_tag.dtype == torch.uint8 and tier_tag.shape == block_table.shape and tier_tag.is_contiguous()
        assert seq_lens.dtype == torch.int32 and seq_lens.numel() == B
        if out is None:
            out = torch.empty((B, self.hq, self.d), dtype=torch.float32, device=q.device)
        ws = self.workspace if workspace is None else workspace
        _check(lib().mkv_decode_attention(self.handle, _ptr(q), _ptr(block_table), _ptr(tier_tag), _ptr(seq_lens), B,
                                          block_table.shape[1], float(scale), _ptr(out), _ptr(lse), _ptr(ws),
                                          ws.numel(), _stream(stream)), "mkv_decode_attention")
        return out

    def decode_attention_scored(self, q, block_table, tier_tag, seq_lens, scale, out=None, lse=None, page_mass=None,
                                workspace=None, stream=None):
        """mkv_decode_attention_scored: returns (out, lse, page_mass [B][hq][max_pages])."""
        B = q.shape[0]
        assert q.dtype == torch.bfloat16 and q.is_contiguous() and q.shape == (B, self.hq, self.d)
        assert block_table.dtype == torch.int32 and block_table.is_contiguous() and block_table.shape[0] == B
        assert tier_tag.dtype == torch.uint8 and tier_tag.shape == block_table.shape and tier_tag.is_contiguous()
        assert seq_lens.dtype == torch.int32 and seq_lens.numel() == B
        if out is None:
            out = torch.empty((B, self.hq, self.d), dtype=torch.float32, device=q.device)
        if lse is None:
            lse = torch.empty((B, self.hq), dtype=torch.float32, device=q.device)
        if page_mass is None:
            page_mass = torch.empty((B, self.hq, block_table.shape[1]), dtype=torch.float32, device=q.device)
        ws = self.workspace if workspace is None else workspace
        _check(lib().mkv_decode_attention_scored(self.handle, _ptr(q), _ptr(block_table), _ptr(tier_tag), _ptr(seq_lens),
                                                 B, block_table.shape[1], float(scale), _ptr(out), _ptr(lse),
                                                 _ptr(page_mass), _ptr(ws), ws.numel(), _stream(stream)),
               "mkv_decode_attention_scored")
        return out, lse, page_mass


def decode_attention_layers(pools, qs, block_tables, tier_tags, seq_lens, scale, outs, lses=None, stream=None):
    """mkv_decode_attention_layers: the decode attention of len(pools) layers in one launch; layer i reads
    pools[i], qs[i], block_tables[i], tier_tags[i] and writes outs[i] (and lses[i]); seq_lens is common."""
    n = len(pools)
    B = qs[0].shape[0]
    calls = (LayerCall * n)()
    for i, pool in enumerate(pools):
        q, bt, tg, out = qs[i], block_tables[i], tier_tags[i], outs[i]
        assert q.dtype == torch.bfloat16 and q.is_contiguous() and q.shape == (B, pool.hq, pool.d)
        assert bt.dtype == torch.int32 and bt.is_contiguous() and bt.shape == block_tables[0].shape and bt.shape[0] == B
        assert tg.dtype == torch.uint8 and tg.is_contiguous() and tg.shape == bt.shape
        assert out.dtype == torch.float32 and out.is_contiguous() and out.shape == (B, pool.hq, pool.d)
        lse = None if lses is None else lses[i]
        calls[i] = LayerCall(pool.handle, q.data_ptr(), bt.data_ptr(), tg.data_ptr(), out.data_ptr(),
                             None if lse is None else lse.data_ptr(), pool.workspace.data_ptr())
    assert seq_lens.dtype == torch.int32 and seq_lens.numel() == B
    _check(lib().mkv_decode_attention_layers(calls, n, _ptr(seq_lens), B, block_tables[0].shape[1], float(scale),
                                             pools[0].ws_bytes, _stream(stream)), "mkv_decode_attention_layers")
    return outs


def append_layers(pools, ks, vs, slot_mapping, stream=None):
    """mkv_append_layers: Append of the same token positions into the pools of several layers in one launch."""
    n = len(pools)
    calls = (LayerAppend * n)()
    for i, pool in enumerate(pools):
        k, v = ks[i], vs[i]
        assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.is_contiguous() and v.is_contiguous()
        assert k.shape == v.shape and k.shape[1:] == (pool.hkv, pool.d) and k.shape[0] == slot_mapping.numel()
        calls[i] = LayerAppend(pool.handle, k.data_ptr(), v.data_ptr())
    assert slot_mapping.dtype == torch.int32
    _check(lib().mkv_append_layers(calls, n, _ptr(slot_mapping), slot_mapping.numel(), _stream(stream)), "mkv_append_layers")


def page_score_update(page_mass, seq_lens, head_mask, beta, score, stream=None, page_tokens=16):
    """mkv_page_score_update[_paged] (Eq. attention-score): score <- beta * score + (1 - beta) * mean over the
    heads in head_mask of page_mass, in place, for the pages below each request's length."""
    B, hq, max_pages = page_mass.shape
    assert page_mass.dtype == torch.float32 and page_mass.is_contiguous()
    assert score.dtype == torch.float32 and score.is_contiguous() and score.shape == (B, max_pages)
    assert seq_lens.dtype == torch.int32 and seq_lens.numel() == B
    if page_tokens == 16:
        _check(lib().mkv_page_score_update(_ptr(page_mass), _ptr(seq_lens), B, hq, max_pages, C.c_uint64(int(head_mask)),
                                           float(beta), _ptr(score), _stream(stream)), "mkv_page_score_update")
    else:
        _check(lib().mkv_page_score_update_paged(_ptr(page_mass), _ptr(seq_lens), B, hq, max_pages, int(page_tokens),
                                                 C.c_uint64(int(head_mask)), float(beta), _ptr(score), _stream(stream)),
               "mkv_page_score_update_paged")
    return score


def decode_attention_static(pool: "Pool", q, block_table, tier_tag, seq_lens, scale, out=None, lse=None, stream=None):
    """mkv_decode_attention_static: decode attention whose scratch is a fixed array inside the library,
    for callers that must not allocate device memory (the output tensor is the caller's, as always)."""
    B = q.shape[0]
    assert q.dtype == torch.bfloat16 and q.is_contiguous() and q.shape == (B, pool.hq, pool.d)
    assert block_table.dtype == torch.int32 and block_table.is_contiguous() and block_table.shape[0] == B
    assert tier_tag.dtype == torch.uint8 and tier_tag.shape == block_table.shape and tier_tag.is_contiguous()
    assert seq_lens.dtype == torch.int32 and seq_lens.numel() == B
    if out is None:
        out = torch.empty((B, pool.hq, pool.d), dtype=torch.float32, device=q.device)
    _check(lib().mkv_decode_attention_static(pool.handle, _ptr(q), _ptr(block_table), _ptr(tier_tag), _ptr(seq_lens),
                                             B, block_table.shape[1], float(scale), _ptr(out), _ptr(lse),
                                             _stream(stream)), "mkv_decode_attention_static")
    return out


class HostPool:
    """Bookkeeping-only pool (no device): free lists, sequence rows, statistics."""

    def __init__(self, head_dim, n_kv_heads, n_q_heads, fp8_pages, tq3_pages, page_tokens=16):
        self.d, self.hkv, self.hq = head_dim, n_kv_heads, n_q_heads
        self.cfg = make_config(head_dim, n_kv_heads, n_q_heads, fp8_pages, tq3_pages, np.ones(head_dim, np.int8),
                               page_tokens=page_tokens)
        h = C.c_void_p()
        _check(lib().mkv_pool_create_host_only(C.byref(self.cfg), C.byref(h)), "mkv_pool_create_host_only")
        self.handle = h

    page_alloc = Pool.page_alloc
    page_free = Pool.page_free
    stats = Pool.stats

    def close(self):
        if self.handle:
            lib().mkv_pool_destroy(self.handle)
            self.handle = None


class Seq:
    """Host bookkeeping of one request's row (Algorithm 1 transitions; plans only, no device work)."""

    def __init__(self, pool: Pool):
        self.pool = pool
        h = C.c_void_p()
        _check(lib().mkv_seq_create(pool.handle, C.byref(h)), "mkv_seq_create")
        self.handle = h

    def append(self):
        a, b, c = C.c_int32(), C.c_int32(), C.c_int32()
        _check(lib().mkv_seq_append(self.handle, C.byref(a), C.byref(b), C.byref(c)), "mkv_seq_append")
        return a.value, b.value, bool(c.value)

    def protect(self, lp: int, flag: bool = True):
        _check(lib().mkv_seq_protect(self.handle, lp, int(flag)), "mkv_seq_protect")

    def demote(self, lp: int):
        a, b = C.c_int32(), C.c_int32()
        _check(lib().mkv_seq_demote(self.handle, lp, C.byref(a), C.byref(b)), "mkv_seq_demote")
        return a.value, b.value

    def promote(self, lp: int):
        a, b = C.c_int32(), C.c_int32()
        _check(lib().mkv_seq_promote(self.handle, lp, C.byref(a), C.byref(b)), "mkv_seq_promote")
        return a.value, b.value

    def release(self, fmt: int, pid: int):
        """mkv_seq_release: the stream point of a planned conversion has passed; its source may be reused."""
        _check(lib().mkv_seq_release(self.handle, int(fmt), int(pid)), "mkv_seq_release")

    def age(self, recent_tokens: int):
        _, n_pages = self.len()
        lp, s, d = (np.zeros(max(n_pages, 1), np.int32) for _ in range(3))
        n = C.c_int32()
        p = lambda a: a.ctypes.data_as(C.POINTER(C.c_int32))
        _check(lib().mkv_seq_age(self.handle, recent_tokens, p(lp), p(s), p(d), n_pages, C.byref(n)), "mkv_seq_age")
        return [(int(lp[i]), int(s[i]), int(d[i])) for i in range(n.value)]

    def len(self):
        a, b = C.c_int32(), C.c_int32()
        _check(lib().mkv_seq_len(self.handle, C.byref(a), C.byref(b)), "mkv_seq_len")
        return a.value, b.value

    def row(self):
        _, n = self.len()
        ids, tags = np.zeros(max(n, 1), np.int32), np.zeros(max(n, 1), np.uint8)
        _check(lib().mkv_seq_row(self.handle, ids.ctypes.data_as(C.POINTER(C.c_int32)),
                                 tags.ctypes.data_as(C.POINTER(C.c_uint8)), n), "mkv_seq_row")
        return ids[:n], tags[:n]

    def finish(self):
        if self.handle:
            _check(lib().mkv_seq_finish(self.handle), "mkv_seq_finish")
            self.handle = None
