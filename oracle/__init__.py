"""CPU oracle for mixed-format (FP8 + TQ3) paged decode attention -- TEST INFRASTRUCTURE ONLY.

Thin ctypes binding over ``mkv_oracle.c`` (plain C, fp32 encoder / fp64 attention) plus the
page-lifecycle model in ``lifecycle.py``.  Only tests, the smoke check and the ``cpu_baseline``
/ ``--impl reference`` legs of the benchmark may import this package; the CUDA library and its
Python binding never do, and this package never imports them.

Section / equation names in the docstrings refer to the Minima-KV paper.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mkv_oracle.c")
_LIB = os.path.join(_HERE, "libmkv_oracle.so")
_lib = None

T = 16  # tokens per page

TAG_RECENT, TAG_ANCHOR, TAG_STALE = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no FMA contraction, OpenMP over units)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        u8p, u16p, i8p, i32p = (C.POINTER(C.c_uint8), C.POINTER(C.c_uint16), C.POINTER(C.c_int8),
                                C.POINTER(C.c_int32))
        f32p, f64p = C.POINTER(C.c_float), C.POINTER(C.c_double)
        L.orc_bf16_to_f32.restype = C.c_float
        L.orc_bf16_to_f32.argtypes = [C.c_uint16]
        L.orc_e4m3_decode.restype = C.c_double
        L.orc_e4m3_decode.argtypes = [C.c_uint8]
        L.orc_e4m3_encode.restype = C.c_uint8
        L.orc_e4m3_encode.argtypes = [C.c_float]
        L.orc_f32_to_f16_sat.restype = C.c_uint16
        L.orc_f32_to_f16_sat.argtypes = [C.c_float]
        L.orc_f16_to_f32.restype = C.c_float
        L.orc_f16_to_f32.argtypes = [C.c_uint16]
        L.orc_set_format.restype = C.c_int
        L.orc_set_format.argtypes = [C.c_int]
        L.orc_get_format.restype = C.c_int
        L.orc_get_format.argtypes = []
        L.orc_codebook_level.restype = C.c_float
        L.orc_codebook_level.argtypes = [C.c_int]
        L.orc_codebook_threshold.restype = C.c_float
        L.orc_codebook_threshold.argtypes = [C.c_int]
        L.orc_tq3_encode_key.restype = None
        L.orc_tq3_encode_key.argtypes = [f32p, C.c_int, i8p, u8p, u16p]
        L.orc_tq3_decode_key.restype = None
        L.orc_tq3_decode_key.argtypes = [u8p, C.c_uint16, C.c_int, i8p, f64p]
        L.orc_tq3_encode_value_page.restype = None
        L.orc_tq3_encode_value_page.argtypes = [f32p, C.c_int, u8p, u16p, u16p]
        L.orc_tq3_decode_value.restype = C.c_double
        L.orc_tq3_decode_value.argtypes = [C.c_uint8, C.c_uint16, C.c_uint16]
        L.orc_fp8_record_bytes.restype = C.c_int64
        L.orc_fp8_record_bytes.argtypes = [C.c_int]
        L.orc_tq3_record_bytes.restype = C.c_int64
        L.orc_tq3_record_bytes.argtypes = [C.c_int]
        L.orc_tq3_pack_record.restype = None
        L.orc_tq3_pack_record.argtypes = [C.c_int, u8p, u16p, u8p, u16p, u16p, u8p]
        L.orc_tq3_unpack_record.restype = None
        L.orc_tq3_unpack_record.argtypes = [C.c_int, u8p, u8p, u16p, u8p, u16p, u16p]
        L.orc_fp8_pack_record.restype = None
        L.orc_fp8_pack_record.argtypes = [C.c_int, f32p, f32p, C.c_int, C.c_float, C.c_float, u8p]
        L.orc_fp8_unpack_record_f32.restype = None
        L.orc_fp8_unpack_record_f32.argtypes = [C.c_int, u8p, C.c_float, C.c_float, f32p, f32p]
        L.orc_demote_record.restype = None
        L.orc_demote_record.argtypes = [C.c_int, u8p, C.c_float, C.c_float, i8p, u8p]
        L.orc_promote_record.restype = None
        L.orc_promote_record.argtypes = [C.c_int, u8p, C.c_float, C.c_float, i8p, u8p]
        L.orc_tq3_record_from_f32.restype = None
        L.orc_tq3_record_from_f32.argtypes = [C.c_int, f32p, f32p, i8p, u8p]
        L.orc_decode_attention.restype = C.c_int
        L.orc_decode_attention.argtypes = [u8p, C.c_int64, u8p, C.c_int64, C.c_int, C.c_int, C.c_int,
                                           C.c_float, C.c_float, i8p, u16p, i32p, u8p, i32p, C.c_int,
                                           C.c_int, C.c_double, f64p, f64p, C.c_int, C.c_int, C.c_int]
        L.orc_page_mass.restype = C.c_int
        L.orc_page_mass.argtypes = [u8p, C.c_int64, u8p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_float, C.c_float,
                                    i8p, u16p, i32p, u8p, i32p, C.c_int, C.c_int, C.c_double, f64p]
        L.orc_page_score_update.restype = None
        L.orc_page_score_update.argtypes = [f64p, i32p, C.c_int, C.c_int, C.c_int, C.c_uint64, C.c_double, f64p]
        L.orc_page_score_update_blocks.restype = None
        L.orc_page_score_update_blocks.argtypes = [f64p, i32p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_uint64, C.c_double, f64p]
        L.orc_page_mass_blocks.restype = C.c_int
        L.orc_page_mass_blocks.argtypes = [u8p, C.c_int64, u8p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float,
                                           C.c_float, i8p, u16p, i32p, u8p, i32p, C.c_int, C.c_int, C.c_double, f64p]
        L.orc_encode_request.restype = C.c_int
        L.orc_encode_request.argtypes = [C.c_int, C.c_int, C.c_int, u16p, u16p, i32p, u8p, i8p,
                                         C.c_float, C.c_float, u8p, u8p]
        L.orc_fp8_block_bytes.restype = C.c_int64
        L.orc_fp8_block_bytes.argtypes = [C.c_int, C.c_int]
        L.orc_tq3_block_bytes.restype = C.c_int64
        L.orc_tq3_block_bytes.argtypes = [C.c_int, C.c_int]
        L.orc_tq3_encode_value_block.restype = None
        L.orc_tq3_encode_value_block.argtypes = [f32p, C.c_int, C.c_int, u8p, u16p, u16p]
        L.orc_tq3_pack_block.restype = None
        L.orc_tq3_pack_block.argtypes = [C.c_int, C.c_int, u8p, u16p, u8p, u16p, u16p, u8p]
        L.orc_tq3_unpack_block.restype = None
        L.orc_tq3_unpack_block.argtypes = [C.c_int, C.c_int, u8p, u8p, u16p, u8p, u16p, u16p]
        L.orc_tq3_block_from_f32.restype = None
        L.orc_tq3_block_from_f32.argtypes = [C.c_int, C.c_int, f32p, f32p, i8p, u8p]
        L.orc_fp8_pack_block.restype = None
        L.orc_fp8_pack_block.argtypes = [C.c_int, C.c_int, f32p, f32p, C.c_int, C.c_float, C.c_float, u8p]
        L.orc_fp8_unpack_block_f32.restype = None
        L.orc_fp8_unpack_block_f32.argtypes = [C.c_int, C.c_int, u8p, C.c_float, C.c_float, f32p, f32p]
        L.orc_demote_block.restype = None
        L.orc_demote_block.argtypes = [C.c_int, C.c_int, u8p, C.c_float, C.c_float, i8p, u8p]
        L.orc_promote_block.restype = None
        L.orc_promote_block.argtypes = [C.c_int, C.c_int, u8p, C.c_float, C.c_float, i8p, u8p]
        L.orc_decode_attention_blocks.restype = C.c_int
        L.orc_decode_attention_blocks.argtypes = [u8p, C.c_int64, u8p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_int,
                                                  C.c_float, C.c_float, i8p, u16p, i32p, u8p, i32p, C.c_int,
                                                  C.c_int, C.c_double, f64p, f64p, C.c_int, C.c_int, C.c_int]
        L.orc_encode_request_blocks.restype = C.c_int
        L.orc_encode_request_blocks.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, u16p, u16p, i32p, u8p, i8p,
                                                C.c_float, C.c_float, u8p, u8p]
        L.orc_kv_bytes_per_token.restype = C.c_int64
        L.orc_kv_bytes_per_token.argtypes = [C.c_int] * 4
        L.orc_page_bytes_dense.restype = C.c_int64
        L.orc_page_bytes_dense.argtypes = [C.c_int] * 4
        L.orc_page_bytes_tq3.restype = C.c_int64
        L.orc_page_bytes_tq3.argtypes = [C.c_int] * 3
        L.orc_tq3_bits_per_scalar.restype = C.c_double
        L.orc_tq3_bits_per_scalar.argtypes = [C.c_int, C.c_int]
        L.orc_effective_bits.restype = C.c_double
        L.orc_effective_bits.argtypes = [C.c_double] * 5
        _lib = L
    return _lib


def set_format(fmt: int) -> None:
    """Select the TQ3 record format (1: fp16 Lloyd-Max codebook; 2: e4m3-exact codebook and the re-cut key
    section) that every oracle function uses from now on."""
    if lib().orc_set_format(int(fmt)) != 0:
        raise ValueError("record format must be 1 or 2")


def get_format() -> int:
    return lib().orc_get_format()


class record_format:
    """with oracle.record_format(2): ...  -- run a block under one record format, then restore."""

    def __init__(self, fmt: int):
        self.fmt = fmt

    def __enter__(self):
        self.prev = get_format()
        set_format(self.fmt)
        return self

    def __exit__(self, *exc):
        set_format(self.prev)


def _p(a: np.ndarray, ty):
    return a.ctypes.data_as(C.POINTER(ty))


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


# ---------------------------------------------------------------------------- scalar formats
def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp32: a bf16 is the upper half of an fp32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def e4m3_decode(b: int) -> float:
    return lib().orc_e4m3_decode(int(b) & 0xFF)


def e4m3_encode(x: float) -> int:
    return lib().orc_e4m3_encode(np.float32(x))


def f32_to_f16_sat(x: float) -> int:
    return lib().orc_f32_to_f16_sat(np.float32(x))


def f16_to_f32(u: int) -> float:
    return lib().orc_f16_to_f32(int(u))


def codebook():
    """(levels C[0..3], thresholds B[0..2]) of the TQ3 key quantiser as fp32."""
    L = lib()
    return (np.array([L.orc_codebook_level(j) for j in range(4)], dtype=np.float32),
            np.array([L.orc_codebook_threshold(j) for j in range(3)], dtype=np.float32))


# ---------------------------------------------------------------------------- TQ3 codec
def tq3_encode_key(x: np.ndarray, sigma: np.ndarray):
    """One key vector (fp32 [d]) -> (codes uint8 [d], g fp16 bits).  Section 4.1 / 3.1."""
    x = _c(x, np.float32)
    sigma = _c(sigma, np.int8)
    d = x.shape[0]
    code = np.zeros(d, np.uint8)
    g = C.c_uint16(0)
    lib().orc_tq3_encode_key(_p(x, C.c_float), d, _p(sigma, C.c_int8), _p(code, C.c_uint8), C.byref(g))
    return code, int(g.value)


def tq3_decode_key(code: np.ndarray, g: int, sigma: np.ndarray) -> np.ndarray:
    code = _c(code, np.uint8)
    sigma = _c(sigma, np.int8)
    out = np.zeros(code.shape[0], np.float64)
    lib().orc_tq3_decode_key(_p(code, C.c_uint8), int(g), code.shape[0], _p(sigma, C.c_int8),
                             _p(out, C.c_double))
    return out


def tq3_encode_value_page(v: np.ndarray):
    """One full page of values (fp32 [16][d]) -> (codes uint8 [16][d], scale fp16 bits [d], zero fp16 bits [d])."""
    v = _c(v, np.float32)
    assert v.shape[0] == T
    d = v.shape[1]
    code = np.zeros((T, d), np.uint8)
    sc = np.zeros(d, np.uint16)
    zp = np.zeros(d, np.uint16)
    lib().orc_tq3_encode_value_page(_p(v, C.c_float), d, _p(code, C.c_uint8), _p(sc, C.c_uint16),
                                    _p(zp, C.c_uint16))
    return code, sc, zp


def tq3_decode_value(code: int, sc: int, zp: int) -> float:
    return lib().orc_tq3_decode_value(int(code), int(sc), int(zp))


def fp8_record_bytes(d: int) -> int:
    return lib().orc_fp8_record_bytes(d)


def tq3_record_bytes(d: int) -> int:
    return lib().orc_tq3_record_bytes(d)


def tq3_pack_record(kcode, g, vcode, sc, zp) -> np.ndarray:
    kcode = _c(kcode, np.uint8)
    vcode = _c(vcode, np.uint8)
    g = _c(g, np.uint16)
    sc = _c(sc, np.uint16)
    zp = _c(zp, np.uint16)
    d = kcode.shape[1]
    rec = np.zeros(tq3_record_bytes(d), np.uint8)
    lib().orc_tq3_pack_record(d, _p(kcode, C.c_uint8), _p(g, C.c_uint16), _p(vcode, C.c_uint8),
                              _p(sc, C.c_uint16), _p(zp, C.c_uint16), _p(rec, C.c_uint8))
    return rec


def tq3_unpack_record(rec: np.ndarray, d: int):
    rec = _c(rec, np.uint8)
    kcode = np.zeros((T, d), np.uint8)
    vcode = np.zeros((T, d), np.uint8)
    g = np.zeros(T, np.uint16)
    sc = np.zeros(d, np.uint16)
    zp = np.zeros(d, np.uint16)
    lib().orc_tq3_unpack_record(d, _p(rec, C.c_uint8), _p(kcode, C.c_uint8), _p(g, C.c_uint16),
                                _p(vcode, C.c_uint8), _p(sc, C.c_uint16), _p(zp, C.c_uint16))
    return kcode, g, vcode, sc, zp


def fp8_pack_record(k: np.ndarray, v: np.ndarray, n_valid: int = T, k_scale=1.0, v_scale=1.0) -> np.ndarray:
    """fp32 K,V [16][d] of one (page, head) -> FP8 record bytes (Append of Algorithm 1, data part)."""
    k = _c(k, np.float32)
    v = _c(v, np.float32)
    d = k.shape[1]
    rec = np.zeros(fp8_record_bytes(d), np.uint8)
    lib().orc_fp8_pack_record(d, _p(k, C.c_float), _p(v, C.c_float), n_valid, k_scale, v_scale,
                              _p(rec, C.c_uint8))
    return rec


def fp8_unpack_record_f32(rec: np.ndarray, d: int, k_scale=1.0, v_scale=1.0):
    rec = _c(rec, np.uint8)
    k = np.zeros((T, d), np.float32)
    v = np.zeros((T, d), np.float32)
    lib().orc_fp8_unpack_record_f32(d, _p(rec, C.c_uint8), k_scale, v_scale, _p(k, C.c_float),
                                    _p(v, C.c_float))
    return k, v


def demote_record(fp8_rec: np.ndarray, d: int, sigma: np.ndarray, k_scale=1.0, v_scale=1.0) -> np.ndarray:
    """FP8 record -> TQ3 record (Retier of Algorithm 1, data part; normalize-rotate-pack)."""
    fp8_rec = _c(fp8_rec, np.uint8)
    sigma = _c(sigma, np.int8)
    out = np.zeros(tq3_record_bytes(d), np.uint8)
    lib().orc_demote_record(d, _p(fp8_rec, C.c_uint8), k_scale, v_scale, _p(sigma, C.c_int8),
                            _p(out, C.c_uint8))
    return out


def promote_record(tq3_rec: np.ndarray, d: int, sigma: np.ndarray, k_scale=1.0, v_scale=1.0) -> np.ndarray:
    """TQ3 record -> FP8 record (Promote of Algorithm 1, data part: reconstruct, then round to e4m3)."""
    tq3_rec = _c(tq3_rec, np.uint8)
    sigma = _c(sigma, np.int8)
    out = np.zeros(fp8_record_bytes(d), np.uint8)
    lib().orc_promote_record(d, _p(tq3_rec, C.c_uint8), k_scale, v_scale, _p(sigma, C.c_int8), _p(out, C.c_uint8))
    return out


def tq3_record_from_f32(k: np.ndarray, v: np.ndarray, sigma: np.ndarray) -> np.ndarray:
    k = _c(k, np.float32)
    v = _c(v, np.float32)
    sigma = _c(sigma, np.int8)
    d = k.shape[1]
    out = np.zeros(tq3_record_bytes(d), np.uint8)
    lib().orc_tq3_record_from_f32(d, _p(k, C.c_float), _p(v, C.c_float), _p(sigma, C.c_int8),
                                  _p(out, C.c_uint8))
    return out


# ---------------------------------------------------------------------------- pages of 16 M tokens
def fp8_block_bytes(d: int, M: int) -> int:
    return lib().orc_fp8_block_bytes(d, M)


def tq3_block_bytes(d: int, M: int) -> int:
    """M (12 d + 32) + 4 d: M tiles of key codes, value codes and g, one scale/zero set per page."""
    return lib().orc_tq3_block_bytes(d, M)


def tq3_encode_value_block(v: np.ndarray):
    """Values of one full page (fp32 [T][d], any T) -> (codes uint8 [T][d], scale fp16 bits [d], zero fp16 bits [d]);
    one scale/zero per channel over all T tokens."""
    v = _c(v, np.float32)
    Tn, d = v.shape
    code = np.zeros((Tn, d), np.uint8)
    sc = np.zeros(d, np.uint16)
    zp = np.zeros(d, np.uint16)
    lib().orc_tq3_encode_value_block(_p(v, C.c_float), d, Tn, _p(code, C.c_uint8), _p(sc, C.c_uint16), _p(zp, C.c_uint16))
    return code, sc, zp


def tq3_pack_block(kcode, g, vcode, sc, zp) -> np.ndarray:
    kcode, vcode = _c(kcode, np.uint8), _c(vcode, np.uint8)
    g, sc, zp = _c(g, np.uint16), _c(sc, np.uint16), _c(zp, np.uint16)
    Tn, d = kcode.shape
    assert Tn % T == 0
    rec = np.zeros(tq3_block_bytes(d, Tn // T), np.uint8)
    lib().orc_tq3_pack_block(d, Tn // T, _p(kcode, C.c_uint8), _p(g, C.c_uint16), _p(vcode, C.c_uint8),
                             _p(sc, C.c_uint16), _p(zp, C.c_uint16), _p(rec, C.c_uint8))
    return rec


def tq3_unpack_block(rec: np.ndarray, d: int, M: int):
    rec = _c(rec, np.uint8)
    kcode = np.zeros((T * M, d), np.uint8)
    vcode = np.zeros((T * M, d), np.uint8)
    g = np.zeros(T * M, np.uint16)
    sc = np.zeros(d, np.uint16)
    zp = np.zeros(d, np.uint16)
    lib().orc_tq3_unpack_block(d, M, _p(rec, C.c_uint8), _p(kcode, C.c_uint8), _p(g, C.c_uint16),
                               _p(vcode, C.c_uint8), _p(sc, C.c_uint16), _p(zp, C.c_uint16))
    return kcode, g, vcode, sc, zp


def tq3_block_from_f32(k: np.ndarray, v: np.ndarray, sigma: np.ndarray) -> np.ndarray:
    k, v, sigma = _c(k, np.float32), _c(v, np.float32), _c(sigma, np.int8)
    Tn, d = k.shape
    assert Tn % T == 0 and v.shape == k.shape
    out = np.zeros(tq3_block_bytes(d, Tn // T), np.uint8)
    lib().orc_tq3_block_from_f32(d, Tn // T, _p(k, C.c_float), _p(v, C.c_float), _p(sigma, C.c_int8), _p(out, C.c_uint8))
    return out


def fp8_pack_block(k: np.ndarray, v: np.ndarray, n_valid=None, k_scale=1.0, v_scale=1.0) -> np.ndarray:
    k, v = _c(k, np.float32), _c(v, np.float32)
    Tn, d = k.shape
    assert Tn % T == 0
    out = np.zeros(fp8_block_bytes(d, Tn // T), np.uint8)
    lib().orc_fp8_pack_block(d, Tn // T, _p(k, C.c_float), _p(v, C.c_float), Tn if n_valid is None else n_valid,
                             k_scale, v_scale, _p(out, C.c_uint8))
    return out


def fp8_unpack_block_f32(rec: np.ndarray, d: int, M: int, k_scale=1.0, v_scale=1.0):
    rec = _c(rec, np.uint8)
    k = np.zeros((T * M, d), np.float32)
    v = np.zeros((T * M, d), np.float32)
    lib().orc_fp8_unpack_block_f32(d, M, _p(rec, C.c_uint8), k_scale, v_scale, _p(k, C.c_float), _p(v, C.c_float))
    return k, v


def demote_block(fp8_block: np.ndarray, d: int, M: int, sigma: np.ndarray, k_scale=1.0, v_scale=1.0) -> np.ndarray:
    fp8_block, sigma = _c(fp8_block, np.uint8), _c(sigma, np.int8)
    out = np.zeros(tq3_block_bytes(d, M), np.uint8)
    lib().orc_demote_block(d, M, _p(fp8_block, C.c_uint8), k_scale, v_scale, _p(sigma, C.c_int8), _p(out, C.c_uint8))
    return out


def promote_block(tq3_block: np.ndarray, d: int, M: int, sigma: np.ndarray, k_scale=1.0, v_scale=1.0) -> np.ndarray:
    tq3_block, sigma = _c(tq3_block, np.uint8), _c(sigma, np.int8)
    out = np.zeros(fp8_block_bytes(d, M), np.uint8)
    lib().orc_promote_block(d, M, _p(tq3_block, C.c_uint8), k_scale, v_scale, _p(sigma, C.c_int8), _p(out, C.c_uint8))
    return out


# ---------------------------------------------------------------------------- bulk page encoding
def encode_fp8_pages(k_bits: np.ndarray, v_bits: np.ndarray, n_valid: int = T, k_scale=1.0,
                     v_scale=1.0) -> np.ndarray:
    """bf16 bits [H][16][d] of one page -> FP8 records [H][32d]."""
    H, _, d = k_bits.shape
    out = np.zeros((H, fp8_record_bytes(d)), np.uint8)
    kf, vf = bf16_bits_to_f32(k_bits), bf16_bits_to_f32(v_bits)
    for h in range(H):
        out[h] = fp8_pack_record(kf[h], vf[h], n_valid, k_scale, v_scale)
    return out


def encode_tq3_pages(k_bits: np.ndarray, v_bits: np.ndarray, sigma: np.ndarray) -> np.ndarray:
    """bf16 bits [H][16][d] of one full page -> TQ3 records [H][16d+32], encoded from the bf16 originals."""
    H, _, d = k_bits.shape
    out = np.zeros((H, tq3_record_bytes(d)), np.uint8)
    kf, vf = bf16_bits_to_f32(k_bits), bf16_bits_to_f32(v_bits)
    for h in range(H):
        out[h] = tq3_record_from_f32(kf[h], vf[h], sigma)
    return out


def encode_request(k_bits, v_bits, row, tags, sigma, fp8_arena, tq3_arena, k_scale=1.0, v_scale=1.0, page_tokens=T):
    """Write all pages of one request (bf16 bits [len][hkv][d]) into the uint8 arenas in place
    (pages of `page_tokens` = 16 M tokens)."""
    k_bits = _c(k_bits, np.uint16)
    v_bits = _c(v_bits, np.uint16)
    row = _c(row, np.int32)
    tags = _c(tags, np.uint8)
    sigma = _c(sigma, np.int8)
    ln, hkv, d = k_bits.shape
    assert fp8_arena.dtype == np.uint8 and fp8_arena.flags.c_contiguous
    assert tq3_arena.dtype == np.uint8 and tq3_arena.flags.c_contiguous
    dummy = np.zeros(16, np.uint8)
    assert page_tokens % T == 0 and page_tokens >= T
    rc = lib().orc_encode_request_blocks(d, hkv, ln, page_tokens // T, _p(k_bits, C.c_uint16), _p(v_bits, C.c_uint16),
                                  _p(row, C.c_int32), _p(tags, C.c_uint8), _p(sigma, C.c_int8),
                                  k_scale, v_scale,
                                  _p(fp8_arena if fp8_arena.size else dummy, C.c_uint8),
                                  _p(tq3_arena if tq3_arena.size else dummy, C.c_uint8))
    if rc != 0:
        raise ValueError("oracle: invalid tag or partial Stale page")


# ---------------------------------------------------------------------------- attention
def decode_attention(fp8_arena, tq3_arena, d, hkv, group, sigma, q_bits, block_table, tier_tag,
                     seq_lens, scale, k_scale=1.0, v_scale=1.0, mode=0, only_b=-1, only_h=-1, page_tokens=T):
    """Dequantise-then-attend in fp64 (Section 3.3).  Returns (out [B][Hq][d], lse [B][Hq]).

    fp8_arena: uint8 [fp8_pages][hkv][32d]; tq3_arena: uint8 [tq3_pages][hkv][16d+32];
    q_bits: bf16 bits [B][Hq][d]; block_table int32 [B][max_pages]; tier_tag uint8 [B][max_pages].
    mode 0 = one softmax; 1 = Eq. (softmax-merge) over the two format partitions;
    n >= 2 = Eq. (softmax-merge) over n contiguous ranges.
    page_tokens = 16 M: pages of M tiles (arenas then hold [pages][hkv][M * 32d] and
    [pages][hkv][M * (12d + 32) + 4d] bytes).
    """
    fp8_arena = _c(fp8_arena, np.uint8)
    tq3_arena = _c(tq3_arena, np.uint8)
    sigma = _c(sigma, np.int8)
    q_bits = _c(q_bits, np.uint16)
    block_table = _c(block_table, np.int32)
    tier_tag = _c(tier_tag, np.uint8)
    seq_lens = _c(seq_lens, np.int32)
    B, max_pages = block_table.shape
    Hq = hkv * group
    assert q_bits.shape == (B, Hq, d)
    assert page_tokens % T == 0 and page_tokens >= T
    M = page_tokens // T
    fp8_pages = fp8_arena.size // (hkv * fp8_block_bytes(d, M)) if fp8_arena.size else 0
    tq3_pages = tq3_arena.size // (hkv * tq3_block_bytes(d, M)) if tq3_arena.size else 0
    out = np.zeros((B, Hq, d), np.float64)
    lse = np.zeros((B, Hq), np.float64)
    dummy = np.zeros(16, np.uint8)
    rc = lib().orc_decode_attention_blocks(
        _p(fp8_arena if fp8_arena.size else dummy, C.c_uint8), fp8_pages,
        _p(tq3_arena if tq3_arena.size else dummy, C.c_uint8), tq3_pages, d, hkv, group, M,
        k_scale, v_scale, _p(sigma, C.c_int8), _p(q_bits, C.c_uint16), _p(block_table, C.c_int32),
        _p(tier_tag, C.c_uint8), _p(seq_lens, C.c_int32), B, max_pages, float(scale),
        _p(out, C.c_double), _p(lse, C.c_double), mode, only_b, only_h)
    if rc != 0:
        raise ValueError("oracle: invalid block-table entry or tier tag")
    return out, lse


def page_mass(fp8_arena, tq3_arena, d, hkv, group, sigma, q_bits, block_table, tier_tag, seq_lens, scale,
              k_scale=1.0, v_scale=1.0, page_tokens=T):
    """Globally normalised attention mass of every page, q~ [B][Hq][max_pages] in fp64 (Eq. score-partial,
    Eq. score-global-weight with the two format partitions).  Arguments as decode_attention."""
    fp8_arena = _c(fp8_arena, np.uint8)
    tq3_arena = _c(tq3_arena, np.uint8)
    sigma = _c(sigma, np.int8)
    q_bits = _c(q_bits, np.uint16)
    block_table = _c(block_table, np.int32)
    tier_tag = _c(tier_tag, np.uint8)
    seq_lens = _c(seq_lens, np.int32)
    B, max_pages = block_table.shape
    Hq = hkv * group
    assert q_bits.shape == (B, Hq, d)
    M = page_tokens // T
    fp8_pages = fp8_arena.size // (hkv * fp8_block_bytes(d, M)) if fp8_arena.size else 0
    tq3_pages = tq3_arena.size // (hkv * tq3_block_bytes(d, M)) if tq3_arena.size else 0
    mass = np.zeros((B, Hq, max_pages), np.float64)
    dummy = np.zeros(16, np.uint8)
    rc = lib().orc_page_mass_blocks(
        _p(fp8_arena if fp8_arena.size else dummy, C.c_uint8), fp8_pages,
        _p(tq3_arena if tq3_arena.size else dummy, C.c_uint8), tq3_pages, d, hkv, group, M,
        k_scale, v_scale, _p(sigma, C.c_int8), _p(q_bits, C.c_uint16), _p(block_table, C.c_int32),
        _p(tier_tag, C.c_uint8), _p(seq_lens, C.c_int32), B, max_pages, float(scale), _p(mass, C.c_double))
    if rc != 0:
        raise ValueError("oracle: invalid block-table entry or tier tag")
    return mass


def page_score_update(mass, seq_lens, head_mask, beta, score, page_tokens=T):
    """Eq. (attention-score): returns beta * score + (1 - beta) * mean_{h in head set} mass[:, h, :] for the
    pages below each request's length (other entries unchanged).  score: [B][max_pages] fp64."""
    mass = _c(mass, np.float64)
    seq_lens = _c(seq_lens, np.int32)
    out = np.array(score, np.float64, copy=True, order="C")
    B, Hq, max_pages = mass.shape
    lib().orc_page_score_update_blocks(_p(mass, C.c_double), _p(seq_lens, C.c_int32), B, Hq, max_pages, int(page_tokens),
                                       C.c_uint64(int(head_mask)), float(beta), _p(out, C.c_double))
    return out


# ---------------------------------------------------------------------------- accounting
def kv_bytes_per_token(layers, hkv, d, bytes_per_scalar):
    """Eq. (kv-per-token): 2 L_f H_kv d_h s."""
    return lib().orc_kv_bytes_per_token(layers, hkv, d, bytes_per_scalar)


def page_bytes_dense(Tp, d, hkv, bytes_per_scalar):
    return lib().orc_page_bytes_dense(Tp, d, hkv, bytes_per_scalar)


def page_bytes_tq3(Tp, d, hkv):
    return lib().orc_page_bytes_tq3(Tp, d, hkv)


def tq3_bits_per_scalar(Tp, d):
    return lib().orc_tq3_bits_per_scalar(Tp, d)


def effective_bits(p_R, p_A, p_S, b_S, b_meta=0.0):
    """Eq. (effective-bits)."""
    return lib().orc_effective_bits(p_R, p_A, p_S, b_S, b_meta)
