"""CPU oracle for paged-KV GQA decode attention (TEST INFRASTRUCTURE ONLY).

This package wraps ``attn_oracle.c`` (plain single-threaded fp64 C) through ctypes.
It is what the CUDA library is checked against; it shares no code with the CUDA
path and imports nothing from it.  Only tests, the smoke check and the benchmark's
CPU-baseline leg may use it; the product path never does.

Operation (the paper, arXiv 2510.07356, decodes long reasoning traces with 32B GQA
models in Sec. 3.3 / Sec. 4.2 but states no formula; this is the textbook
definition): ``out = softmax(scale * q K^T) V`` per query head over the tokens a
block table maps into a paged pool, ``lse = ln sum exp(scale * q k_j)``.

Every function is pinned by tests/test_oracle_pins.py (closed forms, invariances,
brute force, a library second opinion).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "attn_oracle.c"
_LIB = _HERE / "liboracle_attn.so"
_lib = None


class Geom(ctypes.Structure):
    _fields_ = [
        ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("page_size", ctypes.c_int32),
        ("block_table_stride", ctypes.c_int32),
    ]


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (no fast-math: fp64 semantics are kept strict)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fno-fast-math",
             "-ffp-contract=off", "-o", str(tmp), str(_SRC), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        u16p = ctypes.POINTER(ctypes.c_uint16)
        i32p = ctypes.POINTER(ctypes.c_int32)
        f64p = ctypes.POINTER(ctypes.c_double)
        lib.oracle_attn_range.restype = ctypes.c_int
        lib.oracle_attn_range.argtypes = [
            u16p, u16p, u16p, i32p, ctypes.POINTER(Geom), ctypes.c_float,
            ctypes.c_int32, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64, f64p, f64p]
        lib.oracle_decode_attn.restype = ctypes.c_int
        lib.oracle_decode_attn.argtypes = [
            u16p, u16p, u16p, i32p, i32p, ctypes.POINTER(Geom), ctypes.c_float,
            ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, f64p, f64p]
        lib.oracle_lse_merge.restype = None
        lib.oracle_lse_merge.argtypes = [f64p, f64p, ctypes.c_int32, ctypes.c_int32, f64p, f64p]
        _lib = lib
    return _lib


def _u16(a) -> np.ndarray:
    """bf16 bit patterns as a C-contiguous uint16 array (accepts torch bf16 or numpy uint16)."""
    if hasattr(a, "detach"):  # torch tensor
        import torch
        a = a.detach().cpu().contiguous()
        if a.dtype == torch.bfloat16:
            a = a.view(torch.int16)
        a = a.numpy()
    a = np.ascontiguousarray(a)
    if a.dtype == np.int16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError(f"expected bf16 bit patterns (uint16), got {a.dtype}")
    return a


def _i32(a) -> np.ndarray:
    if hasattr(a, "detach"):
        a = a.detach().cpu().numpy()
    return np.ascontiguousarray(a, dtype=np.int32)


def _ptr(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def _geom(q, k_pages, block_table) -> Geom:
    _, hq, d = q.shape
    _, hkv, p, d2 = k_pages.shape
    assert d == d2 and hq % hkv == 0
    return Geom(hq, hkv, d, p, block_table.shape[1])


def decode_attn(q, k_pages, v_pages, block_table, seq_lens, scale: float,
                seqs=None, heads=None):
    """Whole operation.  q [B][Hq][D], k_pages/v_pages [pages][Hkv][P][D] (bf16 bits),
    block_table [B][stride] int32, seq_lens [B] int32.  Returns (out [B][Hq][D] f64,
    lse [B][Hq] f64).  ``seqs``/``heads`` = (begin, end) restrict what is computed;
    entries outside stay NaN."""
    lib = _load()
    q, k_pages, v_pages = _u16(q), _u16(k_pages), _u16(v_pages)
    block_table, seq_lens = _i32(block_table), _i32(seq_lens)
    ge = _geom(q, k_pages, block_table)
    B = q.shape[0]
    out = np.full((B, ge.num_q_heads, ge.head_dim), np.nan, dtype=np.float64)
    lse = np.full((B, ge.num_q_heads), np.nan, dtype=np.float64)
    b0, b1 = seqs if seqs is not None else (0, B)
    h0, h1 = heads if heads is not None else (0, ge.num_q_heads)
    rc = lib.oracle_decode_attn(
        _ptr(q, ctypes.c_uint16), _ptr(k_pages, ctypes.c_uint16), _ptr(v_pages, ctypes.c_uint16),
        _ptr(block_table, ctypes.c_int32), _ptr(seq_lens, ctypes.c_int32), ctypes.byref(ge),
        ctypes.c_float(scale), b0, b1, h0, h1, _ptr(out, ctypes.c_double), _ptr(lse, ctypes.c_double))
    if rc:
        raise MemoryError("oracle score buffer")
    return out, lse


def attn_range(q, k_pages, v_pages, block_table, scale: float, b: int, h: int, j0: int, j1: int):
    """One (sequence, query head) over tokens j0 <= j < j1.  Returns (out [D] f64, lse float)."""
    lib = _load()
    q, k_pages, v_pages = _u16(q), _u16(k_pages), _u16(v_pages)
    block_table = _i32(block_table)
    ge = _geom(q, k_pages, block_table)
    out = np.zeros(ge.head_dim, dtype=np.float64)
    lse = ctypes.c_double(0.0)
    rc = lib.oracle_attn_range(
        _ptr(q, ctypes.c_uint16), _ptr(k_pages, ctypes.c_uint16), _ptr(v_pages, ctypes.c_uint16),
        _ptr(block_table, ctypes.c_int32), ctypes.byref(ge), ctypes.c_float(scale),
        b, h, j0, j1, _ptr(out, ctypes.c_double), ctypes.byref(lse))
    if rc:
        raise MemoryError("oracle score buffer")
    return out, lse.value


def lse_merge(part_out, part_lse):
    """Merge partial results [parts][D], [parts] of disjoint token ranges -> (out [D], lse)."""
    lib = _load()
    part_out = np.ascontiguousarray(part_out, dtype=np.float64)
    part_lse = np.ascontiguousarray(part_lse, dtype=np.float64)
    parts, D = part_out.shape
    out = np.zeros(D, dtype=np.float64)
    lse = ctypes.c_double(0.0)
    lib.oracle_lse_merge(_ptr(part_out, ctypes.c_double), _ptr(part_lse, ctypes.c_double),
                         parts, D, _ptr(out, ctypes.c_double), ctypes.byref(lse))
    return out, lse.value
