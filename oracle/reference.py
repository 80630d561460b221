"""TEST INFRASTRUCTURE -- ctypes loader for the FP64 C++ oracle.

``build()`` compiles ``mla_decode_oracle.cpp`` and ``mla_decode_oracle_fp8.cpp``
with g++ (OpenMP) into ``liboracle_amla.so`` next to them; ``decode`` /
``decode_rows`` / ``decode_fp8`` call it on numpy arrays.  No CUDA, no torch.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mla_decode_oracle.cpp")
_SRC_FP8 = os.path.join(_HERE, "mla_decode_oracle_fp8.cpp")
_LIB = os.path.join(_HERE, "liboracle_amla.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_FP8)):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fopenmp", "-fPIC", "-shared", _SRC, _SRC_FP8, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        vp, i32, f64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_double
        lib.oracle_mla_decode.argtypes = [vp, vp, vp, vp, f64, i32, i32, i32, i32, i32, vp, vp, i32]
        lib.oracle_mla_decode.restype = i32
        lib.oracle_mla_decode_rows.argtypes = [vp, vp, vp, vp, f64, i32, i32, i32, i32, i32, vp, i32, vp, vp, i32]
        lib.oracle_mla_decode_rows.restype = i32
        lib.oracle_num_threads.restype = i32
        lib.oracle_mla_decode_fp8.argtypes = [vp, vp, f64, vp, vp, f64, i32, i32, i32, i32, i32, vp, vp, i32]
        lib.oracle_mla_decode_fp8.restype = i32
        lib.oracle_e4m3_to_double.argtypes = [ctypes.c_uint8]
        lib.oracle_e4m3_to_double.restype = f64
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _prep(q, kv, block_table, seqlens):
    q = np.ascontiguousarray(q, dtype=np.uint16)
    kv = np.ascontiguousarray(kv, dtype=np.uint16)
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    sl = np.ascontiguousarray(seqlens, dtype=np.int32)
    B, Sq, H, d = q.shape
    assert d == 576 and kv.shape[1:] == (64, 576) and bt.shape[0] == B and sl.shape == (B,)
    return q, kv, bt, sl, B, Sq, H


def decode(q, kv, block_table, seqlens, scale, n_threads: int = 0):
    """Full problem: returns (out float64 [B,Sq,H,512], lse float64 [B,Sq,H])."""
    q, kv, bt, sl, B, Sq, H = _prep(q, kv, block_table, seqlens)
    out = np.empty((B, Sq, H, 512), dtype=np.float64)
    lse = np.empty((B, Sq, H), dtype=np.float64)
    rc = _load().oracle_mla_decode(_ptr(q), _ptr(kv), _ptr(bt), _ptr(sl), float(scale), B, Sq, H,
                                   kv.shape[0], bt.shape[1], _ptr(out), _ptr(lse), int(n_threads))
    if rc != 0:
        raise ValueError("oracle: block table entry out of range")
    return out, lse


def decode_rows(q, kv, block_table, seqlens, scale, rows, n_threads: int = 0):
    """Selected (b, t, h) rows: returns (out float64 [n,512], lse float64 [n])."""
    q, kv, bt, sl, B, Sq, H = _prep(q, kv, block_table, seqlens)
    rows = np.ascontiguousarray(rows, dtype=np.int32).reshape(-1, 3)
    n = rows.shape[0]
    out = np.empty((n, 512), dtype=np.float64)
    lse = np.empty((n,), dtype=np.float64)
    rc = _load().oracle_mla_decode_rows(_ptr(q), _ptr(kv), _ptr(bt), _ptr(sl), float(scale), B, Sq, H,
                                        kv.shape[0], bt.shape[1], _ptr(rows), n, _ptr(out), _ptr(lse),
                                        int(n_threads))
    if rc != 0:
        raise ValueError("oracle: row index or block table entry out of range")
    return out, lse


def e4m3_to_double(byte: int) -> float:
    """The oracle's widening of one E4M3 byte."""
    return float(_load().oracle_e4m3_to_double(int(byte) & 0xFF))


def decode_fp8(q, kv_e4m3, kv_scale, block_table, seqlens, scale, n_threads: int = 0):
    """Full problem on an E4M3 cache (uint8 [num_blocks,64,576], element value = decode(byte) * kv_scale):
    returns (out float64 [B,Sq,H,512], lse float64 [B,Sq,H])."""
    q = np.ascontiguousarray(q, dtype=np.uint16)
    kv = np.ascontiguousarray(kv_e4m3, dtype=np.uint8)
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    sl = np.ascontiguousarray(seqlens, dtype=np.int32)
    B, Sq, H, d = q.shape
    assert d == 576 and kv.shape[1:] == (64, 576) and bt.shape[0] == B and sl.shape == (B,)
    out = np.empty((B, Sq, H, 512), dtype=np.float64)
    lse = np.empty((B, Sq, H), dtype=np.float64)
    rc = _load().oracle_mla_decode_fp8(_ptr(q), _ptr(kv), float(kv_scale), _ptr(bt), _ptr(sl), float(scale), B, Sq, H,
                                       kv.shape[0], bt.shape[1], _ptr(out), _ptr(lse), int(n_threads))
    if rc != 0:
        raise ValueError("oracle: block table entry out of range")
    return out, lse
