"""ctypes loader for the FFD CPU oracle (``ffd_oracle.c``).

TEST INFRASTRUCTURE ONLY: the oracle defines correctness for the CUDA library and is timed as a reported
CPU baseline.  Nothing in the product path imports this module, and this module imports nothing from the
CUDA package.  All arguments are numpy arrays on the host; bf16 / fp16 tensors travel as ``uint16`` bit
patterns.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ffd_oracle.c")
_LIB = os.path.join(_HERE, "libffd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, OpenMP for the loop over independent heads)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _ptr(a, ctype):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctype))


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.ffd_oracle_fp16_value.restype = ctypes.c_double
        _lib.ffd_oracle_fp16_value.argtypes = [ctypes.c_uint16]
        _lib.ffd_oracle_bf16_value.restype = ctypes.c_double
        _lib.ffd_oracle_bf16_value.argtypes = [ctypes.c_uint16]
        _lib.ffd_oracle_fp16_round.restype = ctypes.c_uint16
        _lib.ffd_oracle_fp16_round.argtypes = [ctypes.c_float]
        _lib.ffd_oracle_set_threads.argtypes = [ctypes.c_int]
    return _lib


def set_threads(n: int) -> None:
    lib().ffd_oracle_set_threads(int(n))


def max_threads() -> int:
    return int(lib().ffd_oracle_max_threads())


def fp16_value(bits: int) -> float:
    return float(lib().ffd_oracle_fp16_value(int(bits)))


def bf16_value(bits: int) -> float:
    return float(lib().ffd_oracle_bf16_value(int(bits)))


def fp16_round(x: float) -> int:
    return int(lib().ffd_oracle_fp16_round(ctypes.c_float(x)))


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def quantize(k_cache, block_table, seq_lens, max_blocks, bits: int = 2):
    """App. A.1 quantizer over every logical block with a valid token.

    k_cache: uint16 (bf16 bits) [num_pages, Hkv, BLK, D].  Returns (codes u8 [pages,Hkv,BLK,D] with values
    0 .. 2^bits - 1, level = code - (2^bits - 1) / 2; scales uint16 fp16 bits [pages,Hkv,D]).  Tiles that no sequence
    maps stay zero.  bits = 2 is the paper's thumbnail; 4 and 8 are the deeper ones of its quantization-depth appendix.
    """
    k_cache = _u16(k_cache)
    P, Hkv, BLK, D = k_cache.shape
    seq_lens = _i32(seq_lens)
    block_table = _i32(block_table)
    codes = np.zeros((P, Hkv, BLK, D), dtype=np.uint8)
    scales = np.zeros((P, Hkv, D), dtype=np.uint16)
    rc = lib().ffd_oracle_quantize(_ptr(k_cache, ctypes.c_uint16), _ptr(codes, ctypes.c_uint8),
                                   _ptr(scales, ctypes.c_uint16), _ptr(block_table, ctypes.c_int32),
                                   _ptr(seq_lens, ctypes.c_int32), len(seq_lens), Hkv, D, BLK, int(max_blocks), P, int(bits))
    if rc:
        raise ValueError(f"ffd_oracle_quantize: geometry error {rc}")
    return codes, scales


def quantize_residual(k_cache, codes, scales, block_table, seq_lens, max_blocks):
    """Sec. 3.1 residual: int8 [pages,Hkv,BLK,D], the part of K the 2-bit level misses, in units of scale/254
    (this file's reading; the paper prints no residual quantizer).  Padding rows and unmapped tiles are 0."""
    k_cache = _u16(k_cache)
    scales = _u16(scales)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    P, Hkv, BLK, D = k_cache.shape
    seq_lens = _i32(seq_lens)
    block_table = _i32(block_table)
    k_res = np.zeros((P, Hkv, BLK, D), dtype=np.int8)
    rc = lib().ffd_oracle_quantize_residual(
        _ptr(k_cache, ctypes.c_uint16), _ptr(codes, ctypes.c_uint8), _ptr(scales, ctypes.c_uint16),
        _ptr(k_res, ctypes.c_int8), _ptr(block_table, ctypes.c_int32), _ptr(seq_lens, ctypes.c_int32), len(seq_lens),
        Hkv, D, BLK, int(max_blocks), P)
    if rc:
        raise ValueError(f"ffd_oracle_quantize_residual: geometry error {rc}")
    return k_res


@dataclass
class DecodeResult:
    out: np.ndarray        # float64 [B, Hq, D]
    lse: np.ndarray        # float64 [B, Hq]
    kept: np.ndarray       # uint8   [B, Hq, max_blocks]   (entries past a sequence's block count are 0)
    block_max: np.ndarray  # float64 [B, Hq, max_blocks]   (entries past the block count are -inf)
    mtilde: np.ndarray     # float64 [B, Hq]
    thr: np.ndarray = None  # float64 [B, Hq, max_blocks]   the threshold each block maximum was compared with (nan past the block count)


RULE_PSEUDO_MAX, RULE_GLOBAL_MAX, RULE_RUNNING_MAX, RULE_TOP_K = 0, 1, 2, 3


def _units(units):
    if units is None:
        return None, 0
    # duplicates would make two threads write the same output row: keep each (b, h) once
    u = np.unique(np.asarray(units, dtype=np.int32).reshape(-1, 2), axis=0)
    u = np.ascontiguousarray(u)
    return u, len(u)


def decode(q, k_cache, v_cache, codes, scales, block_table, seq_lens, max_blocks, delta, *, n_sink=1, n_local=16,
           sm_scale=None, forced_mask=None, units=None, k_res=None, bits: int = 2, rule: int = RULE_PSEUDO_MAX,
           top_k: int = 0) -> DecodeResult:
    """Alg. 1: approximate scores -> pseudo-max -> top-delta -> exact attention over kept blocks.

    ``rule``: the reference the block maxima are compared with.  RULE_PSEUDO_MAX is the paper's method; the others are
    the comparison rules: RULE_GLOBAL_MAX (Sec. 5.2), RULE_RUNNING_MAX (the pseudo-max raised by the block maxima met so
    far, blocks in logical order), RULE_TOP_K (fixed budget ``top_k`` blocks per head, ties with the k-th kept; ``delta``
    unused).

    ``k_res`` (int8, from ``quantize_residual``): refine from Dequant(codes, k_res) instead of the 16-bit K.

    ``units``: optional list of (b, h) pairs; only those rows of the result are computed (others stay at
    their fill values: out 0, lse nan, block_max -inf).  ``forced_mask`` replaces the top-delta decisions.
    """
    q = _u16(q)
    k_cache = _u16(k_cache)
    v_cache = _u16(v_cache)
    scales = _u16(scales)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    B, Hq, D = q.shape
    P, Hkv, BLK, _ = k_cache.shape
    seq_lens = _i32(seq_lens)
    block_table = _i32(block_table)
    if sm_scale is None:
        sm_scale = 1.0 / math.sqrt(D)
    out = np.zeros((B, Hq, D), dtype=np.float64)
    lse = np.full((B, Hq), np.nan, dtype=np.float64)
    kept = np.zeros((B, Hq, max_blocks), dtype=np.uint8)
    bm = np.full((B, Hq, max_blocks), -np.inf, dtype=np.float64)
    mt = np.full((B, Hq), np.nan, dtype=np.float64)
    thr = np.full((B, Hq, max_blocks), np.nan, dtype=np.float64)
    fm = None if forced_mask is None else np.ascontiguousarray(forced_mask, dtype=np.uint8)
    u, nu = _units(units)
    kr = None if k_res is None else np.ascontiguousarray(k_res, dtype=np.int8)
    assert kr is None or kr.shape == k_cache.shape
    rc = lib().ffd_oracle_decode(
        _ptr(q, ctypes.c_uint16), _ptr(k_cache, ctypes.c_uint16), _ptr(v_cache, ctypes.c_uint16),
        _ptr(codes, ctypes.c_uint8), _ptr(scales, ctypes.c_uint16), _ptr(block_table, ctypes.c_int32),
        _ptr(seq_lens, ctypes.c_int32), B, Hq, Hkv, D, BLK, int(max_blocks), P, int(n_sink), int(n_local),
        ctypes.c_double(sm_scale), ctypes.c_double(delta), _ptr(fm, ctypes.c_uint8), _ptr(u, ctypes.c_int32), nu,
        _ptr(out, ctypes.c_double), _ptr(lse, ctypes.c_double), _ptr(kept, ctypes.c_uint8),
        _ptr(bm, ctypes.c_double), _ptr(mt, ctypes.c_double), _ptr(kr, ctypes.c_int8), int(bits), int(rule), int(top_k),
        _ptr(thr, ctypes.c_double))
    if rc:
        raise ValueError(f"ffd_oracle_decode: error {rc}")
    return DecodeResult(out, lse, kept, bm, mt, thr)


def dense(q, k_cache, v_cache, block_table, seq_lens, max_blocks, *, sm_scale=None, units=None):
    """Dense softmax attention over every valid token.  Returns (out f64 [B,Hq,D], lse f64 [B,Hq])."""
    q = _u16(q)
    k_cache = _u16(k_cache)
    v_cache = _u16(v_cache)
    B, Hq, D = q.shape
    P, Hkv, BLK, _ = k_cache.shape
    seq_lens = _i32(seq_lens)
    block_table = _i32(block_table)
    if sm_scale is None:
        sm_scale = 1.0 / math.sqrt(D)
    out = np.zeros((B, Hq, D), dtype=np.float64)
    lse = np.full((B, Hq), np.nan, dtype=np.float64)
    u, nu = _units(units)
    rc = lib().ffd_oracle_dense(
        _ptr(q, ctypes.c_uint16), _ptr(k_cache, ctypes.c_uint16), _ptr(v_cache, ctypes.c_uint16),
        _ptr(block_table, ctypes.c_int32), _ptr(seq_lens, ctypes.c_int32), B, Hq, Hkv, D, BLK, int(max_blocks), P,
        ctypes.c_double(sm_scale), _ptr(u, ctypes.c_int32), nu, _ptr(out, ctypes.c_double),
        _ptr(lse, ctypes.c_double))
    if rc:
        raise ValueError(f"ffd_oracle_dense: error {rc}")
    return out, lse
