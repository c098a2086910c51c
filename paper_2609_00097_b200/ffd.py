"""Thin ctypes binding over the C ABI declared in ``include/ffd.h``.

Argument marshalling only: every step of the path runs in the CUDA library.  PyTorch supplies device memory
and streams.  The library is loaded from ``libffd_b200.so`` next to this file; if it is missing the import of
any entry point raises (there is no CPU fallback).
"""
from __future__ import annotations

import ctypes
import math
import os
from dataclasses import dataclass

import torch

from .build import LIB_PATH

FFD_OK = 0
STATUS_NAMES = {0: "FFD_OK", 1: "FFD_ERR_NULL", 2: "FFD_ERR_SHAPE", 3: "FFD_ERR_UNSUPPORTED", 4: "FFD_ERR_ALIGN",
                5: "FFD_ERR_WORKSPACE", 6: "FFD_ERR_DELTA", 7: "FFD_ERR_CUDA", 8: "FFD_ERR_DEVICE_STATUS",
                9: "FFD_ERR_STATIC_LIMIT"}
STATIC_SCRATCH_BYTES = 8 << 20
DEV_BAD_PAGE = 1
DEV_BAD_SEQ_LEN = 2
DEV_TIMEOUT = 4
DEV_RANGE = 8
DEV_BAD_WORKSPACE = 16

EXPORTS = ["ffd_status_string", "ffd_workspace_bytes", "ffd_workspace_init", "ffd_quantize_keys", "ffd_decode",
           "ffd_decode_dense", "ffd_unpack_codes", "ffd_read_device_status", "ffd_profile_events", "ffd_decode_static",
           "ffd_append_kv", "ffd_append_decode", "ffd_quantize_residual", "ffd_decode_residual", "ffd_workspace_bytes_residual",
           "ffd_quantize_keys_residual", "ffd_append_kv_residual", "ffd_decode_select"]

RULE_PSEUDO_MAX, RULE_GLOBAL_MAX, RULE_RUNNING_MAX, RULE_TOP_K = 0, 1, 2, 3


class FfdError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({status_string(status)})")


class ffd_config(ctypes.Structure):
    _fields_ = [("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("block_tokens", ctypes.c_int32), ("quant_bits", ctypes.c_int32), ("n_sink_blocks", ctypes.c_int32),
                ("n_local_blocks", ctypes.c_int32), ("sm_scale", ctypes.c_float), ("out_dtype", ctypes.c_int32)]


@dataclass
class Config:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int = 128
    block_tokens: int = 64
    quant_bits: int = 2
    n_sink_blocks: int = 1
    n_local_blocks: int = 16
    sm_scale: float = 0.0          # 0 -> 1/sqrt(head_dim)
    out_dtype: int = 1             # 0 bf16, 1 fp32

    def c(self) -> ffd_config:
        return ffd_config(self.num_q_heads, self.num_kv_heads, self.head_dim, self.block_tokens, self.quant_bits,
                          self.n_sink_blocks, self.n_local_blocks, self.sm_scale, self.out_dtype)


_lib = None
_vp = ctypes.c_void_p


def load_library() -> ctypes.CDLL:
    """Load the CUDA library; fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_00097_b200.build` "
                              "(there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        cfgp = ctypes.POINTER(ffd_config)
        i32 = ctypes.c_int32
        lib.ffd_status_string.restype = ctypes.c_char_p
        lib.ffd_status_string.argtypes = [ctypes.c_int]
        lib.ffd_workspace_bytes.argtypes = [cfgp, i32, i32, ctypes.POINTER(ctypes.c_size_t)]
        lib.ffd_workspace_bytes_residual.argtypes = [cfgp, i32, i32, ctypes.POINTER(ctypes.c_size_t)]
        lib.ffd_workspace_init.argtypes = [_vp, ctypes.c_size_t, _vp]
        lib.ffd_quantize_keys.argtypes = [cfgp, _vp, _vp, _vp, _vp, _vp, _vp, i32, i32, i32, _vp]
        lib.ffd_decode.argtypes = [cfgp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, i32, i32, i32, ctypes.c_float, _vp, _vp,
                                   _vp, _vp, _vp, ctypes.c_size_t, _vp]
        lib.ffd_decode_dense.argtypes = [cfgp, _vp, _vp, _vp, _vp, _vp, i32, i32, i32, _vp, _vp, _vp,
                                         ctypes.c_size_t, _vp]
        lib.ffd_unpack_codes.argtypes = [cfgp, _vp, _vp, i32, _vp]
        lib.ffd_read_device_status.argtypes = [_vp, _vp, ctypes.POINTER(ctypes.c_uint32)]
        lib.ffd_profile_events.argtypes = [_vp, _vp]
        lib.ffd_decode_static.argtypes = [cfgp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, i32, i32, i32, ctypes.c_float, _vp,
                                          _vp, _vp]
        lib.ffd_append_kv.argtypes = [cfgp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, i32, i32, i32, _vp, ctypes.c_size_t,
                                      _vp]
        lib.ffd_append_decode.argtypes = [cfgp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, i32, i32, i32,
                                          ctypes.c_float, _vp, _vp, _vp, _vp, _vp, ctypes.c_size_t, _vp]
        lib.ffd_quantize_residual.argtypes = [cfgp, _vp, _vp, _vp, _vp, _vp, _vp, i32, i32, i32, _vp]
        lib.ffd_decode_residual.argtypes = lib.ffd_decode.argtypes
        lib.ffd_append_kv_residual.argtypes = [cfgp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, i32, i32, i32, _vp,
                                               ctypes.c_size_t, _vp]
        lib.ffd_quantize_keys_residual.argtypes = [cfgp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, i32, i32, i32, _vp]
        for name in EXPORTS:
            if name != "ffd_status_string":
                getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().ffd_status_string(int(status)).decode()


def _p(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _check(status: int, where: str):
    if status != FFD_OK:
        raise FfdError(status, where)


def ffd_workspace_bytes(cfg: Config, batch: int, max_blocks_per_seq: int) -> int:
    n = ctypes.c_size_t(0)
    _check(load_library().ffd_workspace_bytes(ctypes.byref(cfg.c()), batch, max_blocks_per_seq, ctypes.byref(n)),
           "ffd_workspace_bytes")
    return int(n.value)


def ffd_workspace_bytes_residual(cfg: Config, batch: int, max_blocks_per_seq: int) -> int:
    n = ctypes.c_size_t(0)
    _check(load_library().ffd_workspace_bytes_residual(ctypes.byref(cfg.c()), batch, max_blocks_per_seq,
                                                       ctypes.byref(n)), "ffd_workspace_bytes_residual")
    return int(n.value)


def ffd_workspace_init(workspace, stream=None):
    _check(load_library().ffd_workspace_init(_p(workspace), workspace.numel(), _stream(stream)), "ffd_workspace_init")


def new_workspace(cfg: Config, batch: int, max_blocks_per_seq: int, device="cuda", stream=None, *,
                  residual: bool = False) -> torch.Tensor:
    """Allocate (with torch) and initialise a workspace for this geometry (``residual``: one that also serves
    ``ffd_decode_residual``)."""
    size = (ffd_workspace_bytes_residual if residual else ffd_workspace_bytes)(cfg, batch, max_blocks_per_seq)
    ws = torch.empty(size, dtype=torch.uint8, device=device)
    ffd_workspace_init(ws, stream)
    return ws


def ffd_quantize_keys(cfg: Config, k_cache, k_quant, k_scales, block_table, seq_lens, first_token=None, *,
                      max_blocks_per_seq: int, stream=None):
    num_pages = k_cache.shape[0]
    _check(load_library().ffd_quantize_keys(ctypes.byref(cfg.c()), _p(k_cache), _p(k_quant), _p(k_scales),
                                            _p(block_table), _p(seq_lens), _p(first_token), seq_lens.numel(),
                                            max_blocks_per_seq, num_pages, _stream(stream)), "ffd_quantize_keys")


def ffd_quantize_residual(cfg: Config, k_cache, k_scales, k_res, block_table, seq_lens, first_token=None, *,
                          max_blocks_per_seq: int, stream=None):
    _check(load_library().ffd_quantize_residual(ctypes.byref(cfg.c()), _p(k_cache), _p(k_scales), _p(k_res),
                                                _p(block_table), _p(seq_lens), _p(first_token), seq_lens.numel(),
                                                max_blocks_per_seq, k_cache.shape[0], _stream(stream)),
           "ffd_quantize_residual")


def ffd_quantize_keys_residual(cfg: Config, k_cache, k_quant, k_scales, k_res, block_table, seq_lens, first_token=None,
                               *, max_blocks_per_seq: int, stream=None):
    _check(load_library().ffd_quantize_keys_residual(ctypes.byref(cfg.c()), _p(k_cache), _p(k_quant), _p(k_scales),
                                                     _p(k_res), _p(block_table), _p(seq_lens), _p(first_token),
                                                     seq_lens.numel(), max_blocks_per_seq, k_cache.shape[0],
                                                     _stream(stream)), "ffd_quantize_keys_residual")


def ffd_decode_residual(cfg: Config, q, k_res, v_cache, k_quant, k_scales, block_table, seq_lens, delta: float, out, *,
                        max_blocks_per_seq: int, workspace, lse=None, kept_mask=None, block_max=None, stream=None):
    _check(load_library().ffd_decode_residual(ctypes.byref(cfg.c()), _p(q), _p(k_res), _p(v_cache), _p(k_quant),
                                              _p(k_scales), _p(block_table), _p(seq_lens), q.shape[0],
                                              max_blocks_per_seq, k_res.shape[0], ctypes.c_float(delta), _p(out),
                                              _p(lse), _p(kept_mask), _p(block_max), _p(workspace), workspace.numel(),
                                              _stream(stream)), "ffd_decode_residual")


def ffd_append_kv(cfg: Config, k_new, v_new, k_cache, v_cache, k_quant, k_scales, block_table, seq_lens, *,
                  max_blocks_per_seq: int, workspace, stream=None):
    num_pages = k_cache.shape[0]
    _check(load_library().ffd_append_kv(ctypes.byref(cfg.c()), _p(k_new), _p(v_new), _p(k_cache), _p(v_cache),
                                        _p(k_quant), _p(k_scales), _p(block_table), _p(seq_lens), seq_lens.numel(),
                                        max_blocks_per_seq, num_pages, _p(workspace),
                                        ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                        _stream(stream)), "ffd_append_kv")


def ffd_append_kv_residual(cfg: Config, k_new, v_new, k_cache, v_cache, k_quant, k_scales, k_res, block_table, seq_lens,
                           *, max_blocks_per_seq: int, workspace, stream=None):
    _check(load_library().ffd_append_kv_residual(ctypes.byref(cfg.c()), _p(k_new), _p(v_new), _p(k_cache), _p(v_cache),
                                                 _p(k_quant), _p(k_scales), _p(k_res), _p(block_table), _p(seq_lens),
                                                 seq_lens.numel(), max_blocks_per_seq, k_cache.shape[0], _p(workspace),
                                                 ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                                 _stream(stream)), "ffd_append_kv_residual")


def ffd_decode(cfg: Config, q, k_cache, v_cache, k_quant, k_scales, block_table, seq_lens, delta: float, out, *,
               max_blocks_per_seq: int, workspace, lse=None, kept_mask=None, block_max=None, stream=None):
    _check(load_library().ffd_decode(ctypes.byref(cfg.c()), _p(q), _p(k_cache), _p(v_cache), _p(k_quant),
                                     _p(k_scales), _p(block_table), _p(seq_lens), q.shape[0], max_blocks_per_seq,
                                     k_cache.shape[0], ctypes.c_float(delta), _p(out), _p(lse), _p(kept_mask),
                                     _p(block_max), _p(workspace), workspace.numel(), _stream(stream)), "ffd_decode")


def ffd_decode_select(cfg: Config, rule: int, top_k: int, q, k_cache, v_cache, k_quant, k_scales, block_table, seq_lens,
                      delta: float, out, *, max_blocks_per_seq: int, workspace, lse=None, kept_mask=None, block_max=None,
                      stream=None):
    """ffd_decode under one of the comparison selection rules (RULE_*), as scan, select and decode kernels."""
    _check(load_library().ffd_decode_select(ctypes.byref(cfg.c()), int(rule), int(top_k), _p(q), _p(k_cache), _p(v_cache),
                                            _p(k_quant), _p(k_scales), _p(block_table), _p(seq_lens), q.shape[0],
                                            max_blocks_per_seq, k_cache.shape[0], ctypes.c_float(delta), _p(out), _p(lse),
                                            _p(kept_mask), _p(block_max), _p(workspace), workspace.numel(),
                                            _stream(stream)), "ffd_decode_select")


def ffd_append_decode(cfg: Config, k_new, v_new, q, k_cache, v_cache, k_quant, k_scales, block_table, seq_lens,
                      delta: float, out, *, max_blocks_per_seq: int, workspace, lse=None, kept_mask=None,
                      block_max=None, stream=None):
    _check(load_library().ffd_append_decode(ctypes.byref(cfg.c()), _p(k_new), _p(v_new), _p(q), _p(k_cache),
                                            _p(v_cache), _p(k_quant), _p(k_scales), _p(block_table), _p(seq_lens),
                                            q.shape[0], max_blocks_per_seq, k_cache.shape[0], ctypes.c_float(delta),
                                            _p(out), _p(lse), _p(kept_mask), _p(block_max), _p(workspace),
                                            workspace.numel(), _stream(stream)), "ffd_append_decode")


def ffd_decode_static(cfg: Config, q, k_cache, v_cache, k_quant, k_scales, block_table, seq_lens, delta: float, out,
                      *, max_blocks_per_seq: int, lse=None, stream=None):
    """ffd_decode for callers that must not allocate: no workspace argument, the library's built-in scratch array
    (STATIC_SCRATCH_BYTES, shared by every call on the device) is used.  Raises FfdError(FFD_ERR_STATIC_LIMIT) when the
    geometry needs more.  Calls on one device must not overlap on the GPU; make the first call outside stream
    capture (it looks up the array's device address)."""
    _check(load_library().ffd_decode_static(ctypes.byref(cfg.c()), _p(q), _p(k_cache), _p(v_cache), _p(k_quant),
                                            _p(k_scales), _p(block_table), _p(seq_lens), q.shape[0],
                                            max_blocks_per_seq, k_cache.shape[0], ctypes.c_float(delta), _p(out),
                                            _p(lse), _stream(stream)), "ffd_decode_static")


def ffd_decode_dense(cfg: Config, q, k_cache, v_cache, block_table, seq_lens, out, *, max_blocks_per_seq: int,
                     workspace, lse=None, stream=None):
    _check(load_library().ffd_decode_dense(ctypes.byref(cfg.c()), _p(q), _p(k_cache), _p(v_cache), _p(block_table),
                                           _p(seq_lens), q.shape[0], max_blocks_per_seq, k_cache.shape[0], _p(out),
                                           _p(lse), _p(workspace), workspace.numel(), _stream(stream)),
           "ffd_decode_dense")


def ffd_unpack_codes(cfg: Config, k_quant, codes, stream=None):
    _check(load_library().ffd_unpack_codes(ctypes.byref(cfg.c()), _p(k_quant), _p(codes), k_quant.shape[0],
                                           _stream(stream)), "ffd_unpack_codes")


def ffd_read_device_status(workspace, stream=None) -> int:
    """Synchronises the stream; returns the status bits (0 = clean) and clears them on the device."""
    bits = ctypes.c_uint32(0)
    st = load_library().ffd_read_device_status(_p(workspace), _stream(stream), ctypes.byref(bits))
    if st not in (FFD_OK, 8):
        raise FfdError(st, "ffd_read_device_status")
    return int(bits.value)


def ffd_profile_events(start: "torch.cuda.Event | None", stop: "torch.cuda.Event | None"):
    """Time the fused kernel alone: events must have been created with enable_timing=True and recorded once
    (torch creates the CUDA event lazily on first record)."""
    a = None if start is None else ctypes.c_void_p(start.cuda_event)
    b = None if stop is None else ctypes.c_void_p(stop.cuda_event)
    _check(load_library().ffd_profile_events(a, b), "ffd_profile_events")
