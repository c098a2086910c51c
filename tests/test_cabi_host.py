"""Host-side checks of the C-ABI library that need no GPU: it loads, exports what include/ffd.h declares, and
rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2609_00097_b200 import build, ffd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return ffd.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ffd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ffd_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert len(names) >= 8
    for name in names:
        assert hasattr(lib, name), name
    assert names == sorted(ffd.EXPORTS)


def test_status_strings(lib):
    for code in range(10):
        assert len(ffd.status_string(code)) > 1


def test_workspace_bytes_grows_with_geometry():
    cfg = ffd.Config(32, 8)
    a = ffd.ffd_workspace_bytes(cfg, 1, 512)
    b = ffd.ffd_workspace_bytes(cfg, 4, 2048)
    assert 0 < a < b
    assert a % 256 == 0
    # the residual decode's workspace: the same plus the score tiles, whose size does not depend on the geometry
    ra, rb = ffd.ffd_workspace_bytes_residual(cfg, 1, 512), ffd.ffd_workspace_bytes_residual(cfg, 4, 2048)
    assert ra - a == rb - b == 192 * 8 * 32 * 4 * 72 * 4


def test_documented_limits_of_the_static_entry_point_are_the_computed_ones():
    """include/ffd.h quotes, for 32 query / 8 KV heads on a 148-SM GPU, the longest contexts whose workspace fits the
    built-in scratch array of ffd_decode_static; the figures must be the ones ffd_workspace_bytes gives."""
    cfg = ffd.Config(32, 8)

    def longest(batch):
        lo, hi = 1, 1 << 16
        while lo < hi:    # the workspace size is monotone in the block count
            mid = (lo + hi + 1) // 2
            if ffd.ffd_workspace_bytes(cfg, batch, mid) <= ffd.STATIC_SCRATCH_BYTES:
                lo = mid
            else:
                hi = mid - 1
        return lo * 64

    text = " ".join(open(os.path.join(ROOT, "include", "ffd.h")).read().split())
    m = re.search(r"batch 1 up to about (\d+) K tokens of context, batch 4 up to about (\d+) K, batch 16 up to about "
                  r"\* (\d+) K", text)
    assert m, "the limits sentence of ffd_decode_static has changed its wording"
    assert [int(x) for x in m.groups()] == [longest(b) // 1000 for b in (1, 4, 16)]


@pytest.mark.parametrize("field,value,status", [
    ("head_dim", 64, 3), ("block_tokens", 32, 3), ("quant_bits", 3, 3), ("quant_bits", 16, 3), ("num_kv_heads", 5, 2),
    ("num_q_heads", 40, 3), ("num_q_heads", 128, 3), ("n_local_blocks", -1, 2), ("out_dtype", 7, 3), ("sm_scale", -1.0, 2),
])
def test_bad_config_is_rejected(field, value, status):
    cfg = ffd.Config(32, 8)
    setattr(cfg, field, value)
    with pytest.raises(ffd.FfdError) as e:
        ffd.ffd_workspace_bytes(cfg, 1, 16)
    assert e.value.status == status


def test_deeper_thumbnails_are_accepted_except_where_the_format_needs_two_bits():
    for bits in (4, 8):
        cfg = ffd.Config(32, 8, quant_bits=bits)
        assert ffd.ffd_workspace_bytes(cfg, 1, 16) == ffd.ffd_workspace_bytes(ffd.Config(32, 8), 1, 16)
        with pytest.raises(ffd.FfdError) as e:     # the 2 + 8 bit key format is defined on the 2-bit thumbnails
            ffd.ffd_workspace_bytes_residual(cfg, 1, 16)
        assert e.value.status == 3


def test_six_and_eight_query_heads_per_kv_head_are_accepted_where_documented():
    for hq in (48, 64):
        cfg = ffd.Config(hq, 8)
        # two groups per KV head: the geometry of twice the KV heads
        assert ffd.ffd_workspace_bytes(cfg, 2, 64) == ffd.ffd_workspace_bytes(ffd.Config(hq, 16), 2, 64)
        with pytest.raises(ffd.FfdError) as e:
            ffd.ffd_workspace_bytes_residual(cfg, 2, 64)
        assert e.value.status == 3


def test_null_and_range_arguments_are_rejected_before_any_launch(lib):
    cfg = ffd.Config(32, 8).c()
    vp = ctypes.c_void_p
    fake = vp(0x1000)            # aligned, never dereferenced: validation fails first
    odd = vp(0x1008)
    # NULL q
    assert lib.ffd_decode(ctypes.byref(cfg), None, fake, fake, fake, fake, None, fake, 1, 16, 16,
                          ctypes.c_float(6.0), fake, None, None, None, fake, 1 << 30, None) == 1
    # negative / NaN delta
    for d in (-1.0, float("nan")):
        assert lib.ffd_decode(ctypes.byref(cfg), fake, fake, fake, fake, fake, None, fake, 1, 16, 16,
                              ctypes.c_float(d), fake, None, None, None, fake, 1 << 30, None) == 6
    # misaligned pointer
    assert lib.ffd_decode(ctypes.byref(cfg), odd, fake, fake, fake, fake, None, fake, 1, 16, 16,
                          ctypes.c_float(6.0), fake, None, None, None, fake, 1 << 30, None) == 4
    # workspace too small
    assert lib.ffd_decode(ctypes.byref(cfg), fake, fake, fake, fake, fake, None, fake, 1, 16, 16,
                          ctypes.c_float(6.0), fake, None, None, None, fake, 16, None) == 5
    # batch 0
    assert lib.ffd_decode_dense(ctypes.byref(cfg), fake, fake, fake, None, fake, 0, 16, 16, fake, None, fake,
                                1 << 30, None) == 2
    assert lib.ffd_quantize_keys(ctypes.byref(cfg), None, fake, fake, None, fake, None, 1, 16, 16, None) == 1
    assert lib.ffd_unpack_codes(ctypes.byref(cfg), fake, fake, 0, None) == 2
    # append: NULL new rows, workspace below 256 bytes, misaligned lengths
    assert lib.ffd_append_kv(ctypes.byref(cfg), None, fake, fake, fake, fake, fake, None, fake, 1, 16, 16, fake, 256,
                             None) == 1
    assert lib.ffd_append_kv(ctypes.byref(cfg), fake, fake, fake, fake, fake, fake, None, fake, 1, 16, 16, fake, 128,
                             None) == 5
    assert lib.ffd_append_kv(ctypes.byref(cfg), fake, fake, fake, fake, fake, fake, None, odd, 1, 16, 16, fake, 256,
                             None) == 4
    assert lib.ffd_append_kv_residual(ctypes.byref(cfg), fake, fake, fake, fake, fake, fake, None, None, fake, 1, 16, 16,
                                      fake, 256, None) == 1
    assert lib.ffd_append_kv_residual(ctypes.byref(cfg), fake, fake, fake, fake, fake, fake, odd, None, fake, 1, 16, 16,
                                      fake, 256, None) == 4
    # append + decode: NULL new rows; the decode's own checks behind them
    assert lib.ffd_append_decode(ctypes.byref(cfg), None, fake, fake, fake, fake, fake, fake, None, fake, 1, 16, 16,
                                 ctypes.c_float(6.0), fake, None, None, None, fake, 1 << 30, None) == 1
    assert lib.ffd_append_decode(ctypes.byref(cfg), fake, fake, fake, fake, fake, fake, fake, None, fake, 1, 16, 16,
                                 ctypes.c_float(-1.0), fake, None, None, None, fake, 1 << 30, None) == 6
    # 2 + 8 bit key format: NULL residuals, misaligned residuals, a workspace that only fits the 16-bit decode
    assert lib.ffd_quantize_residual(ctypes.byref(cfg), fake, fake, None, None, fake, None, 1, 16, 16, None) == 1
    assert lib.ffd_quantize_residual(ctypes.byref(cfg), fake, fake, odd, None, fake, None, 1, 16, 16, None) == 4
    assert lib.ffd_quantize_residual(ctypes.byref(cfg), fake, fake, fake, None, fake, None, 1, 16, 0, None) == 2
    assert lib.ffd_quantize_keys_residual(ctypes.byref(cfg), fake, fake, fake, None, None, fake, None, 1, 16, 16, None) == 1
    assert lib.ffd_quantize_keys_residual(ctypes.byref(cfg), fake, fake, fake, odd, None, fake, None, 1, 16, 16, None) == 4
    assert lib.ffd_quantize_keys_residual(ctypes.byref(cfg), None, fake, fake, fake, None, fake, None, 1, 16, 16, None) == 1
    assert lib.ffd_decode_residual(ctypes.byref(cfg), fake, None, fake, fake, fake, None, fake, 1, 16, 16,
                                   ctypes.c_float(6.0), fake, None, None, None, fake, 1 << 30, None) == 1
    assert lib.ffd_decode_residual(ctypes.byref(cfg), fake, odd, fake, fake, fake, None, fake, 1, 16, 16,
                                   ctypes.c_float(6.0), fake, None, None, None, fake, 1 << 30, None) == 4
    plain = ffd.ffd_workspace_bytes(ffd.Config(32, 8), 1, 16)
    assert lib.ffd_decode_residual(ctypes.byref(cfg), fake, fake, fake, fake, fake, None, fake, 1, 16, 16,
                                   ctypes.c_float(6.0), fake, None, None, None, fake, plain, None) == 5
    assert lib.ffd_decode_residual(ctypes.byref(cfg), fake, fake, fake, fake, fake, None, fake, 1, 16, 16,
                                   ctypes.c_float(float("nan")), fake, None, None, None, fake, 1 << 30, None) == 6
    assert lib.ffd_read_device_status(None, None, None) == 1


def test_oracle_and_cuda_paths_share_no_code():
    """The oracle imports nothing from the CUDA package and the package imports nothing from the oracle."""
    pkg = os.path.join(ROOT, "paper_2609_00097_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2609_00097_b200" not in text and "ffd.h" not in text, f
