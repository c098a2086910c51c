"""ffd_decode_static: the decode step for callers that cannot allocate device memory (a serving loop whose memory was
handed out at start-up, a plug-in without an allocator).  It must give what ffd_decode gives, call after call, although
every call reuses the same built-in scratch array and finds the previous call's leftovers in it.

This file is collected last on purpose: the entry point is an add-on, and a run that stops at the first failure
should already have exercised everything else.
"""
import numpy as np
import pytest
import torch

from paper_2609_00097_b200.workloads import make_workload
from tests.device_cache import DeviceCache

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ffd():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2609_00097_b200 import ffd as m
    m.load_library()
    return m


def test_static_scratch_decode_matches_workspace_decode_on_consecutive_calls(ffd):
    # two different workloads back to back: the second call starts from the first one's scratch contents
    runs = [make_workload("C2", N=8192, tail=5), make_workload("C5", B=3, lens=(1500, 4000))]
    for w in runs:
        dc = DeviceCache(w)
        dc.quantize()
        assert ffd.ffd_workspace_bytes(dc.cfg, w.B, w.max_blocks) <= ffd.STATIC_SCRATCH_BYTES
        for delta in (6.0, float("inf")):
            dc.decode(delta)
            assert ffd.ffd_read_device_status(dc.workspace) == 0
            want_out, want_lse = dc.out.clone(), dc.lse.clone()
            for call in range(2):   # twice in a row through the allocation-free entry point
                out = torch.full_like(dc.out, float("nan"))
                lse = torch.full_like(dc.lse, float("nan"))
                torch.cuda.synchronize()
                free_before = torch.cuda.mem_get_info()[0]
                ffd.ffd_decode_static(dc.cfg, dc.q, dc.k_cache, dc.v_cache, dc.k_quant, dc.k_scales, dc.block_table,
                                      dc.seq_lens, delta, out, max_blocks_per_seq=w.max_blocks, lse=lse)
                torch.cuda.synchronize()
                # the entry point's one promise: the device's free memory is what it was before the call (the very
                # first call of a process may still make the CUDA runtime load the kernels' module)
                if call > 0 or w is not runs[0] or delta != 6.0:
                    assert torch.cuda.mem_get_info()[0] == free_before
                # same kernels, same split geometry, fixed summation order: the tests' output tolerance is 1e-2 /
                # 1e-3 against the oracle; against the library's own path the results agree to rounding noise
                assert (out - want_out).abs().max().item() <= 1e-6
                assert (lse - want_lse).abs().max().item() <= 1e-5


def test_static_scratch_refuses_geometries_beyond_its_size(ffd):
    w = make_workload("C1")
    dc = DeviceCache(w)
    dc.quantize()
    too_many_blocks = 1 << 16          # a 4 M-token context: far beyond what the built-in array can serve
    assert ffd.ffd_workspace_bytes(dc.cfg, w.B, too_many_blocks) > ffd.STATIC_SCRATCH_BYTES
    with pytest.raises(ffd.FfdError) as e:
        # refused on the host from the sizes alone: nothing is launched and no pointer is dereferenced
        ffd.ffd_decode_static(dc.cfg, dc.q, dc.k_cache, dc.v_cache, dc.k_quant, dc.k_scales, None, dc.seq_lens, 6.0,
                              dc.out, max_blocks_per_seq=too_many_blocks)
    assert e.value.status == 9
    assert "FFD_STATIC_SCRATCH_BYTES" in str(e.value)
