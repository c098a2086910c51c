"""Device-resident copy of a synthetic workload plus the buffers one decode step needs.

A helper of the tests, ``bench.py`` and the smoke entry: it only allocates with torch and forwards to the binding's
entry points; no step of the path lives here.
"""
from __future__ import annotations

import torch

from paper_2609_00097_b200.ffd import (Config, ffd_append_decode, ffd_append_kv, ffd_append_kv_residual, ffd_decode,
                                        ffd_decode_dense, ffd_decode_residual, ffd_decode_select, ffd_quantize_keys,
                                        ffd_quantize_keys_residual, ffd_quantize_residual, ffd_unpack_codes,
                                        new_workspace)


class DeviceCache:
    def __init__(self, w, cfg: Config | None = None, device="cuda"):
        self.w = w
        self.cfg = cfg or Config(w.Hq, w.Hkv)
        self.device = device
        # q and seq_lens, the two inputs that change every step, share one allocation (q first, both 16-byte
        # aligned) so that a serving loop can bring them over with a single host-to-device copy into `step_in`
        qb = w.q.numel() * 2
        self.step_in = torch.zeros(qb + (4 * w.B + 15) // 16 * 16, dtype=torch.uint8, device=device)
        self.q = self.step_in[:qb].view(torch.bfloat16).view(w.q.shape)
        self.q.copy_(w.q)
        self.seq_lens = self.step_in[qb:qb + 4 * w.B].view(torch.int32)
        self.seq_lens.copy_(torch.from_numpy(w.seq_lens))
        self.k_cache = w.k_cache.to(device)
        self.v_cache = w.v_cache.to(device)
        self.block_table = None if w.block_table is None else torch.from_numpy(w.block_table).to(device)
        P, Hkv = w.num_pages, w.Hkv
        self.k_quant = torch.zeros(P, Hkv, 1024 * self.cfg.quant_bits, dtype=torch.uint8, device=device)
        self.k_scales = torch.zeros(P, Hkv, 128, dtype=torch.float16, device=device)
        self.workspace = new_workspace(self.cfg, w.B, w.max_blocks, device)
        odt = torch.float32 if self.cfg.out_dtype == 1 else torch.bfloat16
        self.out = torch.zeros(w.B, w.Hq, 128, dtype=odt, device=device)
        self.lse = torch.zeros(w.B, w.Hq, dtype=torch.float32, device=device)

    def quantize(self, first_token=None):
        ffd_quantize_keys(self.cfg, self.k_cache, self.k_quant, self.k_scales, self.block_table, self.seq_lens,
                          first_token, max_blocks_per_seq=self.w.max_blocks)

    def quantize_residual(self, first_token=None):
        """The 8-bit residuals of the keys (after ``quantize``); on first use allocates ``k_res`` and swaps the
        workspace for one that also holds the residual decode's score tiles."""
        if getattr(self, "k_res", None) is None:
            self.k_res = torch.zeros(self.w.num_pages, self.w.Hkv, 64, 128, dtype=torch.int8, device=self.device)
            self.workspace = new_workspace(self.cfg, self.w.B, self.w.max_blocks, self.device, residual=True)
        ffd_quantize_residual(self.cfg, self.k_cache, self.k_scales, self.k_res, self.block_table, self.seq_lens,
                              first_token, max_blocks_per_seq=self.w.max_blocks)

    def quantize_both(self, first_token=None):
        """Thumbnails and residuals in one call (one launch when ``first_token`` is given)."""
        if getattr(self, "k_res", None) is None:
            self.quantize_residual()
        ffd_quantize_keys_residual(self.cfg, self.k_cache, self.k_quant, self.k_scales, self.k_res, self.block_table,
                                   self.seq_lens, first_token, max_blocks_per_seq=self.w.max_blocks)

    def decode_residual(self, delta, kept_mask=None, block_max=None):
        ffd_decode_residual(self.cfg, self.q, self.k_res, self.v_cache, self.k_quant, self.k_scales, self.block_table,
                            self.seq_lens, delta, self.out, max_blocks_per_seq=self.w.max_blocks,
                            workspace=self.workspace, lse=self.lse, kept_mask=kept_mask, block_max=block_max)

    def append(self, k_new, v_new):
        ffd_append_kv(self.cfg, k_new, v_new, self.k_cache, self.v_cache, self.k_quant, self.k_scales,
                      self.block_table, self.seq_lens, max_blocks_per_seq=self.w.max_blocks, workspace=self.workspace)

    def append_residual(self, k_new, v_new):
        """Append one token per sequence on the 2 + 8 bit format (thumbnails and residuals of its block redone)."""
        ffd_append_kv_residual(self.cfg, k_new, v_new, self.k_cache, self.v_cache, self.k_quant, self.k_scales,
                               self.k_res, self.block_table, self.seq_lens, max_blocks_per_seq=self.w.max_blocks,
                               workspace=self.workspace)

    def append_decode(self, k_new, v_new, delta, kept_mask=None, block_max=None):
        ffd_append_decode(self.cfg, k_new, v_new, self.q, self.k_cache, self.v_cache, self.k_quant, self.k_scales,
                          self.block_table, self.seq_lens, delta, self.out, max_blocks_per_seq=self.w.max_blocks,
                          workspace=self.workspace, lse=self.lse, kept_mask=kept_mask, block_max=block_max)

    def decode(self, delta, kept_mask=None, block_max=None):
        ffd_decode(self.cfg, self.q, self.k_cache, self.v_cache, self.k_quant, self.k_scales, self.block_table,
                   self.seq_lens, delta, self.out, max_blocks_per_seq=self.w.max_blocks, workspace=self.workspace,
                   lse=self.lse, kept_mask=kept_mask, block_max=block_max)

    def decode_select(self, rule, top_k, delta, kept_mask=None, block_max=None):
        ffd_decode_select(self.cfg, rule, top_k, self.q, self.k_cache, self.v_cache, self.k_quant, self.k_scales,
                          self.block_table, self.seq_lens, delta, self.out, max_blocks_per_seq=self.w.max_blocks,
                          workspace=self.workspace, lse=self.lse, kept_mask=kept_mask, block_max=block_max)

    def dense(self):
        ffd_decode_dense(self.cfg, self.q, self.k_cache, self.v_cache, self.block_table, self.seq_lens, self.out,
                         max_blocks_per_seq=self.w.max_blocks, workspace=self.workspace, lse=self.lse)

    def canonical_codes(self):
        codes = torch.zeros(self.w.num_pages, self.w.Hkv, 64, 128, dtype=torch.uint8, device=self.device)
        ffd_unpack_codes(self.cfg, self.k_quant, codes)
        return codes
