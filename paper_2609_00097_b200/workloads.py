"""Seeded synthetic decode-attention workloads (inputs only: none of the method's arithmetic lives here).

The paper measures its kernel on Llama-3.1-8B activations and public long-context suites; none of that is
available offline, so these generators stand in for it.  Shapes follow the Llama-3-8B attention layer
(32 query heads, 8 KV heads, head_dim 128, contexts 4K-256K); structure follows what the paper reports:
attention maxima sit on sink / recent tokens (Sec. 3.2) and per-head keep ratios range from under 1 % to
100 % (App. D).  Everything is drawn on the CPU from ``torch.Generator().manual_seed(seed)`` in fp32 and
rounded to bf16.

Recipe
------
q, V ~ N(0,1).  Background K ~ N(0, sigma_bg) with sigma_bg = 1 (0.2 for "flat" heads).  ``q_dir[h]`` is
``q[h]`` scaled to unit RMS.  A *needle block* of KV head g overwrites all 64 rows of the block: row r
becomes ``amp * q_dir[g*G + r % G] + N(0, 0.3)``, so every query head of the group sees 16 aligned keys.
Needle blocks per (sequence, KV head): ``round(frac * nb)`` distinct blocks from the middle ``[1, nb-16)``,
plus block 0 as an attention sink where the config says so.  Rows past ``seq_len`` in the tail block and
all unused pages hold the finite poison value 1e4 in K and V: reading them shows up at once.

Magnitude knobs (tests of the input range; the five configurations leave them at 1): ``q_gain`` / ``k_gain``
multiply every query / key value; ``k_outliers = (count, gain)`` multiplies ``count`` seeded key channels per KV
head by ``gain`` and ``q_outliers`` does the same to the queries of those channels, as the key and query caches of
some model families show (a few channels hundreds of times larger than the rest).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

HEAD_DIM = 128
BLOCK_TOKENS = 64
POISON = 1.0e4
INF = float("inf")

# name -> recipe.  `N` is the context length (tokens); `lens` = (lo, hi) draws per-sequence lengths.
CONFIGS = {
    "C1": dict(seed=1001, B=1, Hq=8, Hkv=2, N=4096, frac=0.02, amp=3.0, sink=True, deltas=(6.0, INF)),
    "C2": dict(seed=1002, B=1, Hq=32, Hkv=8, N=32768, frac=0.01, amp=3.0, sink=True, deltas=(4.0, 6.0, 8.0)),
    "C3": dict(seed=1003, B=4, Hq=32, Hkv=8, N=131072, frac=0.005, amp=4.0, sink=True, flat_odd_heads=True,
               deltas=(6.0,)),
    "C4": dict(seed=1004, B=1, Hq=32, Hkv=8, N=262144, frac=0.005, amp=3.0, sink=False, recency_tokens=2048,
               recency_amp=2.0, deltas=(4.0, 6.0, 8.0, INF)),
    "C5": dict(seed=1005, B=16, Hq=32, Hkv=8, lens=(16384, 65536), frac=0.01, amp=3.0, sink=True, paged=True,
               spare_pages=64, deltas=(6.0,)),
}


@dataclass
class Workload:
    name: str
    B: int
    Hq: int
    Hkv: int
    seq_lens: np.ndarray               # int32 [B]
    max_blocks: int
    num_pages: int
    block_table: np.ndarray | None     # int32 [B, max_blocks]; None = identity (page = b*max_blocks + blk)
    q: torch.Tensor                    # bf16 [B, Hq, 128]
    k_cache: torch.Tensor              # bf16 [num_pages, Hkv, 64, 128]
    v_cache: torch.Tensor              # bf16 [num_pages, Hkv, 64, 128]
    deltas: tuple
    needles: dict = field(default_factory=dict)   # (b, g) -> sorted list of planted logical blocks
    flat_heads: tuple = ()
    seed: int = 0

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    def page(self, b: int, blk: int) -> int:
        return int(self.block_table[b, blk]) if self.block_table is not None else b * self.max_blocks + blk

    def num_blocks(self, b: int) -> int:
        return (int(self.seq_lens[b]) + BLOCK_TOKENS - 1) // BLOCK_TOKENS

    def bits(self, name: str) -> np.ndarray:
        """bf16 tensor -> uint16 bit patterns (for host-side consumers that take raw bits)."""
        return getattr(self, name).view(torch.int16).numpy().view(np.uint16)


def make_workload(name: str, *, variant: int = 0, N: int | None = None, B: int | None = None,
                  lens: tuple | None = None, sink: bool | None = None, tail: int = 0, q_gain: float = 1.0,
                  k_gain: float = 1.0, k_outliers: tuple | None = None, q_outliers: tuple | None = None,
                  heads: tuple | None = None) -> Workload:
    """Build config ``name`` (C1..C5).  ``N`` / ``B`` / ``lens`` shrink or reshape it for tests; ``tail`` subtracts
    that many tokens from every sequence (ragged last block); ``variant`` k adds 10*k to the seed;
    ``sink=False`` gives the "no-sink" correctness variant; the gains and outlier channels are described in the
    module's header."""
    cfg = dict(CONFIGS[name])
    seed = cfg["seed"] + 10 * variant
    gen = torch.Generator().manual_seed(seed)
    Bn = B if B is not None else cfg["B"]
    Hq, Hkv = heads if heads is not None else (cfg["Hq"], cfg["Hkv"])   # heads = (query heads, KV heads) of a variant
    G = Hq // Hkv
    use_sink = cfg["sink"] if sink is None else sink
    lens = lens if lens is not None else cfg.get("lens")
    if lens is not None and N is None:
        lo, hi = lens
        seq = torch.randint(lo, hi + 1, (Bn,), generator=gen).numpy().astype(np.int32)
    else:
        seq = np.full((Bn,), (N if N is not None else cfg["N"]), dtype=np.int32)
    seq = np.maximum(seq - tail, 1).astype(np.int32)
    nbs = (seq + BLOCK_TOKENS - 1) // BLOCK_TOKENS
    max_blocks = int(nbs.max())
    paged = bool(cfg.get("paged"))
    if paged:
        num_pages = int(nbs.sum()) + int(cfg.get("spare_pages", 0))
        perm = torch.randperm(num_pages, generator=gen).numpy().astype(np.int32)
        block_table = np.zeros((Bn, max_blocks), dtype=np.int32)
        off = 0
        for b in range(Bn):
            block_table[b, : nbs[b]] = perm[off: off + nbs[b]]
            off += int(nbs[b])
    else:
        num_pages = Bn * max_blocks
        block_table = None

    q32 = torch.randn(Bn, Hq, HEAD_DIM, generator=gen)
    q_dir = q32 / q32.pow(2).mean(dim=-1, keepdim=True).sqrt()
    # per-channel multipliers of the magnitude knobs, drawn from a generator of their own (the five configurations'
    # streams are the same with and without them)
    k_mult = torch.full((Hkv, HEAD_DIM), float(k_gain))
    q_mult = torch.full((Hq, HEAD_DIM), float(q_gain))
    side = torch.Generator().manual_seed(seed + 7777)
    for spec, which in ((k_outliers, "k"), (q_outliers, "q")):
        if spec:
            count, gain = spec
            for g in range(Hkv):
                chans = torch.randperm(HEAD_DIM, generator=side)[:count]
                if which == "k":
                    k_mult[g, chans] *= gain
                else:
                    q_mult[g * G:(g + 1) * G, chans] *= gain
    q = (q32 * q_mult.unsqueeze(0)).to(torch.bfloat16)

    k_cache = torch.full((num_pages, Hkv, BLOCK_TOKENS, HEAD_DIM), POISON, dtype=torch.bfloat16)
    v_cache = torch.full((num_pages, Hkv, BLOCK_TOKENS, HEAD_DIM), POISON, dtype=torch.bfloat16)
    flat = tuple(g for g in range(Hkv) if cfg.get("flat_odd_heads") and g % 2 == 1)
    needles: dict = {}
    rows = torch.arange(BLOCK_TOKENS)

    def aligned_rows(b, g, amp, shape_blocks):
        heads = g * G + (rows % G)                                    # [64]
        base = amp * q_dir[b, heads]                                  # [64, 128]
        noise = 0.3 * torch.randn(shape_blocks, BLOCK_TOKENS, HEAD_DIM, generator=gen)
        return base.unsqueeze(0) + noise

    for b in range(Bn):
        nb = int(nbs[b])
        pages = torch.from_numpy(block_table[b, :nb].astype(np.int64)) if paged else torch.arange(
            b * max_blocks, b * max_blocks + nb)
        K = torch.randn(nb, Hkv, BLOCK_TOKENS, HEAD_DIM, generator=gen)
        for g in flat:
            K[:, g] *= 0.2
        V = torch.randn(nb, Hkv, BLOCK_TOKENS, HEAD_DIM, generator=gen)
        for g in range(Hkv):
            planted = []
            if g not in flat:
                lo_blk, hi_blk = 1, nb - 16
                count = int(round(cfg["frac"] * nb)) if hi_blk > lo_blk else 0
                count = min(count, max(hi_blk - lo_blk, 0))
                if count > 0:
                    pick = torch.randperm(hi_blk - lo_blk, generator=gen)[:count] + lo_blk
                    planted = sorted(int(x) for x in pick)
                if use_sink:
                    planted = [0] + planted
                if planted:
                    K[planted, g] = aligned_rows(b, g, cfg["amp"], len(planted))
                if cfg.get("recency_tokens"):
                    # sink / recency bias: block 0 and the last `recency_tokens` tokens aligned to q
                    n_rec = int(math.ceil(cfg["recency_tokens"] / BLOCK_TOKENS))
                    rec = sorted(set([0] + list(range(max(nb - n_rec, 0), nb))))
                    K[rec, g] = aligned_rows(b, g, cfg["recency_amp"], len(rec))
            needles[(b, g)] = planted
        K *= k_mult.view(1, Hkv, 1, HEAD_DIM)
        valid_last = int(seq[b]) - (nb - 1) * BLOCK_TOKENS
        if valid_last < BLOCK_TOKENS:
            K[nb - 1, :, valid_last:] = POISON
            V[nb - 1, :, valid_last:] = POISON
        k_cache[pages] = K.to(torch.bfloat16)
        v_cache[pages] = V.to(torch.bfloat16)
        del K, V
    return Workload(name=name, B=Bn, Hq=Hq, Hkv=Hkv, seq_lens=seq, max_blocks=max_blocks, num_pages=num_pages,
                    block_table=block_table, q=q, k_cache=k_cache, v_cache=v_cache, deltas=tuple(cfg["deltas"]),
                    needles=needles, flat_heads=flat, seed=seed)


def repage(w: Workload, seed: int = 7, spare_pages: int = 5) -> Workload:
    """The same logical content behind a seeded random page table (paged == contiguous checks)."""
    gen = torch.Generator().manual_seed(seed)
    nbs = [w.num_blocks(b) for b in range(w.B)]
    num_pages = sum(nbs) + spare_pages
    perm = torch.randperm(num_pages, generator=gen).numpy().astype(np.int32)
    table = np.zeros((w.B, w.max_blocks), dtype=np.int32)
    k = torch.full((num_pages,) + tuple(w.k_cache.shape[1:]), POISON, dtype=torch.bfloat16)
    v = torch.full((num_pages,) + tuple(w.v_cache.shape[1:]), POISON, dtype=torch.bfloat16)
    off = 0
    for b in range(w.B):
        for blk in range(nbs[b]):
            table[b, blk] = perm[off]
            k[perm[off]] = w.k_cache[w.page(b, blk)]
            v[perm[off]] = w.v_cache[w.page(b, blk)]
            off += 1
    return Workload(name=w.name + "-paged", B=w.B, Hq=w.Hq, Hkv=w.Hkv, seq_lens=w.seq_lens.copy(),
                    max_blocks=w.max_blocks, num_pages=num_pages, block_table=table, q=w.q.clone(), k_cache=k,
                    v_cache=v, deltas=w.deltas, needles=dict(w.needles), flat_heads=w.flat_heads, seed=w.seed)
