"""Seeded synthetic inputs for the Pulsar context-encoding path.

These stand in for the RULER-shaped Llama-3.1-8B workloads the paper measures
on (its data and weights are not available here): token ids follow a finite
Zipf law over the vocabulary, Q/K/V are N(0,1) rounded to bf16.  The module
only draws inputs; it contains none of the method's arithmetic, so the CUDA
path and the CPU oracle can both be fed from it.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    """One configuration: sequence shape, selection parameters, attention shape."""
    name: str
    L: int              # context tokens
    block_size: int     # tokens per logical block (n_b)
    chunk: int          # m
    k: int              # chunks kept per block
    sink: int           # s_sink
    vocab_size: int
    Hq: int
    Hkv: int
    d: int
    nq: int             # Phase-2 query rows (batch flattened)
    zipf_s: float = 1.1
    ids_seed: int = 0
    inject_rare_frac: float = 0.0   # share of chunks that get one Zipf-tail token

    @property
    def n_blocks(self) -> int:
        return -(-self.L // self.block_size)            # the last block may be shorter

    @property
    def chunks_per_block(self) -> int:
        return -(-self.block_size // self.chunk)        # the last chunk of a block may be shorter

    @property
    def sigma(self) -> int:
        return self.k * self.chunk

    @property
    def prefix_total(self) -> int:
        return self.sink + max(self.n_blocks - 1, 0) * self.sigma


CONFIGS = {
    "tiny": Workload("tiny", 4096, 1024, 16, 4, 64, 32000, 4, 1, 64, 32),
    "16k": Workload("16k", 16384, 4096, 32, 8, 64, 128256, 32, 8, 128, 64),
    "32k": Workload("32k", 32768, 4096, 32, 8, 64, 128256, 32, 8, 128, 64, inject_rare_frac=0.10),
    "64k": Workload("64k", 65536, 8192, 32, 16, 64, 128256, 32, 8, 128, 128),
    "128k": Workload("128k", 131072, 8192, 32, 16, 64, 128256, 32, 8, 128, 512),
}
CONFIG_ORDER = ["tiny", "16k", "32k", "64k", "128k"]
# Beside the five configurations: the 32K shape with head dimension 64 (the tiny configuration is the only one of
# the five with d = 64 and is too small to time anything but launches), and the 128K shape at twice the length
# (32 blocks of 8192: the prefixes grow to 15,936 rows).
MORE_WORKLOADS = {
    "32k_d64": Workload("32k_d64", 32768, 4096, 32, 8, 64, 128256, 32, 8, 64, 64),
    "256k": Workload("256k", 262144, 8192, 32, 16, 64, 128256, 32, 8, 128, 512),
}


def zipf_ids(L: int, vocab_size: int, s: float = 1.1, seed: int = 0) -> np.ndarray:
    """L ids with p(rank r) proportional to r**-s, r = 1..V, id = r-1 (inverse CDF)."""
    r = np.arange(1, vocab_size + 1, dtype=np.float64)
    w = r ** (-s)
    cdf = np.cumsum(w) / w.sum()
    u = np.random.default_rng(seed).random(L)
    return np.searchsorted(cdf, u, side="right").clip(0, vocab_size - 1).astype(np.uint32)


def token_ids(w: Workload) -> np.ndarray:
    """The workload's token ids (uint32 [L])."""
    ids = zipf_ids(w.L, w.vocab_size, w.zipf_s, w.ids_seed)
    if w.inject_rare_frac > 0.0:
        rng = np.random.default_rng(3)
        n_chunks = w.L // w.chunk
        n_inj = int(round(w.inject_rare_frac * n_chunks))
        chunks = rng.choice(n_chunks, size=n_inj, replace=False)
        offs = rng.integers(0, w.chunk, size=n_inj)
        rare = rng.integers(w.vocab_size // 2, w.vocab_size, size=n_inj)
        ids[chunks * w.chunk + offs] = rare.astype(np.uint32)
    return ids


def needle_ids(w: Workload, needle_frac: float = 0.10, seed: int = 7) -> np.ndarray:
    """Ids that exercise top-k: a background of a few frequent ids (present in every
    block), a share of chunks carrying an id found nowhere else, and ids planted in
    exactly j blocks for j = 2..B-1 so that every score level occurs."""
    B, nb, m = w.n_blocks, w.block_size, w.chunk
    n_bg = max(2, min(64, nb // 4))
    base = zipf_ids(w.L, n_bg, w.zipf_s, seed)
    rng = np.random.default_rng(seed + 1)
    bg_chunks = -(-n_bg // m)                      # leading chunks that carry the background
    free = []
    for b in range(B):
        base[b * nb: b * nb + n_bg] = np.arange(n_bg, dtype=np.uint32)
        cs = np.arange(bg_chunks, nb // m)
        rng.shuffle(cs)
        free.append(cs.tolist())
    next_id = n_bg
    n_needle = int(round(needle_frac * (nb // m)))
    for b in range(B):
        for _ in range(min(n_needle, max(len(free[b]) - 2 * B, 0))):
            c = free[b].pop()
            base[b * nb + c * m + rng.integers(0, m)] = next_id
            next_id += 1
    for j in range(2, B):
        for _rep in range(2):
            blocks = rng.choice(B, size=j, replace=False)
            if any(not free[b] for b in blocks):
                continue
            for b in blocks:
                c = free[b].pop()
                base[b * nb + c * m + rng.integers(0, m)] = next_id
            next_id += 1
    assert next_id <= w.vocab_size
    return base


def _randn_bf16(gen: torch.Generator, rows: int, heads: int, d: int, scale: float = 1.0,
                rows_per_draw: int = 8192) -> torch.Tensor:
    out = torch.empty(rows, heads, d, dtype=torch.bfloat16)
    for r0 in range(0, rows, rows_per_draw):
        r1 = min(rows, r0 + rows_per_draw)
        x = torch.randn(r1 - r0, heads, d, generator=gen, dtype=torch.float32)
        if scale != 1.0:
            x = x * scale
        out[r0:r1] = x.to(torch.bfloat16)
    return out


def qkv(w: Workload, q_scale: float = 1.0, seed: int = 1):
    """Q [L,Hq,d], K, V [L,Hkv,d] bf16 on the CPU, N(0,1) (Q times ``q_scale``)."""
    gen = torch.Generator(device="cpu").manual_seed(seed)
    Q = _randn_bf16(gen, w.L, w.Hq, w.d, q_scale)
    K = _randn_bf16(gen, w.L, w.Hkv, w.d)
    V = _randn_bf16(gen, w.L, w.Hkv, w.d)
    return Q, K, V


def phase2_query(w: Workload, q_scale: float = 1.0, seed: int = 2, nq: int | None = None):
    """Phase-2 query rows [nq,Hq,d] bf16 on the CPU."""
    gen = torch.Generator(device="cpu").manual_seed(seed)
    return _randn_bf16(gen, w.nq if nq is None else nq, w.Hq, w.d, q_scale)


def first_k_prefix(w: Workload):
    """A valid prefix list that needs no selection run: sink + the first k chunks
    of every block but the last (what Max-IDF picks when all chunks tie)."""
    idx = list(range(w.sink))
    for b in range(w.n_blocks - 1):
        idx.extend(range(b * w.block_size, b * w.block_size + w.sigma))
    plen = [0] + [w.sink + i * w.sigma for i in range(1, w.n_blocks)]
    return np.asarray(idx, np.int32), np.asarray(plen, np.int32)


def star_anchor_prefix(w: Workload):
    """Star-Attention-style anchor: every later block is prefixed by all of block 0."""
    idx = np.arange(w.block_size, dtype=np.int32)
    plen = np.asarray([0] + [w.block_size] * (w.n_blocks - 1), np.int32)
    return idx, plen


def sample_rows(w: Workload, per_block: int = 64, seed: int = 11) -> np.ndarray:
    """A deterministic sample of query positions: the first 4 and last 4 rows of
    every block plus seeded random rows, ascending."""
    rng = np.random.default_rng(seed)
    rows = []
    for b in range(w.n_blocks):
        lo, hi = b * w.block_size, min((b + 1) * w.block_size, w.L)
        fixed = list(range(lo, min(lo + 4, hi))) + list(range(max(hi - 4, lo), hi))
        inner = np.arange(lo + 4, hi - 4)
        extra = rng.choice(inner, size=min(max(per_block - 8, 0), len(inner)), replace=False).tolist() \
            if len(inner) else []
        rows.extend(sorted(set(fixed + extra)))
    return np.asarray(rows, np.int64)


def shrink(w: Workload, **kw) -> Workload:
    """A copy of the workload with some fields replaced (for test-sized variants)."""
    return replace(w, **kw)
