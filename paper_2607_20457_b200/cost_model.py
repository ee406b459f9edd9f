"""Work counts for the Pulsar context-encoding path (host arithmetic only).

Two models live here.  ``paper_*`` restates the analytical per-layer model
behind the paper's Table 6 (dense-square cost in the assembled length n,
Eq. 14).  ``phase1_pairs`` / ``phase1_flops`` / ``phase2_*`` count what this
library's kernels actually have to compute: block rows only, the causal half
of the block triangle, the prefix fully visible.
"""
from __future__ import annotations

# Llama-3.1-8B widths behind the paper's per-token constants: Q 4096, K 1024,
# V 1024, O 4096 (Table 6: FLOPs = 10240 n^2, activation = n * 10240 * 2 bytes).
PAPER_WIDTH = 4096 + 1024 + 1024 + 4096


def paper_input_len(L: int, B: int, sink: int, sigma: int, i: int) -> int:
    """n_i = L/B + s_sink + i*sigma (Eq. 14); n_0 = L/B."""
    return L // B if i == 0 else L // B + sink + i * sigma


def paper_flops(n: int) -> int:
    """Table 6's Phase-1 FLOPs per layer for an assembled length n."""
    return PAPER_WIDTH * n * n


def paper_activation_bytes(n: int) -> int:
    """Table 6's peak activation bytes per layer (Q+K+V+O in bf16)."""
    return PAPER_WIDTH * 2 * n


def prefix_lens(n_blocks: int, sink: int, sigma: int):
    return [0] + [sink + i * sigma for i in range(1, n_blocks)]


def phase1_pairs(block_size: int, prefix_len) -> int:
    """(query, key) pairs per head: each block row sees its prefix and the causal
    part of its own block."""
    nb = block_size
    return sum(nb * int(p) + nb * (nb + 1) // 2 for p in prefix_len)


def phase1_flops(block_size: int, prefix_len, Hq: int, d: int) -> int:
    """Two contractions (QK^T and PV), 2*d flops each per pair and head."""
    return 4 * d * Hq * phase1_pairs(block_size, prefix_len)


def phase1_hbm_bytes(L: int, Hq: int, Hkv: int, d: int) -> int:
    """Q, K, V read once, O written once (bf16), LSE written (fp32)."""
    return L * (Hq + 2 * Hkv) * d * 2 + L * Hq * d * 2 + L * Hq * 4


def phase2_flops(nq: int, L: int, Hq: int, d: int) -> int:
    return 4 * d * Hq * nq * L


def phase2_hbm_bytes(nq: int, L: int, Hq: int, Hkv: int, d: int, n_splits: int = 0) -> int:
    """K and V streamed once, Q read, O and LSE written; plus fp32 partials
    written then read when the KV range is split ``n_splits`` ways."""
    kv = 2 * L * Hkv * d * 2
    qo = 2 * nq * Hq * d * 2 + nq * Hq * 4
    part = 2 * n_splits * nq * Hq * (d + 1) * 4
    return kv + qo + part


def select_bytes(L: int, vocab_size: int, n_blocks: int, prefix_total: int, k: int) -> int:
    """ids read twice (presence pass, scoring pass), presence bitmaps written and
    read, df table written and read, outputs."""
    bitmap = n_blocks * ((vocab_size + 31) // 32) * 4
    return 2 * 4 * L + 2 * bitmap + 2 * 4 * vocab_size + 4 * (prefix_total + n_blocks * k + n_blocks)


# ---- block-to-host mapping (Appendix J, Eq. 15) -------------------------------------------------
MAPPINGS = ("contiguous", "round_robin", "zigzag")


def block_to_host(n_blocks: int, n_hosts: int, kind: str = "zigzag"):
    """pi: logical block -> host, every host getting n_blocks / n_hosts blocks.

    ``contiguous``  host h holds blocks [h*m, (h+1)*m)
    ``round_robin`` block i goes to host i mod H
    ``zigzag``      rounds of H blocks dealt alternately forwards and backwards, so that early
                    (cheap) and late (costly) blocks meet on one host
    The paper leaves pi open (its 128K runs put two blocks on each of four hosts)."""
    if n_hosts <= 0 or n_blocks % n_hosts != 0:
        raise ValueError("n_blocks must be a positive multiple of n_hosts")
    m = n_blocks // n_hosts
    if kind == "contiguous":
        return [i // m for i in range(n_blocks)]
    if kind == "round_robin":
        return [i % n_hosts for i in range(n_blocks)]
    if kind == "zigzag":
        return [(i % n_hosts) if (i // n_hosts) % 2 == 0 else (n_hosts - 1 - i % n_hosts) for i in range(n_blocks)]
    raise ValueError(f"unknown mapping {kind!r}")


def host_costs(pi, block_cost):
    """C_h = sum of block_cost(i) over the blocks with pi(i) = h (Eq. 15)."""
    costs = [0] * (max(pi) + 1)
    for i, h in enumerate(pi):
        costs[h] += block_cost(i)
    return costs


def critical_path(pi, block_cost):
    """C_crit = max_h C_h (Eq. 15)."""
    return max(host_costs(pi, block_cost))


# ---- position ids of the Phase-2 query (Appendix E) ---------------------------------------------
def phase2_query_position_start(L: int, n_blocks: int, sink: int, sigma: int, mode: str = "sparse") -> int:
    """First position id of the query tokens.  Sparse mode keeps global positions, so the query
    follows the context at L.  In contiguous mode every Phase-1 input was renumbered from 0, and the
    query starts just past the longest of them, n_{B-1} = L/B + sink + (B-1)*sigma (n_0 = L/B)."""
    if mode == "sparse":
        return L
    if mode == "contiguous":
        return max(paper_input_len(L, n_blocks, sink, sigma, i) for i in range(n_blocks))
    raise ValueError(f"unknown position mode {mode!r}")
