"""Context encoding with the logical blocks spread over several GPUs (block-to-host mapping pi,
Section 3 and Appendix J; Phase-2 exchange of Appendix H).

One process per GPU.  Every rank holds Q, K, V of its own blocks only (ascending logical order,
back to back) and the replicated token ids.  Two exchanges, both one all-gather into local
memory followed by a kernel that reads only local memory:

* Phase 1: each rank packs the summary K/V rows of its blocks (``pulsar_pack_summary_kv``); the
  packed buffers are all-gathered; ``pulsar_gather_kv_rows`` puts them into prefix-list order;
  ``pulsar_phase1_attn_sharded`` attends over the local blocks.
* Phase 2: each rank attends the query to its retained KV (``pulsar_phase2_attn``), merges its
  own parts into one float32 partial (``pulsar_lse_merge_strided``); the partials (o_h, l_h) are
  all-gathered and every rank merges the gathered set.  ``phase2_fused`` instead lets rank r merge
  1/H of the rows straight out of every rank's peer-mapped partial (``pulsar_lse_merge_peers``:
  the exchange and the merge in one kernel, H times fewer bytes over NVLink) and gathers the bf16
  slices.

All arithmetic is in the CUDA library; this module computes layouts on the host and calls the
collective.  ``TorchCollective`` wraps ``torch.distributed``; a test can pass any object with
the same ``all_gather`` method (e.g. one that concatenates buffers of ranks run in turn).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from . import cost_model


@dataclass(frozen=True)
class ShardLayout:
    """Host-side index arithmetic of the sharded path (no tensors on any device)."""
    n_blocks: int
    n_hosts: int
    block_size: int
    chunk: int
    k: int
    sink: int
    pi: tuple

    @staticmethod
    def make(n_blocks, n_hosts, block_size, chunk, k, sink, mapping="zigzag") -> "ShardLayout":
        pi = tuple(cost_model.block_to_host(n_blocks, n_hosts, mapping))
        return ShardLayout(n_blocks, n_hosts, block_size, chunk, k, sink, pi)

    @property
    def sigma(self) -> int:
        return self.k * self.chunk

    @property
    def n_local(self) -> int:
        return self.n_blocks // self.n_hosts

    @property
    def send_rows(self) -> int:
        """Rows each rank contributes to the prefix exchange."""
        return self.sink + self.n_local * self.sigma

    @property
    def prefix_total(self) -> int:
        return self.sink + (self.n_blocks - 1) * self.sigma

    def local_blocks(self, h: int):
        return [i for i in range(self.n_blocks) if self.pi[i] == h]

    def local_token_rows(self, h: int) -> np.ndarray:
        """Global token positions of rank h's rows, in its local order."""
        return np.concatenate([np.arange(i * self.block_size, (i + 1) * self.block_size)
                               for i in self.local_blocks(h)])

    def prefix_len_local(self, h: int) -> np.ndarray:
        return np.array([0 if i == 0 else self.sink + i * self.sigma for i in self.local_blocks(h)], np.int32)

    def row_slice(self, h: int, rows: int):
        """Rows of a [rows, d] result that rank h merges when the Phase-2 exchange is fused into the
        merge: (first row, count).  ceil(rows / H) rows per rank, the last ranks taking what is left
        (possibly nothing)."""
        per = (rows + self.n_hosts - 1) // self.n_hosts
        begin = min(h * per, rows)
        return begin, min(per, rows - begin)

    def prefix_order(self) -> np.ndarray:
        """For each position of the prefix list, its row in the all-gathered send buffers, the
        buffer of rank h holding [K rows | V rows], ``send_rows`` each (so rank h's K rows start at
        row 2*h*send_rows; V rows lie send_rows further on)."""
        slot = {}
        for h in range(self.n_hosts):
            for s, i in enumerate(self.local_blocks(h)):
                slot[i] = (h, s)
        out = np.empty(self.prefix_total, np.int64)
        h0 = self.pi[0]
        out[: self.sink] = 2 * h0 * self.send_rows + np.arange(self.sink)
        for i in range(self.n_blocks - 1):
            h, s = slot[i]
            base = 2 * h * self.send_rows + self.sink + s * self.sigma
            out[self.sink + i * self.sigma: self.sink + (i + 1) * self.sigma] = base + np.arange(self.sigma)
        return out.astype(np.int32)


class TorchCollective:
    """all_gather over a ``torch.distributed`` process group (NCCL on GPUs, gloo on CPU)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self._dist, self._group = dist, group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)

    def all_gather(self, send: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
        """``out`` (optional): a preallocated contiguous tensor of world * send.numel() elements."""
        flat = send.contiguous().view(-1)
        if out is None:
            out = torch.empty(self.world * flat.numel(), dtype=send.dtype, device=send.device)
        self._dist.all_gather_into_tensor(out.view(-1), flat, group=self._group)
        return out.view((self.world,) + tuple(send.shape))


class SingleRankCollective:
    """The all_gather of a one-rank job: the send buffer with a leading dimension of 1."""
    world, rank = 1, 0

    def all_gather(self, send: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
        return send.unsqueeze(0)


class LocalPeers:
    """Peer buffers of ranks that live in one process on one GPU (tests): a registry of the
    ranks' exchange buffers, whose device addresses every rank can read directly."""

    def __init__(self, world: int):
        self.world = world
        self.buffers = [None] * world

    def alloc(self, rank: int, nfloats: int, device) -> torch.Tensor:
        self.buffers[rank] = torch.empty(nfloats, dtype=torch.float32, device=device)
        return self.buffers[rank]

    def ptrs(self):
        return [b.data_ptr() for b in self.buffers]

    def barrier(self):
        pass                                  # the ranks run one after the other


class SymmetricMemoryPeers:
    """Peer buffers through ``torch.distributed._symmetric_memory``: every rank allocates the same
    buffer, the rendezvous maps all of them into every process.  Exercised with one rank only (no
    machine with several GPUs was available); the kernel itself is covered through ``LocalPeers``."""

    def __init__(self, group=None):
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm_mem
        self._symm, self.group = symm_mem, group if group is not None else dist.group.WORLD
        self.world = dist.get_world_size(self.group)
        self.handle = None

    def alloc(self, rank: int, nfloats: int, device) -> torch.Tensor:
        t = self._symm.empty(nfloats, dtype=torch.float32, device=device)
        self.handle = self._symm.rendezvous(t, self.group)
        return t

    def ptrs(self):
        return [int(p) for p in self.handle.buffer_ptrs]

    def barrier(self):
        self.handle.barrier()                 # a device-side barrier enqueued on the current stream


class ShardedContextEncoder:
    """One rank's part of the sharded context encoding.  ``collective`` supplies all_gather.

    Every buffer a step needs -- selection outputs and workspace, exchange buffers, Phase-1 outputs,
    Phase-2 partials, send and receive buffers, results -- is allocated here (the Phase-2 ones for
    ``nq`` query rows, by ``plan_phase2``), and with ``peers`` the peer-visible buffer is allocated
    and its rendezvous done here too: a step allocates nothing and meets no other rank outside its
    collectives.  A Phase-2 call with a different number of query rows re-plans first."""

    def __init__(self, layout: ShardLayout, rank: int, Hq: int, Hkv: int, d: int, vocab_size: int, device,
                 collective=None, nq: int | None = None, peers=None, phase2_splits: int = 0):
        from . import binding
        self.b = binding
        self.lay, self.rank, self.Hq, self.Hkv, self.d, self.V = layout, rank, Hq, Hkv, d, vocab_size
        self.dev = dev = torch.device(device)
        self.coll = collective
        self.status = binding.new_status(dev)
        self.block_ids = torch.tensor(layout.local_blocks(rank), dtype=torch.int32, device=dev)
        self.plen_local = torch.from_numpy(layout.prefix_len_local(rank)).to(dev)
        self.order = torch.from_numpy(layout.prefix_order()).to(dev)
        self.send_kv = torch.empty((2, layout.send_rows, Hkv, d), dtype=torch.bfloat16, device=dev)
        self.Kp = torch.empty((max(layout.prefix_total, 1), Hkv, d), dtype=torch.bfloat16, device=dev)
        self.Vp = torch.empty_like(self.Kp)
        L = layout.n_blocks * layout.block_size
        L_local = layout.n_local * layout.block_size
        self.ws_select = binding._workspace(binding.maxidf_select_workspace_bytes(
            L, vocab_size, layout.block_size, layout.chunk, layout.k, layout.sink), dev)
        self.sel_out = (torch.empty(layout.n_blocks * layout.k + 4, dtype=torch.int32, device=dev),
                        torch.empty(layout.prefix_total + 4, dtype=torch.int32, device=dev),
                        torch.empty(max(layout.n_blocks, 1), dtype=torch.int32, device=dev))
        self.gathered_kv = torch.empty((layout.n_hosts,) + tuple(self.send_kv.shape), dtype=torch.bfloat16, device=dev)
        self.O1 = torch.empty((L_local, Hq, d), dtype=torch.bfloat16, device=dev)
        self.LSE1 = torch.empty((L_local, Hq), dtype=torch.float32, device=dev)
        self.ws_p1 = binding._workspace(256, dev)
        self._p2 = None
        self._peers = peers
        if nq is not None:
            self.plan_phase2(nq, phase2_splits)

    def plan_phase2(self, nq: int, n_splits: int = 0):
        """Allocates what Phase 2 needs for ``nq`` query rows; with peers, also the peer-visible
        buffer (all ranks must call this together: the rendezvous is a collective)."""
        lay, dev, rows = self.lay, self.dev, nq * self.Hq
        J = n_splits or self.b.phase2_choose_splits(nq, lay.n_local, lay.block_size, self.Hq, self.Hkv, self.d)
        per = (rows + lay.n_hosts - 1) // lay.n_hosts
        _, n_mine = self.row_slice(nq)
        p = dict(nq=nq, J=J,
                 pO=torch.empty((J, nq, self.Hq, self.d), dtype=torch.float32, device=dev),
                 pL=torch.empty((J, nq, self.Hq), dtype=torch.float32, device=dev),
                 ws=self.b._workspace(256, dev),
                 O_local=torch.empty((nq, self.Hq, self.d), dtype=torch.bfloat16, device=dev),
                 L_local=torch.empty((nq, self.Hq), dtype=torch.float32, device=dev),
                 send=torch.empty(self.partial_stride(nq), dtype=torch.float32, device=dev),
                 gathered=torch.empty((lay.n_hosts, self.partial_stride(nq)), dtype=torch.float32, device=dev),
                 O=torch.empty((nq, self.Hq, self.d), dtype=torch.bfloat16, device=dev),
                 LSE=torch.empty((nq, self.Hq), dtype=torch.float32, device=dev),
                 O_slice=torch.empty((max(n_mine, 1), self.d), dtype=torch.bfloat16, device=dev),
                 L_slice=torch.empty(max(n_mine, 1), dtype=torch.float32, device=dev),
                 o_pad=torch.zeros((per, self.d), dtype=torch.bfloat16, device=dev),
                 l_pad=torch.zeros(per, dtype=torch.float32, device=dev),
                 o_all=torch.empty((lay.n_hosts, per, self.d), dtype=torch.bfloat16, device=dev),
                 l_all=torch.empty((lay.n_hosts, per), dtype=torch.float32, device=dev),
                 peer_buf=None)
        if self._peers is not None:
            p["peer_buf"] = self._peers.alloc(self.rank, self.partial_stride(nq), dev)
        self._p2 = p
        return p

    def _plan_for(self, nq: int, n_splits: int = 0):
        p = self._p2
        if p is None or p["nq"] != nq or (n_splits and p["J"] != n_splits):
            p = self.plan_phase2(nq, n_splits)
        return p

    # ---- selection: replicated, no communication ------------------------------------------------
    def select(self, token_ids: torch.Tensor):
        lay = self.lay
        self.sel = self.b.pulsar_maxidf_select(token_ids, self.V, lay.block_size, lay.chunk, lay.k, lay.sink,
                                               workspace=self.ws_select, status=self.status, out=self.sel_out)
        return self.sel

    # ---- Phase 1 ---------------------------------------------------------------------------------
    def phase1_pack(self, K: torch.Tensor, V: torch.Tensor) -> torch.Tensor:
        lay = self.lay
        self.b.pulsar_pack_summary_kv(K, V, lay.block_size, self.sel["sel_chunks"], self.block_ids, lay.n_blocks,
                                      lay.chunk, lay.k, lay.sink, self.send_kv[0], self.send_kv[1],
                                      status=self.status)
        return self.send_kv

    def phase1_finish(self, gathered: torch.Tensor, Q, K, V, softmax_scale: float = 0.0):
        """gathered: [H, 2, send_rows, Hkv, d] bf16 in local memory."""
        lay = self.lay
        if lay.prefix_total > 0:
            rows = gathered.reshape(-1, self.Hkv, self.d)
            n = rows.shape[0] - lay.send_rows
            self.b.pulsar_gather_kv_rows(rows[:n], rows[lay.send_rows:], self.order, self.Kp[: lay.prefix_total],
                                         self.Vp[: lay.prefix_total], status=self.status)
            Kp, Vp = self.Kp[: lay.prefix_total], self.Vp[: lay.prefix_total]
        else:
            Kp = Vp = None
        return self.b.pulsar_phase1_attn_sharded(Q, K, V, lay.block_size, Kp, Vp, self.plen_local,
                                                 softmax_scale=softmax_scale, out=self.O1, lse_out=self.LSE1,
                                                 workspace=self.ws_p1, status=self.status)

    def phase1(self, Q, K, V, softmax_scale: float = 0.0):
        gathered = self._all_gather(self.phase1_pack(K, V), self.gathered_kv)
        return self.phase1_finish(gathered, Q, K, V, softmax_scale)

    def _all_gather(self, send, out):
        """The collective's all_gather into a preallocated buffer where it takes one."""
        try:
            return self.coll.all_gather(send, out=out)
        except TypeError:                      # a test collective with the one-argument form
            return self.coll.all_gather(send)

    # ---- Phase 2 ---------------------------------------------------------------------------------
    def partial_stride(self, nq: int) -> int:
        """Floats per rank in the Phase-2 exchange: [nq*Hq*d outputs | nq*Hq LSE], padded to 4."""
        rows = nq * self.Hq
        return (rows * (self.d + 1) + 3) // 4 * 4

    def phase2_local(self, Qq, K, V, softmax_scale: float = 0.0, n_splits: int = 0) -> torch.Tensor:
        """(o_h, l_h) of this rank's retained KV as one float32 buffer."""
        return self._phase2_local(Qq, K, V, softmax_scale, n_splits, into_peer_buffer=False)

    def _phase2_local(self, Qq, K, V, softmax_scale, n_splits, into_peer_buffer: bool):
        lay = self.lay
        nq = Qq.shape[0]
        rows = nq * self.Hq
        p = self._plan_for(nq, n_splits)
        J, pO, pL = p["J"], p["pO"], p["pL"]
        self.b.pulsar_phase2_attn(Qq, K, V, lay.n_local, lay.block_size, softmax_scale, n_splits=J,
                                  partials=(pO, pL), out=p["O_local"], lse_out=p["L_local"], workspace=p["ws"],
                                  status=self.status)
        send = p["peer_buf"] if into_peer_buffer else p["send"]
        self.b.pulsar_lse_merge_strided(pO.view(-1), pL.view(-1), J, rows * self.d, rows, rows, self.d,
                                        send[: rows * self.d].view(rows, self.d), send[rows * self.d:])
        return send

    def phase2_finish(self, gathered: torch.Tensor, nq: int):
        """gathered: [H, partial_stride] float32 in local memory -> (O bf16 [nq,Hq,d], LSE f32 [nq,Hq])."""
        rows = nq * self.Hq
        stride = self.partial_stride(nq)
        flat = gathered.reshape(-1)
        p = self._plan_for(nq)
        O, LSE = p["O"], p["LSE"]
        self.b.pulsar_lse_merge_strided(flat, flat[rows * self.d:], gathered.shape[0], stride, stride, rows, self.d,
                                        O.view(rows, self.d), LSE.view(rows))
        return O, LSE

    # ---- Phase 2 with the exchange fused into the merge (each rank reduces 1/H of the rows) --------
    def row_slice(self, nq: int):
        """Rows of the [nq*Hq, d] result this rank merges: (first row, count)."""
        return self.lay.row_slice(self.rank, nq * self.Hq)

    def phase2_local_into(self, peers, Qq, K, V, softmax_scale: float = 0.0, n_splits: int = 0):
        """As phase2_local, with (o_h, l_h) written to this rank's peer-visible buffer."""
        if self._peers is not peers:           # first use with these peers: allocate and meet (a collective)
            self._peers = peers
            self._p2 = None
        return self._phase2_local(Qq, K, V, softmax_scale, n_splits, into_peer_buffer=True)

    def phase2_merge_slice(self, peers, nq: int):
        """This rank's slice of the merged result, read from every rank's buffer in place
        (``pulsar_lse_merge_peers``).  Call after ``peers.barrier()``; returns (O bf16 [n,d], LSE [n],
        first row)."""
        rows = nq * self.Hq
        begin, n = self.row_slice(nq)
        p = self._plan_for(nq)
        O, LSE = p["O_slice"], p["L_slice"]
        if n > 0:
            self.b.pulsar_lse_merge_peers(peers.ptrs(), rows, begin, n, self.d, O, LSE)
        return O[:n], LSE[:n], begin

    def phase2_fused(self, peers, Qq, K, V, softmax_scale: float = 0.0, n_splits: int = 0):
        """Phase 2 with the partial exchange fused into the merge; the bf16 slices are then gathered
        with the collective so that every rank holds the whole result."""
        nq = Qq.shape[0]
        rows = nq * self.Hq
        self.phase2_local_into(peers, Qq, K, V, softmax_scale, n_splits)
        peers.barrier()                                     # stream-ordered: every buffer is complete before it is read
        O, LSE, _ = self.phase2_merge_slice(peers, nq)
        p = self._p2
        o_pad, l_pad = p["o_pad"], p["l_pad"]                # padded to ceil(rows / H) rows; the padding stays zero
        o_pad[: O.shape[0]].copy_(O)
        l_pad[: LSE.shape[0]].copy_(LSE)
        Oall = self._all_gather(o_pad, p["o_all"]).reshape(-1, self.d)[:rows].view(nq, self.Hq, self.d)
        Lall = self._all_gather(l_pad, p["l_all"]).reshape(-1)[:rows].view(nq, self.Hq)
        peers.barrier()                                     # nobody overwrites its buffer while others still read
        return Oall, Lall

    def phase2(self, Qq, K, V, softmax_scale: float = 0.0, n_splits: int = 0):
        send = self.phase2_local(Qq, K, V, softmax_scale, n_splits)
        return self.phase2_finish(self._all_gather(send, self._p2["gathered"]), Qq.shape[0])
