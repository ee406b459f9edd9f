"""One pass of the context-encoding hot path: selection -> Phase 1 -> Phase 2.

``ContextEncoder`` owns device buffers, workspaces and the status word for one
workload shape, so that a step allocates nothing.  ``step_device`` takes inputs
already resident on the GPU.  ``step_host`` takes pinned host tensors, copies them
in, runs the same three C-ABI calls and copies every result back to pinned host
memory.  ``run_host_pipelined`` does that for a sequence of steps with two buffer
sets and three streams, so that one step's copies overlap its neighbours'
compute (PCIe is full duplex).  ``capture_step`` records a step as a CUDA graph.  All
arithmetic happens in the library's kernels.
"""
from __future__ import annotations

import torch

from . import binding
from .workloads import Workload

_INPUTS = ("ids", "Q", "K", "V", "Qq")
_OUTPUTS = ("O1", "LSE1", "O2", "LSE2", "prefix_idx")


class ContextEncoder:
    def __init__(self, w: Workload, device, phase2_splits: int = 0, slots: int = 1):
        self.w = w
        self.dev = torch.device(device)
        dev = self.dev
        B = w.n_blocks
        self.status = binding.new_status(dev)
        self.ws_select = binding._workspace(
            binding.maxidf_select_workspace_bytes(w.L, w.vocab_size, w.block_size, w.chunk, w.k, w.sink), dev)
        self.ws_p1 = binding._workspace(
            binding.phase1_workspace_bytes(w.L, w.Hq, w.Hkv, w.d, w.block_size, w.prefix_total), dev)
        # Phase 2 only needs the number of retained rows: a sequence that ends inside a block is one run of L rows
        self.kv_shape = (B, w.block_size) if w.L % w.block_size == 0 else (1, w.L)
        self.n_splits = phase2_splits or binding.phase2_choose_splits(w.nq, *self.kv_shape, w.Hq, w.Hkv, w.d)
        self.ws_p2 = binding._workspace(
            binding.phase2_workspace_bytes(w.nq, *self.kv_shape, w.Hq, w.Hkv, w.d, self.n_splits), dev)
        self.slots = [self._new_slot() for _ in range(slots)]

    def _new_slot(self):
        """Device-side inputs and outputs of one step in flight."""
        w, dev, bf = self.w, self.dev, torch.bfloat16
        B = w.n_blocks
        return dict(
            ids=torch.empty(w.L, dtype=torch.int32, device=dev),
            Q=torch.empty(w.L, w.Hq, w.d, dtype=bf, device=dev), K=torch.empty(w.L, w.Hkv, w.d, dtype=bf, device=dev),
            V=torch.empty(w.L, w.Hkv, w.d, dtype=bf, device=dev), Qq=torch.empty(w.nq, w.Hq, w.d, dtype=bf, device=dev),
            O1=torch.empty(w.L, w.Hq, w.d, dtype=bf, device=dev),
            LSE1=torch.empty(w.L, w.Hq, dtype=torch.float32, device=dev),
            O2=torch.empty(w.nq, w.Hq, w.d, dtype=bf, device=dev),
            LSE2=torch.empty(w.nq, w.Hq, dtype=torch.float32, device=dev),
            sel=(torch.empty(B * w.k + 4, dtype=torch.int32, device=dev),
                 torch.empty(w.prefix_total + 4, dtype=torch.int32, device=dev),
                 torch.empty(max(B, 1), dtype=torch.int32, device=dev)),
        )

    # ---- the hot path -------------------------------------------------------------------
    def step_device(self, ids, Q, K, V, Qq, record=None, slot=None):
        """Run selection, Phase 1 and Phase 2 on device tensors; outputs land in ``slot``
        (default: slot 0).  ``record``: optional list of four CUDA events recorded before,
        between and after the three calls."""
        w = self.w
        slot = self.slots[0] if slot is None else slot
        if record:
            record[0].record()
        sel = binding.pulsar_maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink,
                                           workspace=self.ws_select, status=self.status, out=slot["sel"])
        if record:
            record[1].record()
        O1, LSE1, K_ret, V_ret = binding.pulsar_phase1_attn(
            Q, K, V, w.block_size, sel["prefix_idx"], sel["prefix_len"], out=slot["O1"], lse_out=slot["LSE1"],
            workspace=self.ws_p1, status=self.status)
        if record:
            record[2].record()
        O2, LSE2 = binding.pulsar_phase2_attn(Qq, K_ret, V_ret, *self.kv_shape, n_splits=self.n_splits,
                                              out=slot["O2"], lse_out=slot["LSE2"], workspace=self.ws_p2,
                                              status=self.status)
        if record:
            record[3].record()
        return dict(sel=sel, O1=O1, LSE1=LSE1, O2=O2, LSE2=LSE2, prefix_idx=sel["prefix_idx"])

    def capture_step(self, slot_index: int = 0):
        """The three calls of a step captured once as a CUDA graph on the slot's own device buffers
        (fill ``slots[i]["ids" | "Q" | "K" | "V" | "Qq"]``, then ``graph.replay()``): one launch from
        the host instead of nine, which matters when a step is shorter than the host's launch cadence.
        Returns (graph, results); the results are the slot's output tensors."""
        slot = self.slots[slot_index]
        args = (slot["ids"], slot["Q"], slot["K"], slot["V"], slot["Qq"])
        side = torch.cuda.Stream(device=self.dev)                 # a first run outside the capture: library
        side.wait_stream(torch.cuda.current_stream(self.dev))     # load, kernel attributes, driver entry point
        with torch.cuda.stream(side):
            self.step_device(*args, slot=slot)
        torch.cuda.current_stream(self.dev).wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            res = self.step_device(*args, slot=slot)
        return graph, res

    def host_buffers(self):
        """Pinned host buffers for the host-side entry points: inputs and outputs."""
        w = self.w
        pin = dict(pin_memory=True)
        bf = torch.bfloat16
        return dict(
            ids=torch.empty(w.L, dtype=torch.int32, **pin),
            Q=torch.empty(w.L, w.Hq, w.d, dtype=bf, **pin), K=torch.empty(w.L, w.Hkv, w.d, dtype=bf, **pin),
            V=torch.empty(w.L, w.Hkv, w.d, dtype=bf, **pin), Qq=torch.empty(w.nq, w.Hq, w.d, dtype=bf, **pin),
            O1=torch.empty(w.L, w.Hq, w.d, dtype=bf, **pin), LSE1=torch.empty(w.L, w.Hq, dtype=torch.float32, **pin),
            O2=torch.empty(w.nq, w.Hq, w.d, dtype=bf, **pin), LSE2=torch.empty(w.nq, w.Hq, dtype=torch.float32, **pin),
            prefix_idx=torch.empty(w.prefix_total, dtype=torch.int32, **pin),
        )

    @staticmethod
    def _copy_in(slot, h):
        n = 0
        for name in _INPUTS:
            slot[name].copy_(h[name], non_blocking=True)
            n += slot[name].numel() * slot[name].element_size()
        return n

    @staticmethod
    def _copy_out(res, h):
        n = 0
        for name in _OUTPUTS:
            h[name].copy_(res[name], non_blocking=True)
            n += res[name].numel() * res[name].element_size()
        return n

    def step_host(self, h):
        """One step, everything in order on the current stream: inputs from pinned host memory,
        results back to pinned host memory.  Returns (bytes host->device, bytes device->host)."""
        slot = self.slots[0]
        h2d = self._copy_in(slot, h)
        res = self.step_device(slot["ids"], slot["Q"], slot["K"], slot["V"], slot["Qq"], slot=slot)
        return h2d, self._copy_out(res, h)

    def run_host_pipelined(self, h_in, h_out, steps: int):
        """``steps`` steps from the pinned inputs ``h_in`` (read only) with results written to the
        pinned output sets ``h_out`` (one per slot, used in turn).  Copies in, compute and copies
        out run on three streams; a slot is reused only after its previous results have left.
        The caller synchronises.  Returns (bytes host->device, bytes device->host) per step."""
        assert len(self.slots) >= 2 and len(h_out) >= len(self.slots)
        cur = torch.cuda.current_stream()
        if not hasattr(self, "_streams"):
            self._streams = [torch.cuda.Stream(device=self.dev) for _ in range(3)]
        s_in, s_run, s_out = self._streams
        start = torch.cuda.Event()
        start.record(cur)
        for s in self._streams:
            s.wait_event(start)
        n = len(self.slots)
        ran = [None] * n          # compute finished with the slot's inputs
        left = [None] * n         # results of the slot copied out
        h2d = d2h = 0
        for i in range(steps):
            slot = self.slots[i % n]
            with torch.cuda.stream(s_in):
                if ran[i % n] is not None:
                    s_in.wait_event(ran[i % n])
                h2d = self._copy_in(slot, h_in)
                arrived = torch.cuda.Event()
                arrived.record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(arrived)
                if left[i % n] is not None:
                    s_run.wait_event(left[i % n])
                res = self.step_device(slot["ids"], slot["Q"], slot["K"], slot["V"], slot["Qq"], slot=slot)
                ran[i % n] = torch.cuda.Event()
                ran[i % n].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ran[i % n])
                d2h = self._copy_out(res, h_out[i % n])
                left[i % n] = torch.cuda.Event()
                left[i % n].record(s_out)
        for s in self._streams:
            done = torch.cuda.Event()
            done.record(s)
            cur.wait_event(done)
        return h2d, d2h
