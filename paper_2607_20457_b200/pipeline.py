"""One pass of the context-encoding hot path: selection -> Phase 1 -> Phase 2.

``ContextEncoder`` owns the device buffers, workspaces and status word for one
workload shape so that a step allocates nothing.  ``step_device`` takes inputs
already resident on the GPU; ``step_host`` takes pinned host tensors, copies them
in, runs the same three C-ABI calls and copies every result back to pinned host
memory.  All arithmetic happens inside the library's kernels.
"""
from __future__ import annotations

import torch

from . import binding
from .workloads import Workload


class ContextEncoder:
    def __init__(self, w: Workload, device, phase2_splits: int = 0):
        self.w = w
        self.dev = torch.device(device)
        dev = self.dev
        B = w.n_blocks
        bf = torch.bfloat16
        self.status = binding.new_status(dev)
        self.ws_select = binding._workspace(
            binding.maxidf_select_workspace_bytes(w.L, w.vocab_size, w.block_size, w.chunk, w.k, w.sink), dev)
        self.ws_p1 = binding._workspace(
            binding.phase1_workspace_bytes(w.L, w.Hq, w.Hkv, w.d, w.block_size, w.prefix_total), dev)
        self.n_splits = phase2_splits or binding.phase2_choose_splits(w.nq, B, w.block_size, w.Hq, w.Hkv, w.d)
        self.ws_p2 = binding._workspace(
            binding.phase2_workspace_bytes(w.nq, B, w.block_size, w.Hq, w.Hkv, w.d, self.n_splits), dev)
        # device-side inputs (used by step_host) and outputs
        self.ids = torch.empty(w.L, dtype=torch.int32, device=dev)
        self.Q = torch.empty(w.L, w.Hq, w.d, dtype=bf, device=dev)
        self.K = torch.empty(w.L, w.Hkv, w.d, dtype=bf, device=dev)
        self.V = torch.empty(w.L, w.Hkv, w.d, dtype=bf, device=dev)
        self.Qq = torch.empty(w.nq, w.Hq, w.d, dtype=bf, device=dev)
        self.O1 = torch.empty(w.L, w.Hq, w.d, dtype=bf, device=dev)
        self.O2 = torch.empty(w.nq, w.Hq, w.d, dtype=bf, device=dev)
        self.events = None

    # ---- the hot path -------------------------------------------------------------------
    def step_device(self, ids, Q, K, V, Qq, record=None):
        """Run selection, Phase 1 and Phase 2 on device tensors.  ``record``: optional list of
        four CUDA events recorded before, between and after the three calls."""
        w = self.w
        if record:
            record[0].record()
        sel = binding.pulsar_maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink,
                                           workspace=self.ws_select, status=self.status)
        if record:
            record[1].record()
        O1, LSE1, K_ret, V_ret = binding.pulsar_phase1_attn(
            Q, K, V, w.block_size, sel["prefix_idx"], sel["prefix_len"], out=self.O1,
            workspace=self.ws_p1, status=self.status)
        if record:
            record[2].record()
        O2, LSE2 = binding.pulsar_phase2_attn(Qq, K_ret, V_ret, w.n_blocks, w.block_size, n_splits=self.n_splits,
                                              out=self.O2, workspace=self.ws_p2, status=self.status)
        if record:
            record[3].record()
        return dict(sel=sel, O1=O1, LSE1=LSE1, O2=O2, LSE2=LSE2)

    def host_buffers(self):
        """Pinned host buffers for step_host: inputs and outputs."""
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

    def step_host(self, h):
        """Inputs from pinned host memory, results back to pinned host memory.  Returns
        (bytes copied host->device, bytes copied device->host)."""
        h2d = d2h = 0
        for name in ("ids", "Q", "K", "V", "Qq"):
            dst = getattr(self, name)
            dst.copy_(h[name], non_blocking=True)
            h2d += dst.numel() * dst.element_size()
        r = self.step_device(self.ids, self.Q, self.K, self.V, self.Qq)
        for name, src in (("O1", r["O1"]), ("LSE1", r["LSE1"]), ("O2", r["O2"]), ("LSE2", r["LSE2"]),
                          ("prefix_idx", r["sel"]["prefix_idx"])):
            h[name].copy_(src, non_blocking=True)
            d2h += src.numel() * src.element_size()
        return h2d, d2h
