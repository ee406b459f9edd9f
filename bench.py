#!/usr/bin/env python
"""Benchmark of the Pulsar context-encoding hot path on B200.

A step is one pass of the whole path -- Max-IDF selection, Phase-1 prefix-block
attention, Phase-2 query attention with LSE merge -- over one synthetic 128K-token
sequence with Llama-3.1-8B attention shapes (one layer).  The metric is context
tokens per second per layer.  One process per GPU; with N > 1 every rank encodes
its own sequence (independent problems, no data-path collective: weak scaling).
``--shard blocks`` instead spreads the blocks of ONE sequence over the N GPUs the way the
paper does (block-to-host mapping, two all-gathers per step: strong scaling).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 128k] [--impl reference]

Prints one JSON line on rank 0.  ``--impl reference`` times the float64 CPU oracle
on a bounded sample of the same workload instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2607_20457_b200 import cost_model as cm
from paper_2607_20457_b200 import workloads as W

METRIC = "context_tokens_per_s_per_layer"
UNIT = "tokens/s"
# Measured DRAM bytes of the dominant kernel, per workload: a small text file (JSON) written by
# `bench.py --traffic-from-ncu-csv <csv>` from an ncu capture of dram__bytes_read.sum and
# dram__bytes_write.sum of this bench command.  Absent or for another workload: traffic is null.
TRAFFIC_JSON = os.path.join(os.path.dirname(os.path.abspath(__file__)), "profiles", "phase1_attn_dram_traffic.txt")


# --------------------------------------------------------------------------------------------
# helpers
# --------------------------------------------------------------------------------------------
def load_traffic(workload: str):
    """DRAM bytes (read + write) per Phase-1 attention launch at ``workload`` from the tracked
    capture, or None."""
    try:
        rec = json.load(open(TRAFFIC_JSON)).get(workload)
        return float(rec["dram_bytes_read"] + rec["dram_bytes_write"]) if rec else None
    except (OSError, ValueError, KeyError, TypeError):
        return None


def traffic_from_ncu_csv(path: str, workload: str):
    """Reads an ncu --csv log holding dram__bytes_read.sum and dram__bytes_write.sum of the bench's
    kernels, takes the Phase-1 attention launches (the attention kernel launches with the larger
    DRAM reads: Phase 2 reads K and V once), and records their per-launch median in TRAFFIC_JSON."""
    import csv
    rows = [r for r in csv.reader(open(path, errors="replace")) if len(r) > 10]
    head = next(r for r in rows if "Metric Name" in r)
    ix = {n: head.index(n) for n in ("ID", "Kernel Name", "Metric Name", "Metric Unit", "Metric Value")}
    unit = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    per_launch = {}
    for r in rows:
        if r is head or "attn_kernel" not in r[ix["Kernel Name"]] or not r[ix["Metric Name"]].startswith("dram__bytes_"):
            continue
        val = float(r[ix["Metric Value"]].replace(",", "")) * unit.get(r[ix["Metric Unit"]], 1.0)
        per_launch.setdefault(r[ix["ID"]], {})[r[ix["Metric Name"]]] = val
    launches = [v for v in per_launch.values() if len(v) == 2]
    if not launches:
        raise SystemExit(f"{path}: no attention launches with both DRAM metrics")
    big = max(v["dram__bytes_read.sum"] for v in launches)
    p1 = [v for v in launches if v["dram__bytes_read.sum"] > 0.5 * big]
    rec = {}
    if os.path.exists(TRAFFIC_JSON):
        rec = json.load(open(TRAFFIC_JSON))
    rec[workload] = dict(kernel="attn_kernel (Phase 1)", launches=len(p1),
                         dram_bytes_read=statistics.median(v["dram__bytes_read.sum"] for v in p1),
                         dram_bytes_write=statistics.median(v["dram__bytes_write.sum"] for v in p1),
                         source=os.path.basename(path))
    json.dump(rec, open(TRAFFIC_JSON, "w"), indent=1, sort_keys=True)
    print(json.dumps(rec[workload]))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap,power.draw.instant")

    def __init__(self, device_index: int):
        self.proc = None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["unsampled"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, power, instant, reasons = [], [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
            try:                                   # power.draw is a running average; this one is not
                instant.append(float(f[7]))
            except (IndexError, ValueError):
                pass
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["unsampled"])
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), power_w_max=max(power),
                    power_w_instant_max=max(instant) if instant else None, samples=len(sm), reasons=sorted(reasons))


def dist_setup(n_gpus: int):
    """Returns (rank, world, local_rank).  Initialises NCCL only when launched with N > 1."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    return rank, world, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def rank_workload(w, rank: int):
    """The sequence a rank encodes: same shape for every rank, its own seed."""
    return W.shrink(w, ids_seed=w.ids_seed + 17 * rank)


def max_over_ranks(value: float, world: int, device) -> float:
    """The slowest rank's figure (what a whole job waits for)."""
    if world <= 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# --------------------------------------------------------------------------------------------
# CPU oracle on a bounded sample (cpu_baseline leg and --impl reference)
# --------------------------------------------------------------------------------------------
def oracle_sample(w, ids, Q, K, V, Qq, rows_per_block=40, p2_rows=20):
    """Times the float64 oracle, as it stands, on a bounded sample of the workload and scales
    the three parts to one full step by exact work counts.  Every Phase-1 / Phase-2 call of the
    oracle first widens all of K and V to float (a fixed cost that does not grow with the rows
    asked for); it is timed on its own -- a call that asks for no rows -- and counted once per
    call of the full step instead of being scaled with the rows.  Returns a dict with the timing
    and the oracle's outputs on the sample."""
    import oracle
    t0 = time.perf_counter()
    sel = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    t_sel = time.perf_counter() - t0
    pidx, plen = sel["prefix_idx"], sel["prefix_len"]
    t0 = time.perf_counter()
    oracle.phase1_attn(Q, K, V, w.block_size, pidx, plen, rows=np.zeros(0, np.int64))
    t_fixed = time.perf_counter() - t0
    rows = W.sample_rows(w, per_block=rows_per_block)
    t0 = time.perf_counter()
    O1, L1 = oracle.phase1_attn(Q, K, V, w.block_size, pidx, plen, rows=rows)
    t_p1 = time.perf_counter() - t0
    sample_pairs = int(sum(int(plen[r // w.block_size]) + (r % w.block_size) + 1 for r in rows))
    total_pairs = cm.phase1_pairs(w.block_size, plen)
    n2 = min(p2_rows, w.nq)
    q_rows = np.unique(np.linspace(0, w.nq - 1, n2).round().astype(np.int64))
    n2 = len(q_rows)
    t0 = time.perf_counter()
    O2, L2 = oracle.phase2_attn(Qq[torch.from_numpy(q_rows)].contiguous(), K, V, 1, w.L)
    t_p2 = time.perf_counter() - t0
    fixed = min(t_fixed, t_p1, t_p2)
    est_step = (t_sel + fixed + (t_p1 - fixed) * total_pairs / sample_pairs + fixed + (t_p2 - fixed) * w.nq / n2)
    return dict(
        value=w.L / est_step, seconds_measured=t_sel + t_fixed + t_p1 + t_p2, est_step_seconds=est_step,
        fixed_seconds=fixed, cores=oracle.num_threads(),
        sample=(f"selection in full ({t_sel:.3f}s); Phase 1 on {len(rows)} sampled query positions x all heads "
                f"({sample_pairs} of {total_pairs} (q,k) pairs per head, {t_p1:.2f}s); Phase 2 on {n2} of {w.nq} "
                f"query rows ({t_p2:.2f}s); each part scaled to the full step by its exact work count after taking "
                f"out the oracle's fixed cost per call (widening K and V: {fixed:.2f}s, counted once per call)"),
        outputs=dict(sel=sel, rows=rows, O1=O1, L1=L1, q_rows=q_rows, O2=O2, L2=L2))


def parity_of_last_step(slot, ref):
    """Compares the GPU results of the last timed step with the oracle's outputs on the sample the
    CPU baseline computed anyway: selection bit for bit, attention outputs element-wise
    (|dO| <= 1e-2 * max(1, |O_ref|)) and |dLSE| <= 1e-3."""
    sel_buf, pidx, plen = slot["sel"]
    sel = ref["sel"]
    n_sel, n_pref = sel["sel_chunks"].size, sel["prefix_idx"].size
    exact = (np.array_equal(sel_buf[:n_sel].cpu().numpy(), sel["sel_chunks"].reshape(-1)) and
             np.array_equal(pidx[:n_pref].cpu().numpy(), sel["prefix_idx"]) and
             np.array_equal(plen[: sel["prefix_len"].size].cpu().numpy(), sel["prefix_len"]))

    def errs(O, L, Oref, Lref):
        o = O.float().cpu().numpy().astype(np.float64)
        e = np.abs(o - Oref)
        return float(e.max()), float((e / (1e-2 * np.maximum(1.0, np.abs(Oref)))).max()), \
            float(np.abs(L.cpu().numpy().astype(np.float64) - Lref).max())
    r1 = torch.from_numpy(ref["rows"]).to(slot["O1"].device)
    r2 = torch.from_numpy(ref["q_rows"]).to(slot["O2"].device)
    d1, w1, l1 = errs(slot["O1"][r1], slot["LSE1"][r1], ref["O1"], ref["L1"])
    d2, w2, l2 = errs(slot["O2"][r2], slot["LSE2"][r2], ref["O2"], ref["L2"])
    return {"selection_exact": bool(exact), "phase1_max_abs_dO": d1, "phase1_max_abs_dLSE": l1,
            "phase2_max_abs_dO": d2, "phase2_max_abs_dLSE": l2, "phase1_rows": int(len(ref["rows"])),
            "phase2_rows": int(len(ref["q_rows"])),
            "pass": bool(exact and w1 <= 1.0 and w2 <= 1.0 and l1 <= 1e-3 and l2 <= 1e-3)}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    ids = W.token_ids(w)
    Q, K, V = W.qkv(w)
    Qq = W.phase2_query(w)
    import oracle
    oracle.build()
    times, last = [], None
    for i in range(args.warmup + args.steps):
        last = oracle_sample(w, ids, Q, K, V, Qq)      # the same sample as the GPU arm's cpu_baseline leg
        if i >= args.warmup:
            times.append(last["est_step_seconds"])
    est = statistics.mean(times)
    value = w.L / est
    line = dict(
        impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
        warmup=args.warmup, ms_per_step=est * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
        dtype="f64", data="synthetic",
        config=dict(workload=w.name, L=w.L, blocks=w.n_blocks, block_size=w.block_size, chunk=w.chunk, k=w.k,
                    sink=w.sink, Hq=w.Hq, Hkv=w.Hkv, d=w.d, phase2_query_rows=w.nq),
        cpu_baseline=dict(value=value, unit=UNIT, cores=last["cores"], kind="oracle", sample=last["sample"],
                          fixed_seconds=last["fixed_seconds"]),
        e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
        gpu_launches=0,
        note="float64 CPU oracle; each step is a bounded sample scaled to a full step by exact work counts")
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
def time_calls(fn, iters, warmup=3):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for a, b in evs:
        a.record(); fn(); b.record()
    torch.cuda.synchronize()
    ts = sorted(a.elapsed_time(b) for a, b in evs)
    return dict(median_ms=ts[len(ts) // 2], min_ms=ts[0])


def time_after_flush(call, flush, iters, warmup=3):
    """Median and minimum time of ``call`` between two events, with ``flush`` run before every
    call and outside the events (the call's launches are queued behind the flush, so host launch
    latency does not enter)."""
    for _ in range(warmup):
        flush(); call()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for a, b in evs:
        flush(); a.record(); call(); b.record()
    torch.cuda.synchronize()
    ts = sorted(a.elapsed_time(b) for a, b in evs)
    return dict(median_ms=ts[len(ts) // 2], min_ms=ts[0])


def run_gpu(args, w):
    from paper_2607_20457_b200 import binding
    from paper_2607_20457_b200.pipeline import ContextEncoder

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (B200); there is no CPU path")
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    binding.load_library()
    peaks = load_peaks()

    # every rank encodes its own sequence
    wl = rank_workload(w, rank)
    ids = W.token_ids(wl)
    Q, K, V = W.qkv(wl, seed=1 + 100 * rank)
    Qq = W.phase2_query(wl, seed=2 + 100 * rank)
    enc = ContextEncoder(wl, dev, slots=2)
    h = enc.host_buffers()
    h["ids"].copy_(torch.from_numpy(ids.view(np.int32)))
    h["Q"].copy_(Q); h["K"].copy_(K); h["V"].copy_(V); h["Qq"].copy_(Qq)
    ids_d, Q_d, K_d, V_d, Qq_d = (h[n].to(dev) for n in ("ids", "Q", "K", "V", "Qq"))

    # ---- device-resident steps -----------------------------------------------------------
    for _ in range(args.warmup):
        enc.step_device(ids_d, Q_d, K_d, V_d, Qq_d)
    torch.cuda.synchronize()
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = binding.launch_count()
    barrier(world); torch.cuda.synchronize()
    start.record()
    for i in range(args.steps):
        enc.step_device(ids_d, Q_d, K_d, V_d, Qq_d, record=marks[i])
    stop.record()
    torch.cuda.synchronize(); barrier(world)
    launches = binding.launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    dev_ms = max_over_ranks(start.elapsed_time(stop), world, dev)
    status = int(enc.status.item())
    sel_ms = statistics.mean(m[0].elapsed_time(m[1]) for m in marks)
    p1_ms = statistics.mean(m[1].elapsed_time(m[2]) for m in marks)
    p2_ms = statistics.mean(m[2].elapsed_time(m[3]) for m in marks)
    p1_all = sorted(m[1].elapsed_time(m[2]) for m in marks)
    p2_all = sorted(m[2].elapsed_time(m[3]) for m in marks)
    sel_all = sorted(m[0].elapsed_time(m[1]) for m in marks)

    # ---- end to end from pinned host buffers ---------------------------------------------
    # (a) one step at a time, everything in order on one stream (latency of a single call);
    # (b) the same steps pipelined over two buffer sets and three streams (throughput): every
    #     step still copies all of its inputs in and all of its results out inside the timed region.
    e2e_steps = max(2, min(args.steps, 5))
    h2d = d2h = 0
    for _ in range(2):
        enc.step_host(h)
    torch.cuda.synchronize(); barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        h2d, d2h = enc.step_host(h)
    e1.record()
    torch.cuda.synchronize(); barrier(world)
    e2e_serial_ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / e2e_steps

    pipe_steps = max(4, args.steps)
    h_out = [h, enc.host_buffers()]
    enc.run_host_pipelined(h, h_out, 2)
    torch.cuda.synchronize(); barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    enc.run_host_pipelined(h, h_out, pipe_steps)
    e1.record()
    torch.cuda.synchronize(); barrier(world)
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / pipe_steps
    e2e_steps_report = pipe_steps

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    ms_per_step = dev_ms / args.steps
    value = world * wl.L / (ms_per_step * 1e-3)
    plen = cm.prefix_lens(wl.n_blocks, wl.sink, wl.sigma)
    p1_flops = cm.phase1_flops(wl.block_size, plen, wl.Hq, wl.d)
    achieved_tf = p1_flops / (p1_ms * 1e-3) / 1e12
    p2_flops = cm.phase2_flops(wl.nq, wl.L, wl.Hq, wl.d)
    p2_bytes = cm.phase2_hbm_bytes(wl.nq, wl.L, wl.Hq, wl.Hkv, wl.d, enc.n_splits if enc.n_splits > 1 else 0)

    extras = {}
    if args.extras:
        extras = run_extras(binding, wl, dev, K_d, V_d, peaks)

    cpu = oracle_sample(wl, ids, Q, K, V, Qq) if args.cpu_baseline else None

    line = dict(
        metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
        ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None,
        dtype="bf16", data="synthetic",
        config=dict(workload=wl.name, L=wl.L, blocks=wl.n_blocks, block_size=wl.block_size, chunk=wl.chunk, k=wl.k,
                    sink=wl.sink, vocab=wl.vocab_size, Hq=wl.Hq, Hkv=wl.Hkv, d=wl.d, phase2_query_rows=wl.nq,
                    phase2_splits=enc.n_splits, ids="zipf(1.1)", qkv="N(0,1) bf16",
                    cache="inputs (2.5 GiB) larger than the 126 MB L2; no flush needed",
                    sequences_per_gpu=1),
        parts=dict(select_us=sel_ms * 1e3, phase1_ms=p1_ms, phase2_ms=p2_ms,
                   select_us_median=sel_all[len(sel_all) // 2] * 1e3, select_us_min=sel_all[0] * 1e3,
                   select_bytes=cm.select_bytes(wl.L, wl.vocab_size, wl.n_blocks, wl.prefix_total, wl.k),
                   phase1_ms_median=p1_all[len(p1_all) // 2], phase1_ms_min=p1_all[0],
                   phase2_ms_median=p2_all[len(p2_all) // 2], phase2_ms_min=p2_all[0],
                   phase2_tensor_floor_ms=p2_flops / (peaks["bf16_burst"] * 1e12) * 1e3,
                   phase2_hbm_floor_ms=p2_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3,
                   phase1_tokens_per_s=wl.L / (p1_ms * 1e-3),
                   phase1_tflops=achieved_tf, phase1_frac_of_spec_2250=achieved_tf / 2250.0,
                   phase1_frac_of_measured_burst=achieved_tf / peaks["bf16_burst"],
                   phase2_tflops=p2_flops / (p2_ms * 1e-3) / 1e12,
                   phase2_gbs=p2_bytes / (p2_ms * 1e-3) / 1e9,
                   phase2_bound="tensor (2048 query rows share every KV row)"),
        roofline=dict(bound="tensor", kernel="attn_kernel<128> (Phase 1)", achieved=achieved_tf,
                      peak=peaks["bf16_sustained"], unit="TFLOP/s", frac=achieved_tf / peaks["bf16_sustained"],
                      peak_source=f"{peaks['source']} sustained bf16 (kernel timed inside a long step)",
                      algorithmic_flops_per_launch=p1_flops,
                      algorithmic_hbm_bytes_per_launch=cm.phase1_hbm_bytes(wl.L, wl.Hq, wl.Hkv, wl.d),
                      frac_burst=achieved_tf / peaks["bf16_burst"], peak_burst=peaks["bf16_burst"],
                      frac_spec_2250=achieved_tf / 2250.0,
                      traffic=args.traffic_bytes if args.traffic_bytes is not None else load_traffic(wl.name),
                      timed="CUDA events around pulsar_phase1_attn (prefix gather + attention kernel)"),
        e2e=dict(value=world * wl.L / (e2e_ms * 1e-3), unit=UNIT, ms_per_step=e2e_ms,
                 h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h, steps=e2e_steps_report,
                 how="pinned host buffers; copies in, compute and copies out pipelined over two buffer sets",
                 single_call_ms=e2e_serial_ms, single_call_value=world * wl.L / (e2e_serial_ms * 1e-3)),
        gpu_launches=launches, device_status=status, clocks=clocks,
        paper_context=("paper reports up to 3.3x fewer Phase-1 FLOPs per GPU than Star Attention "
                       "(analytical, B=4, 64K, 4xA100-80GB); no absolute throughput published"),
    )
    if cpu is not None:
        line["cpu_baseline"] = dict(value=cpu["value"], unit=UNIT, cores=cpu["cores"], kind="oracle",
                                    sample=cpu["sample"], seconds_measured=cpu["seconds_measured"],
                                    fixed_seconds=cpu["fixed_seconds"])
        line["parity"] = parity_of_last_step(enc.slots[0], cpu["outputs"])
    if extras:
        line["extras"] = extras
    print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_gpu_blocks(args, w):
    """One sequence, its logical blocks spread over the ranks (the paper's own layout): selection
    replicated, the summary K/V rows all-gathered before Phase 1, the Phase-2 partials all-gathered
    before the merge.  Whole-job throughput = L / slowest rank's time."""
    from paper_2607_20457_b200 import binding
    from paper_2607_20457_b200.sharding import (ShardLayout, ShardedContextEncoder, SingleRankCollective,
                                                TorchCollective)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (B200); there is no CPU path")
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    binding.load_library()
    peaks = load_peaks()
    if w.n_blocks % world != 0:
        raise SystemExit(f"--shard blocks needs the {w.n_blocks} blocks to divide over {world} ranks")
    lay = ShardLayout.make(w.n_blocks, world, w.block_size, w.chunk, w.k, w.sink, args.mapping)
    coll = TorchCollective() if world > 1 else SingleRankCollective()
    peers = None
    if args.exchange == "fused":                      # Phase-2 partials read in place by the merge kernel
        from paper_2607_20457_b200.sharding import LocalPeers, SymmetricMemoryPeers
        peers = SymmetricMemoryPeers() if world > 1 else LocalPeers(1)
    # every buffer of a step is allocated here, and the peer buffers meet here: a step allocates nothing
    enc = ShardedContextEncoder(lay, rank, w.Hq, w.Hkv, w.d, w.vocab_size, dev, coll, nq=w.nq, peers=peers)

    # every rank generates the same sequence and keeps its own blocks (pinned host copies for e2e)
    ids = W.token_ids(w)
    Q, K, V = W.qkv(w)
    Qq = W.phase2_query(w)
    rows = torch.from_numpy(lay.local_token_rows(rank))
    host = dict(ids=torch.from_numpy(ids.view(np.int32)).pin_memory(), Q=Q[rows].pin_memory(),
                K=K[rows].pin_memory(), V=V[rows].pin_memory(), Qq=Qq.pin_memory())
    d_ = {n: t.to(dev) for n, t in host.items()}
    out_host = dict(O=torch.empty_like(host["Q"]).pin_memory(),
                    O2=torch.empty((w.nq, w.Hq, w.d), dtype=torch.bfloat16).pin_memory())

    def step(t, record=None):
        if record: record[0].record()
        enc.select(t["ids"])
        if record: record[1].record()
        O1, _ = enc.phase1(t["Q"], t["K"], t["V"])
        if record: record[2].record()
        if peers is not None:
            O2, _ = enc.phase2_fused(peers, t["Qq"], t["K"], t["V"])
        else:
            O2, _ = enc.phase2(t["Qq"], t["K"], t["V"])
        if record: record[3].record()
        return O1, O2

    for _ in range(args.warmup):
        step(d_)
    torch.cuda.synchronize()
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = binding.launch_count()
    barrier(world); torch.cuda.synchronize()
    start.record()
    for i in range(args.steps):
        step(d_, marks[i])
    stop.record()
    torch.cuda.synchronize(); barrier(world)
    launches = binding.launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    dev_ms = max_over_ranks(start.elapsed_time(stop), world, dev) / args.steps
    p1_ms = max_over_ranks(statistics.mean(m[1].elapsed_time(m[2]) for m in marks), world, dev)
    p2_ms = max_over_ranks(statistics.mean(m[2].elapsed_time(m[3]) for m in marks), world, dev)
    sel_ms = statistics.mean(m[0].elapsed_time(m[1]) for m in marks)

    # end to end: this rank's inputs from pinned host memory, its results back, every step
    e2e_steps = max(2, min(args.steps, 5))
    def host_step():
        t = {n: h.to(dev, non_blocking=True) for n, h in host.items()}
        O1, O2 = step(t)
        out_host["O"].copy_(O1, non_blocking=True)
        out_host["O2"].copy_(O2, non_blocking=True)
    host_step()
    torch.cuda.synchronize(); barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        host_step()
    e1.record()
    torch.cuda.synchronize(); barrier(world)
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / e2e_steps
    status = int(enc.status.item())
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    if rank != 0:
        return

    plen = cm.prefix_lens(w.n_blocks, w.sink, w.sigma)
    mine = lay.local_blocks(0)
    crit = cm.critical_path(lay.pi, lambda i: cm.phase1_flops(w.block_size, [plen[i]], w.Hq, w.d))
    achieved_tf = crit / (p1_ms * 1e-3) / 1e12
    nbytes = lambda ts: sum(t.numel() * t.element_size() for t in ts)
    line = dict(
        metric=METRIC, value=w.L / (dev_ms * 1e-3), unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
        ms_per_step=dev_ms, higher_is_better=True, scaling="strong", vs_baseline=None, dtype="bf16",
        data="synthetic",
        config=dict(workload=w.name, L=w.L, blocks=w.n_blocks, block_size=w.block_size, chunk=w.chunk, k=w.k,
                    sink=w.sink, vocab=w.vocab_size, Hq=w.Hq, Hkv=w.Hkv, d=w.d, phase2_query_rows=w.nq,
                    shard="blocks", mapping=args.mapping, phase2_exchange=args.exchange, blocks_per_gpu=lay.n_local, rank0_blocks=mine,
                    collectives_per_step="all_gather of summary K/V rows + all_gather of Phase-2 partials",
                    cache="inputs larger than the 126 MB L2; no flush needed"),
        parts=dict(select_us=sel_ms * 1e3, phase1_ms_slowest_rank=p1_ms, phase2_ms_slowest_rank=p2_ms,
                   phase1_exchange_bytes_per_rank=2 * lay.send_rows * w.Hkv * w.d * 2,
                   phase2_exchange_bytes_per_rank=enc.partial_stride(w.nq) * 4),
        roofline=dict(bound="tensor", kernel="attn_kernel<128> (Phase 1, costliest rank)", achieved=achieved_tf,
                      peak=peaks["bf16_sustained"], unit="TFLOP/s", frac=achieved_tf / peaks["bf16_sustained"],
                      peak_source=f"{peaks['source']} sustained bf16", algorithmic_flops_per_launch=crit,
                      traffic=None, timed="CUDA events around pack + all_gather + reorder + attention, max over ranks"),
        e2e=dict(value=w.L / (e2e_ms * 1e-3), unit=UNIT, ms_per_step=e2e_ms,
                 h2d_bytes_per_step=nbytes(host.values()), d2h_bytes_per_step=nbytes(out_host.values()),
                 steps=e2e_steps, how="per rank: pinned host buffers in, results out, one stream"),
        gpu_launches=launches, device_status=status, clocks=clocks)
    print(json.dumps(line), flush=True)


def run_extras(binding, w, dev, K_d, V_d, peaks):
    """Context measurements beside the headline: decode-shaped Phase 2 (HBM-bound) and the
    Star-anchor prefix against the Pulsar prefix through the same Phase-1 kernel (64K config)."""
    out = {}
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    flush_words = flush.view(torch.int32)

    # L2 is flushed before every timed call by writing a 512 MiB buffer and reading it back: after
    # the write alone the L2 would be full of dirty lines whose write-back (up to 126 MB) competes
    # with the call's own reads of K and V -- traffic that belongs to the flush, not to the call.
    # The time after a write-only flush is reported beside it.
    def flush_clean():
        flush.zero_()
        flush_words.sum()

    def flush_dirty():
        flush.zero_()

    how = ("L2 flushed before every call by writing a 512 MiB buffer and reading it back (clean lines); "
           "events around the call only; ms_after_write_only_flush: the same after a memset alone, whose "
           "dirty lines are written back during the call")
    for name, nq in (("phase2_decode_8x1", 8), ("phase2_decode_1x1", 1), ("phase2_decode_32x1", 32)):
        Qd = W.phase2_query(w, nq=nq).to(dev)
        J = binding.phase2_choose_splits(nq, w.n_blocks, w.block_size, w.Hq, w.Hkv, w.d)
        ws = binding._workspace(binding.phase2_workspace_bytes(nq, w.n_blocks, w.block_size, w.Hq, w.Hkv, w.d, J), dev)
        O = torch.empty_like(Qd)

        def call():
            binding.pulsar_phase2_attn(Qd, K_d, V_d, w.n_blocks, w.block_size, n_splits=J, out=O, workspace=ws)
        ms = time_after_flush(call, flush_clean, 12)["median_ms"]
        ms_dirty = time_after_flush(call, flush_dirty, 12)["median_ms"]
        # four partials per KV part while all query rows of a KV head fit a quarter tile (8 and 1 tokens)
        nbytes = cm.phase2_hbm_bytes(nq, w.L, w.Hq, w.Hkv, w.d, (4 if nq * (w.Hq // w.Hkv) <= 32 else 1) * J)
        out[name] = dict(ms=ms, splits=J, gbs=nbytes / (ms * 1e-3) / 1e9,
                         frac_of_measured_hbm=nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                         ms_after_write_only_flush=ms_dirty,
                         frac_after_write_only_flush=nbytes / (ms_dirty * 1e-3) / 1e9 / peaks["hbm_gbs"], l2=how)
    # one generation step (Algorithm 1 lines 11-16): a single new token appended to a shard of 64 rows
    cap = 256
    Kg = torch.zeros(cap, w.Hkv, w.d, dtype=torch.bfloat16, device=dev)
    Vg = torch.zeros_like(Kg)
    qn, kn, vn = (W.phase2_query(w, nq=1, seed=5).to(dev), torch.randn(1, w.Hkv, w.d, device=dev).to(torch.bfloat16),
                  torch.randn(1, w.Hkv, w.d, device=dev).to(torch.bfloat16))
    J = binding.phase2_choose_splits(1, w.n_blocks, w.block_size, w.Hq, w.Hkv, w.d)
    wsg = binding._workspace(binding.load_library().pulsar_phase2_generate_workspace_bytes(
        1, w.n_blocks, w.block_size, w.Hq, w.Hkv, w.d, J), dev)
    Og = torch.empty_like(qn)

    def gen_call():
        binding.pulsar_phase2_generate_step(qn, kn, vn, K_d, V_d, w.n_blocks, w.block_size, Kg, Vg, 64, n_splits=J,
                                            out=Og, workspace=wsg)
    ms = time_after_flush(gen_call, flush_clean, 12)["median_ms"]
    ms_dirty = time_after_flush(gen_call, flush_dirty, 12)["median_ms"]
    nbytes = cm.phase2_hbm_bytes(1, w.L, w.Hq, w.Hkv, w.d, 4 * (J + 1))
    out["phase2_generate_step_1tok"] = dict(ms=ms, context_parts=J, shard_rows=65, gbs=nbytes / (ms * 1e-3) / 1e9,
                                            frac_of_measured_hbm=nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                            ms_after_write_only_flush=ms_dirty,
                                            frac_after_write_only_flush=nbytes / (ms_dirty * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                            launches="append + attention + merge", l2=how)
    del flush_words
    del flush
    w4 = W.CONFIGS["64k"]
    Q, K, V = (t.to(dev) for t in W.qkv(w4))
    ws = binding._workspace(binding.phase1_workspace_bytes(w4.L, w4.Hq, w4.Hkv, w4.d, w4.block_size, w4.block_size), dev)
    O = torch.empty_like(Q)
    res = {}
    for tag, (pidx, plen) in (("pulsar", W.first_k_prefix(w4)), ("star_anchor", W.star_anchor_prefix(w4))):
        pi, pl = torch.from_numpy(pidx).to(dev), torch.from_numpy(plen).to(dev)
        t = time_calls(lambda: binding.pulsar_phase1_attn(Q, K, V, w4.block_size, pi, pl, out=O, workspace=ws), 5)
        fl = cm.phase1_flops(w4.block_size, plen, w4.Hq, w4.d)
        res[tag] = dict(ms=t["median_ms"], tflop=fl / 1e12, tflops=fl / (t["median_ms"] * 1e-3) / 1e12)
    # the same 64K inputs as whole assembled sequences (every token of Input_i a query, Alg. 1 l.8)
    pidx, plen = W.first_k_prefix(w4)
    cu = [0]
    rows = []
    for i in range(w4.n_blocks):
        rows += list(pidx[: plen[i]]) + list(range(i * w4.block_size, (i + 1) * w4.block_size))
        cu.append(len(rows))
    sel_rows = torch.tensor(rows, device=dev)
    Qa, Ka, Va = Q[sel_rows].contiguous(), K[sel_rows].contiguous(), V[sel_rows].contiguous()
    Oa = torch.empty_like(Qa)
    wsa = binding._workspace(256, dev)
    t = time_calls(lambda: binding.pulsar_causal_varlen_attn(Qa, Ka, Va, cu, out=Oa, workspace=wsa, want_lse=False), 5)
    pairs = sum((b - a) * (b - a + 1) // 2 for a, b in zip(cu[:-1], cu[1:]))
    fl = 4 * w4.d * w4.Hq * pairs
    res["pulsar_assembled_all_rows"] = dict(ms=t["median_ms"], rows=cu[-1], tflop=fl / 1e12,
                                            tflops=fl / (t["median_ms"] * 1e-3) / 1e12)
    # rotary embedding of the assembled 64K inputs at their sparse position ids (Appendix E): a stream
    pos = binding.pulsar_assemble_positions(torch.from_numpy(pidx).to(dev), torch.from_numpy(plen).to(dev),
                                            w4.n_blocks, w4.block_size, cu[-1], "sparse")
    t = time_calls(lambda: binding.pulsar_rope_apply_qk(Qa, Ka, pos, q_out=Oa, k_out=Ka), 10)
    rope_bytes = 2 * (Qa.numel() + Ka.numel()) * 2 + 2 * pos.numel() * 4
    out["rope_sparse_positions_64k_assembled"] = dict(
        ms=t["median_ms"], rows=cu[-1], bytes=rope_bytes, gbs=rope_bytes / (t["median_ms"] * 1e-3) / 1e9,
        frac_of_measured_hbm=rope_bytes / (t["median_ms"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
        what="Q (32 heads) and K (8 heads) of all assembled inputs, read once and written once")
    # whole steps at the small configurations, launched call by call and replayed as one CUDA graph
    from paper_2607_20457_b200.pipeline import ContextEncoder
    graph_res = {}
    for name in ("tiny", "16k"):
        ws_ = W.CONFIGS[name]
        enc_s = ContextEncoder(ws_, dev)
        sl = enc_s.slots[0]
        sl["ids"].copy_(torch.from_numpy(W.token_ids(ws_).view(np.int32)))
        for nm, t_ in zip(("Q", "K", "V"), W.qkv(ws_)):
            sl[nm].copy_(t_)
        sl["Qq"].copy_(W.phase2_query(ws_))
        eager = time_calls(lambda: enc_s.step_device(sl["ids"], sl["Q"], sl["K"], sl["V"], sl["Qq"]), 20)
        graph, _ = enc_s.capture_step()
        replay = time_calls(graph.replay, 20)
        graph_res[name] = dict(call_by_call_ms=eager["median_ms"], graph_replay_ms=replay["median_ms"])
        del graph, enc_s
    out["step_as_cuda_graph"] = graph_res
    res["flop_ratio_star_over_pulsar"] = res["star_anchor"]["tflop"] / res["pulsar"]["tflop"]
    res["time_ratio_star_over_pulsar"] = res["star_anchor"]["ms"] / res["pulsar"]["ms"]
    out["phase1_64k_prefix_comparison"] = res
    return out


def self_launch(n_gpus: int) -> int:
    """Re-runs this command line as ``n_gpus`` ranks under torch.distributed.run on this node and
    returns its exit code; rank 0 prints the JSON line."""
    import socket
    if torch.cuda.is_available() and torch.cuda.device_count() < n_gpus:
        raise SystemExit(f"--gpus {n_gpus}: this node shows {torch.cuda.device_count()} GPU(s)")
    with socket.socket() as sock:                      # a free port for the rendezvous
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="128k", choices=list(W.CONFIGS) + list(W.MORE_WORKLOADS))
    ap.add_argument("--impl", default="pulsar", choices=["pulsar", "reference"])
    ap.add_argument("--shard", default="sequences", choices=["sequences", "blocks"],
                    help="sequences: every GPU encodes its own sequence; blocks: one sequence, blocks spread over GPUs")
    ap.add_argument("--mapping", default="zigzag", choices=list(cm.MAPPINGS), help="block-to-GPU mapping for --shard blocks")
    ap.add_argument("--exchange", default="allgather", choices=["allgather", "fused"],
                    help="--shard blocks: all-gather the Phase-2 partials, or let the merge kernel read them from peers")
    ap.add_argument("--no-extras", dest="extras", action="store_false")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="DRAM bytes per Phase-1 launch from an ncu capture (reported as roofline.traffic)")
    ap.add_argument("--traffic-from-ncu-csv", default=None, metavar="CSV",
                    help="no benchmark: read an ncu --csv log of dram__bytes_read.sum,dram__bytes_write.sum taken on "
                         "this command and record the Phase-1 launch's bytes for --workload")
    args = ap.parse_args()
    if args.traffic_from_ncu_csv:
        traffic_from_ncu_csv(args.traffic_from_ncu_csv, args.workload)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "pulsar" else args.warmup
    w = W.CONFIGS.get(args.workload) or W.MORE_WORKLOADS[args.workload]
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # Started by hand with --gpus N: start the N ranks ourselves (one process per GPU, NCCL over
        # 127.0.0.1), which is what a launch under torch.distributed.run does.
        raise SystemExit(self_launch(args.gpus))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus and args.impl == "pulsar":
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch one rank per GPU "
                         f"(python -m torch.distributed.run --nproc-per-node {args.gpus} bench.py --gpus {args.gpus} ...)")
    if args.impl == "reference":
        run_reference(args, w)
        return
    if world > 1:
        args.extras = False
        args.cpu_baseline = False
    if args.shard == "blocks":
        run_gpu_blocks(args, w)
    else:
        run_gpu(args, w)


if __name__ == "__main__":
    main()
