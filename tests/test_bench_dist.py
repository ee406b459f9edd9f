"""Host-side logic of the multi-process bench path, run as two gloo ranks on the CPU."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # the slowest rank's time is what the job reports
    slow = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")
    # every rank encodes its own sequence: different seeds, same shape
    w = bench.rank_workload(bench.W.CONFIGS["tiny"], rank)
    ids = bench.W.token_ids(w)
    bench.barrier(world)
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump(dict(slow=slow, seed=w.ids_seed, first=int(ids[:64].sum()), L=w.L), f)
    dist.destroy_process_group()


def test_two_ranks_max_time_and_independent_sequences(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = json.load(open(tmp_path / "r0.json"))
    r1 = json.load(open(tmp_path / "r1.json"))
    assert r0["slow"] == r1["slow"] == 15.0
    assert r0["seed"] != r1["seed"] and r0["first"] != r1["first"] and r0["L"] == r1["L"]


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
    bench.barrier(1)


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["gpu_launches"] == 0


def test_gpu_arm_refuses_to_run_without_a_gpu():
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "tiny", "--steps", "1"],
                         capture_output=True, text=True, timeout=300)
    assert out.returncode != 0 and "no CPU path" in (out.stderr + out.stdout)


def test_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` started by hand (no WORLD_SIZE in the environment) launches two ranks;
    shown here with the CPU-only reference arm: one JSON line, from rank 0, reporting two ranks."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                         timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["fixed_seconds"] >= 0


def test_traffic_json_is_written_from_an_ncu_csv(tmp_path, monkeypatch):
    """`bench.py --traffic-from-ncu-csv`: the Phase-1 attention launches are the attention launches with
    the large DRAM reads; their median bytes land in the tracked JSON, and load_traffic reads them back."""
    import bench
    head = ('"ID","Process ID","Process Name","Host Name","Kernel Name","Context","Stream","Block Size","Grid Size",'
            '"Device","CC","Section Name","Metric Name","Metric Unit","Metric Value"')
    def row(i, kernel, metric, unit, value):
        return f'"{i}","1","python","box","{kernel}","1","7","(384, 1, 1)","(148, 1, 1)","0","10.0","Command line profiler metrics","{metric}","{unit}","{value}"'
    lines = ["==PROF== Connected to process 1", head]
    launches = [("gather_prefix_kernel", 31.5e6, 0.9e6), ("attn_kernel<128, 0>", 2.26e9, 1.078e9), ("attn_kernel<128, 0>", 0.571e9, 0.063e9),
                ("lse_merge_kernel<0>", 76e6, 0.1e6), ("attn_kernel<128, 0>", 2.27e9, 1.080e9), ("attn_kernel<128, 0>", 0.571e9, 0.063e9)]
    for i, (k, rd, wr) in enumerate(launches):
        lines.append(row(i, k, "dram__bytes_read.sum", "byte", f"{int(rd):,}"))
        lines.append(row(i, k, "dram__bytes_write.sum", "Mbyte", f"{wr / 1e6:.3f}"))
    csv_path = tmp_path / "dram.csv"
    csv_path.write_text("\n".join(lines) + "\n")
    monkeypatch.setattr(bench, "TRAFFIC_JSON", str(tmp_path / "traffic.json"))
    bench.traffic_from_ncu_csv(str(csv_path), "128k")
    rec = json.load(open(tmp_path / "traffic.json"))["128k"]
    assert rec["launches"] == 2 and rec["dram_bytes_read"] == 2.265e9 and abs(rec["dram_bytes_write"] - 1.079e9) < 1e3
    assert bench.load_traffic("128k") == rec["dram_bytes_read"] + rec["dram_bytes_write"]
    assert bench.load_traffic("16k") is None
