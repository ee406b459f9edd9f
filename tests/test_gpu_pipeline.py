"""The step wrappers: device-resident, host buffers in order, host buffers pipelined -- same results."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_20457_b200 import workloads as W
from paper_2607_20457_b200.pipeline import ContextEncoder

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_host_and_pipelined_steps_equal_the_device_step_and_the_oracle_selection():
    w = W.shrink(W.CONFIGS["tiny"], L=2048, block_size=512, nq=16)
    ids = W.needle_ids(w)
    Q, K, V = W.qkv(w)
    Qq = W.phase2_query(w)
    enc = ContextEncoder(w, DEV, slots=2)
    h = enc.host_buffers()
    h["ids"].copy_(torch.from_numpy(ids.view(np.int32)))
    h["Q"].copy_(Q); h["K"].copy_(K); h["V"].copy_(V); h["Qq"].copy_(Qq)
    dev_in = [h[n].to(DEV) for n in ("ids", "Q", "K", "V", "Qq")]
    ref = enc.step_device(*dev_in)
    ref = {k: ref[k].clone() for k in ("O1", "LSE1", "O2", "LSE2", "prefix_idx")}
    torch.cuda.synchronize()
    sel = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    np.testing.assert_array_equal(ref["prefix_idx"].cpu().numpy(), sel["prefix_idx"])

    h2d, d2h = enc.step_host(h)
    torch.cuda.synchronize()
    assert h2d == sum(h[n].numel() * h[n].element_size() for n in ("ids", "Q", "K", "V", "Qq"))
    for k, v in ref.items():
        assert torch.equal(h[k], v.cpu()), k

    outs = [enc.host_buffers(), enc.host_buffers()]
    for o in outs:
        for k in ref:
            o[k].zero_()
    enc.run_host_pipelined(h, outs, 5)
    torch.cuda.synchronize()
    for o in outs:
        for k, v in ref.items():
            assert torch.equal(o[k], v.cpu()), k
    assert int(enc.status.item()) == 0


@pytest.mark.parametrize("exchange", ["allgather", "fused"])
def test_bench_block_sharded_mode_runs_and_reports(exchange):
    """`bench.py --shard blocks` at one rank: same contract line, strong scaling, clean status."""
    import json, os, subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--workload", "tiny", "--shard", "blocks",
                          "--exchange", exchange, "--steps", "3", "--warmup", "3"], capture_output=True, text=True,
                         timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["scaling"] == "strong" and line["config"]["shard"] == "blocks" and line["device_status"] == 0
    assert line["value"] > 0 and line["gpu_launches"] > 0 and line["e2e"]["h2d_bytes_per_step"] > 0


def test_step_captured_as_a_cuda_graph_replays_to_the_same_results():
    w = W.CONFIGS["tiny"]
    enc = ContextEncoder(w, DEV)
    slot = enc.slots[0]
    ids = W.needle_ids(w)
    Q, K, V = W.qkv(w)
    slot["ids"].copy_(torch.from_numpy(ids.view(np.int32)))
    slot["Q"].copy_(Q); slot["K"].copy_(K); slot["V"].copy_(V); slot["Qq"].copy_(W.phase2_query(w))
    eager = {k: v.clone() for k, v in enc.step_device(slot["ids"], slot["Q"], slot["K"], slot["V"], slot["Qq"]).items()
             if k != "sel"}
    graph, res = enc.capture_step()
    for k in eager:
        res[k].zero_()
    graph.replay()
    torch.cuda.synchronize()
    for k in eager:
        assert torch.equal(res[k], eager[k]), k
    # new inputs in the same buffers, replayed: equals an eager run on them
    Q2, K2, V2 = W.qkv(w, seed=77)
    slot["Q"].copy_(Q2); slot["K"].copy_(K2); slot["V"].copy_(V2)
    graph.replay()
    torch.cuda.synchronize()
    got = {k: res[k].clone() for k in eager}
    again = enc.step_device(slot["ids"], slot["Q"], slot["K"], slot["V"], slot["Qq"])
    torch.cuda.synchronize()
    for k in eager:
        assert torch.equal(got[k], again[k]), k
    assert int(enc.status.item()) == 0
