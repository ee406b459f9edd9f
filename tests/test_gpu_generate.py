"""GPU parity: the Phase-2 generation step against the oracle (Algorithm 1 lines 11-16)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_attention
from paper_2607_20457_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_steps(w, steps, cap, q_scale=1.0, n_splits=0, shard_fill=0.0):
    _, K, V = W.qkv(w)
    Kd, Vd = K.to(DEV), V.to(DEV)
    gen = torch.Generator().manual_seed(21)
    Kgen_o = np.zeros((cap, w.Hkv, w.d), np.uint16); Vgen_o = np.zeros_like(Kgen_o)
    Kgen_d = torch.full((cap, w.Hkv, w.d), shard_fill, dtype=torch.bfloat16, device=DEV); Vgen_d = Kgen_d.clone()
    status = binding.new_status(DEV)
    gen_len = 0
    for n_new in steps:
        Qn = (torch.randn(n_new, w.Hq, w.d, generator=gen) * q_scale).to(torch.bfloat16)
        Kn = torch.randn(n_new, w.Hkv, w.d, generator=gen).to(torch.bfloat16)
        Vn = torch.randn(n_new, w.Hkv, w.d, generator=gen).to(torch.bfloat16)
        O, LSE = binding.pulsar_phase2_generate_step(Qn.to(DEV), Kn.to(DEV), Vn.to(DEV), Kd, Vd, w.n_blocks,
                                                     w.block_size, Kgen_d, Vgen_d, gen_len, n_splits=n_splits,
                                                     status=status)
        Oref, Lref = oracle.generate_step(Qn, Kn, Vn, K, V, Kgen_o, Vgen_o, gen_len)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        print(check_attention(O, LSE, Oref, Lref, f"{w.name} step n_new={n_new} gen_len={gen_len}"))
        gen_len += n_new
        # the shard on the device holds the same bits as the oracle's
        got = Kgen_d[:gen_len].cpu().view(torch.int16).numpy().view(np.uint16)
        np.testing.assert_array_equal(got, Kgen_o[:gen_len])
    return gen_len


def test_tiny_config_query_then_tokens():
    run_steps(W.CONFIGS["tiny"], [32, 1, 1, 1, 7], cap=64)


def test_shard_longer_than_one_key_tile_and_peaked_logits():
    # 150 + 140 rows: the shard spans three key tiles, the new tokens two query tiles
    w = W.shrink(W.CONFIGS["tiny"], L=2048, block_size=512, Hq=8, Hkv=2, d=128)
    run_steps(w, [150, 140, 1], cap=320, q_scale=3.0, n_splits=4)


def test_unwritten_shard_rows_may_hold_anything():
    """The rows of the generation shard past the live ones belong to nobody yet (a cache taken from
    an uninitialised allocation): filled with NaN they must not reach the result, neither while the
    shard is shorter than one key tile nor when its last tile is partial."""
    w = W.shrink(W.CONFIGS["tiny"], L=2048, block_size=512, Hq=8, Hkv=2, d=128)
    run_steps(w, [5, 1, 130, 1], cap=512, shard_fill=float("nan"))
    run_steps(W.CONFIGS["tiny"], [1, 1], cap=200, shard_fill=float("nan"))


def test_16k_config_query_of_64_then_decode():
    run_steps(W.CONFIGS["16k"], [64, 1, 1], cap=128)


def test_capacity_is_checked_on_the_host():
    w = W.CONFIGS["tiny"]
    _, K, V = W.qkv(w)
    z = lambda n, h: torch.zeros(n, h, w.d, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(binding.PulsarError) as e:
        binding.pulsar_phase2_generate_step(z(4, w.Hq), z(4, w.Hkv), z(4, w.Hkv), K.to(DEV), V.to(DEV), w.n_blocks,
                                            w.block_size, z(8, w.Hkv), z(8, w.Hkv), gen_len=6)
    assert e.value.status == 2


def test_step_captured_as_a_cuda_graph_replays_to_the_same_results():
    """One generation step (append, attention started beside it, merge started beside the attention)
    recorded as a CUDA graph: the replay equals the call-by-call step bit for bit, also after the
    inputs in the captured buffers have changed."""
    w = W.CONFIGS["tiny"]
    _, K, V = W.qkv(w)
    Kd, Vd = K.to(DEV), V.to(DEV)
    gen = torch.Generator().manual_seed(5)
    cap, gen_len, n_new = 64, 9, 1
    rnd = lambda n, h: torch.randn(n, h, w.d, generator=gen).to(torch.bfloat16).to(DEV)
    Kgen, Vgen = rnd(cap, w.Hkv), rnd(cap, w.Hkv)
    Qn, Kn, Vn = rnd(n_new, w.Hq), rnd(n_new, w.Hkv), rnd(n_new, w.Hkv)
    status = binding.new_status(DEV)
    n_splits = binding.phase2_choose_splits(n_new, w.n_blocks, w.block_size, w.Hq, w.Hkv, w.d)
    ws = binding._workspace(binding.load_library().pulsar_phase2_generate_workspace_bytes(
        n_new, w.n_blocks, w.block_size, w.Hq, w.Hkv, w.d, n_splits), DEV)
    O = torch.empty_like(Qn)

    def step():
        return binding.pulsar_phase2_generate_step(Qn, Kn, Vn, Kd, Vd, w.n_blocks, w.block_size, Kgen, Vgen, gen_len,
                                                   n_splits=n_splits, out=O, workspace=ws, status=status)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        _, LSE_g = step()
    for fresh in (False, True):
        if fresh:                                       # new token in the captured buffers
            Qn.copy_(rnd(n_new, w.Hq)); Kn.copy_(rnd(n_new, w.Hkv)); Vn.copy_(rnd(n_new, w.Hkv))
        O.zero_(); LSE_g.zero_()
        graph.replay()
        torch.cuda.synchronize()
        O_replay, LSE_replay, K_row = O.clone(), LSE_g.clone(), Kgen[gen_len].clone()
        _, LSE_e = step()
        torch.cuda.synchronize()
        assert torch.equal(O_replay, O) and torch.equal(LSE_replay, LSE_e)
        assert torch.equal(K_row, Kn[0]) and torch.equal(Kgen[gen_len], Kn[0])
        to_np = lambda t: t.cpu().view(torch.int16).numpy().view(np.uint16)
        Oref, Lref = oracle.generate_step(Qn.cpu(), Kn.cpu(), Vn.cpu(), K, V, to_np(Kgen).copy(), to_np(Vgen).copy(),
                                          gen_len)
        print(check_attention(O_replay, LSE_replay, Oref, Lref, f"graph replay fresh={fresh}"))
    assert int(status.item()) == 0
