"""GPU parity of the sharded path (block-to-host mapping, Appendix J; Phase-2 exchange, Appendix H).

One GPU: the H ranks run one after the other in this process and the all-gather is a concatenation
of their send buffers (no kernel waits on another).  The sharded result is compared with the
oracle and, row for row, with the unsharded entry points."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_attention, to_dev_ids
from paper_2607_20457_b200 import binding, cost_model as cm, workloads as W
from paper_2607_20457_b200.sharding import ShardLayout, ShardedContextEncoder

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def make_ranks(w, H, kind):
    lay = ShardLayout.make(w.n_blocks, H, w.block_size, w.chunk, w.k, w.sink, kind)
    return lay, [ShardedContextEncoder(lay, h, w.Hq, w.Hkv, w.d, w.vocab_size, DEV) for h in range(H)]


def sharded_phase1(w, H, kind, ids, Q, K, V):
    lay, ranks = make_ranks(w, H, kind)
    dev_ids = to_dev_ids(ids, DEV)
    local = []
    for h, r in enumerate(ranks):
        rows = torch.from_numpy(lay.local_token_rows(h)).to(DEV)
        local.append((Q[rows].contiguous(), K[rows].contiguous(), V[rows].contiguous(), rows))
        r.select(dev_ids)
    sends = [r.phase1_pack(l[1], l[2]).clone() for r, l in zip(ranks, local)]
    gathered = torch.stack(sends)                                  # what all_gather returns on every rank
    O = torch.empty_like(Q)
    LSE = torch.empty((w.L, w.Hq), dtype=torch.float32, device=DEV)
    for r, (q, k, v, rows) in zip(ranks, local):
        o, lse = r.phase1_finish(gathered, q, k, v)
        O[rows] = o
        LSE[rows] = lse
    torch.cuda.synchronize()
    assert all(int(r.status.item()) == 0 for r in ranks)
    return O, LSE


@pytest.mark.parametrize("kind", cm.MAPPINGS)
@pytest.mark.parametrize("H", [1, 2, 4])
def test_phase1_sharded_equals_unsharded(H, kind):
    w = W.CONFIGS["tiny"]
    ids = W.needle_ids(w)
    Q, K, V = (t.to(DEV) for t in W.qkv(w))
    O, LSE = sharded_phase1(w, H, kind, ids, Q, K, V)
    sel = binding.pulsar_maxidf_select(to_dev_ids(ids, DEV), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    O1, LSE1, _, _ = binding.pulsar_phase1_attn(Q, K, V, w.block_size, sel["prefix_idx"], sel["prefix_len"])
    torch.cuda.synchronize()
    assert torch.equal(O, O1) and torch.equal(LSE, LSE1)            # same kernel, same key order
    ref = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    O_ref, LSE_ref = oracle.phase1_attn(Q.cpu(), K.cpu(), V.cpu(), w.block_size, ref["prefix_idx"], ref["prefix_len"])
    check_attention(O, LSE, O_ref, LSE_ref, f"sharded phase 1 H={H} {kind}")


def test_phase1_sharded_16k_sampled_rows():
    w = W.CONFIGS["16k"]
    ids = W.needle_ids(w)
    Q, K, V = (t.to(DEV) for t in W.qkv(w))
    O, LSE = sharded_phase1(w, 4, "zigzag", ids, Q, K, V)
    ref = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    rows = W.sample_rows(w, per_block=6)
    O_ref, LSE_ref = oracle.phase1_attn(Q.cpu(), K.cpu(), V.cpu(), w.block_size, ref["prefix_idx"], ref["prefix_len"],
                                        rows=rows)
    r = torch.from_numpy(np.asarray(rows)).to(DEV)
    check_attention(O[r], LSE[r], O_ref, LSE_ref, "sharded phase 1, 16k")


@pytest.mark.parametrize("H,kind", [(1, "contiguous"), (2, "zigzag"), (4, "round_robin"), (4, "zigzag")])
@pytest.mark.parametrize("nq", [1, 37, 512])
def test_phase2_sharded(H, kind, nq):
    w = W.CONFIGS["tiny"]
    _, K, V = (t.to(DEV) for t in W.qkv(w))
    Qq = W.phase2_query(w)
    Qq = (Qq[:nq] if nq <= Qq.shape[0] else Qq.repeat((nq + Qq.shape[0] - 1) // Qq.shape[0], 1, 1)[:nq]).to(DEV)
    Qq = Qq.contiguous()
    lay, ranks = make_ranks(w, H, kind)
    sends = []
    for h, r in enumerate(ranks):
        rows = torch.from_numpy(lay.local_token_rows(h)).to(DEV)
        sends.append(r.phase2_local(Qq, K[rows].contiguous(), V[rows].contiguous()))
    gathered = torch.stack(sends)
    outs = [r.phase2_finish(gathered, nq) for r in ranks]
    torch.cuda.synchronize()
    assert all(int(r.status.item()) == 0 for r in ranks)
    for o, lse in outs[1:]:                                          # every rank ends with the same result
        assert torch.equal(o, outs[0][0]) and torch.equal(lse, outs[0][1])
    O_ref, LSE_ref = oracle.phase2_attn(Qq.cpu(), K.cpu(), V.cpu(), w.n_blocks, w.block_size)
    check_attention(outs[0][0], outs[0][1], O_ref, LSE_ref, f"sharded phase 2 H={H} {kind} nq={nq}")


def test_strided_merge_float32_partial_matches_oracle():
    rng = np.random.default_rng(3)
    J, rows, d, stride = 5, 77, 64, 77 * 64 + 77 + 3 + 16
    stride = (stride + 3) // 4 * 4
    buf = torch.zeros(J * stride, dtype=torch.float32)
    pO = rng.standard_normal((J, rows, d))
    pL = rng.standard_normal((J, rows)) * 4
    pL[2, :5] = -np.inf
    for j in range(J):
        buf[j * stride: j * stride + rows * d] = torch.from_numpy(pO[j].reshape(-1)).float()
        buf[j * stride + rows * d: j * stride + rows * d + rows] = torch.from_numpy(pL[j]).float()
    buf = buf.to(DEV)
    out = torch.empty((rows, d), dtype=torch.float32, device=DEV)
    lse = torch.empty(rows, dtype=torch.float32, device=DEV)
    binding.pulsar_lse_merge_strided(buf, buf[rows * d:], J, stride, stride, rows, d, out, lse)
    O_ref, L_ref = oracle.lse_merge(pO.astype(np.float32).astype(np.float64), pL.astype(np.float32).astype(np.float64))
    assert np.abs(out.cpu().numpy() - O_ref).max() < 2e-6 * max(1.0, np.abs(O_ref).max())
    assert np.abs(lse.cpu().numpy() - L_ref).max() < 1e-5
    with pytest.raises(binding.PulsarError):
        binding.pulsar_lse_merge_strided(buf, buf[rows * d:], J, rows * d - 4, stride, rows, d, out, lse)


def test_gather_rows_and_bad_index():
    K = torch.randn(300, 2, 64, device=DEV).bfloat16()
    V = torch.randn(300, 2, 64, device=DEV).bfloat16()
    idx = torch.tensor([5, 0, 299, 5, 17], dtype=torch.int32, device=DEV)
    Ko, Vo = torch.empty(5, 2, 64, device=DEV, dtype=torch.bfloat16), torch.empty(5, 2, 64, device=DEV, dtype=torch.bfloat16)
    st = binding.new_status(DEV)
    binding.pulsar_gather_kv_rows(K, V, idx, Ko, Vo, status=st)
    assert torch.equal(Ko, K[idx.long()]) and torch.equal(Vo, V[idx.long()]) and int(st.item()) == 0
    idx[2] = 300
    binding.pulsar_gather_kv_rows(K, V, idx, Ko, Vo, status=st)
    assert int(st.item()) & 0x2 and torch.equal(Ko[2], K[0])


@pytest.mark.parametrize("H,nq", [(1, 5), (2, 37), (4, 1), (4, 130)])
def test_phase2_with_the_exchange_fused_into_the_merge(H, nq):
    """Every rank merges its slice of the rows straight from all ranks' partial buffers (here all on
    one GPU, addressed through a pointer table as peer memory would be)."""
    from paper_2607_20457_b200.sharding import LocalPeers
    w = W.CONFIGS["tiny"]
    _, K, V = (t.to(DEV) for t in W.qkv(w))
    Qq = W.phase2_query(w)
    Qq = Qq.repeat((nq + Qq.shape[0] - 1) // Qq.shape[0], 1, 1)[:nq].contiguous().to(DEV)
    lay, ranks = make_ranks(w, H, "zigzag")
    peers = LocalPeers(H)
    for h, r in enumerate(ranks):
        rows = torch.from_numpy(lay.local_token_rows(h)).to(DEV)
        r.phase2_local_into(peers, Qq, K[rows].contiguous(), V[rows].contiguous())
    n_rows = nq * w.Hq
    O = torch.empty((n_rows, w.d), dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(n_rows, dtype=torch.float32, device=DEV)
    covered = 0
    for r in ranks:
        o, lse, begin = r.phase2_merge_slice(peers, nq)
        O[begin: begin + o.shape[0]] = o
        LSE[begin: begin + o.shape[0]] = lse
        covered += o.shape[0]
    torch.cuda.synchronize()
    assert covered == n_rows
    O_ref, LSE_ref = oracle.phase2_attn(Qq.cpu(), K.cpu(), V.cpu(), w.n_blocks, w.block_size)
    check_attention(O.view(nq, w.Hq, w.d), LSE.view(nq, w.Hq), O_ref, LSE_ref, f"fused exchange H={H} nq={nq}")
    # and it is the all-gather path's result exactly (same parts, same order)
    sends = torch.stack([p.clone() for p in peers.buffers])
    O2, LSE2 = ranks[0].phase2_finish(sends, nq)
    assert torch.equal(O2.view(n_rows, w.d), O) and torch.equal(LSE2.view(n_rows), LSE)


_SYMM_WORLD1 = r"""
import os, sys, torch, torch.distributed as dist
os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(29650 + os.getpid() % 200), RANK="0", WORLD_SIZE="1")
torch.cuda.set_device(0)
dist.init_process_group("nccl", device_id=torch.device("cuda", 0))
from paper_2607_20457_b200 import binding, workloads as W
from paper_2607_20457_b200.sharding import ShardLayout, ShardedContextEncoder, SymmetricMemoryPeers, TorchCollective
w = W.CONFIGS["tiny"]
_, K, V = (t.cuda() for t in W.qkv(w))
Qq = W.phase2_query(w).cuda()
lay = ShardLayout.make(w.n_blocks, 1, w.block_size, w.chunk, w.k, w.sink, "zigzag")
enc = ShardedContextEncoder(lay, 0, w.Hq, w.Hkv, w.d, w.vocab_size, "cuda:0", TorchCollective())
peers = SymmetricMemoryPeers()
O, LSE = enc.phase2_fused(peers, Qq, K, V)
O2, LSE2 = enc.phase2(Qq, K, V)                      # NCCL all-gather path at world size 1
O1, LSE1 = binding.pulsar_phase2_attn(Qq, K, V, w.n_blocks, w.block_size)
torch.cuda.synchronize()
assert torch.equal(O, O2) and torch.equal(LSE, LSE2)
assert (O.float() - O1.float()).abs().max().item() < 1e-2 and (LSE - LSE1).abs().max().item() < 1e-3
assert int(enc.status.item()) == 0
dist.destroy_process_group()
print("SYMM-OK")
"""


def test_symmetric_memory_and_nccl_plumbing_at_world_size_one():
    """The rendezvous, the device-side barrier and the NCCL all-gather as one rank (the only
    multi-process configuration a single GPU allows)."""
    import os, subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, PYTHONPATH=root + os.pathsep + os.environ.get("PYTHONPATH", ""))
    out = subprocess.run([sys.executable, "-c", _SYMM_WORLD1], capture_output=True, text=True, timeout=600, env=env,
                         cwd=root)
    assert out.returncode == 0 and "SYMM-OK" in out.stdout, (out.stdout + out.stderr)[-3000:]


def test_phase1_sharded_at_the_128k_configuration_equals_the_unsharded_call():
    """Eight ranks with two blocks each (zigzag), run in turn: bit-identical to pulsar_phase1_attn, whose
    output at this configuration is checked against the oracle in test_gpu_phase1.py."""
    w = W.CONFIGS["128k"]
    ids = W.token_ids(w)
    Q, K, V = (t.to(DEV) for t in W.qkv(w))
    O, LSE = sharded_phase1(w, 8, "zigzag", ids, Q, K, V)
    sel = binding.pulsar_maxidf_select(to_dev_ids(ids, DEV), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    O1, LSE1, _, _ = binding.pulsar_phase1_attn(Q, K, V, w.block_size, sel["prefix_idx"], sel["prefix_len"])
    torch.cuda.synchronize()
    assert torch.equal(O, O1) and torch.equal(LSE, LSE1)
