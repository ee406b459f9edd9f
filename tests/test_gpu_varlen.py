"""GPU parity: causal attention over assembled inputs of different lengths (Algorithm 1 line 8)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_attention
from paper_2607_20457_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def assemble(w, X, pidx, plen):
    """Rows of Input_i = [prefix_i | block_i] for every block, packed back to back (Eq. 4)."""
    parts, cu = [], [0]
    for i in range(w.n_blocks):
        rows = list(pidx[: plen[i]]) + list(range(i * w.block_size, (i + 1) * w.block_size))
        parts.append(X[torch.tensor(rows)])
        cu.append(cu[-1] + len(rows))
    return torch.cat(parts).contiguous(), cu


def test_arbitrary_lengths():
    w = W.shrink(W.CONFIGS["tiny"], L=1500, block_size=1500, Hq=4, Hkv=2, d=128)
    Q, K, V = W.qkv(w, q_scale=2.0)
    cu = [0, 1, 130, 131, 515, 900, 1500]                      # 1 row, ragged tiles, odd and even tile counts
    status = binding.new_status(DEV)
    O, LSE = binding.pulsar_causal_varlen_attn(Q.to(DEV), K.to(DEV), V.to(DEV), cu, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    Oref, Lref = oracle.causal_varlen_attn(Q, K, V, cu)
    print(check_attention(O, LSE, Oref, Lref, "varlen"))


def test_assembled_pulsar_inputs_and_agreement_with_the_gathering_operator():
    # At the first layer the prefix keys are the global rows, so the block rows of the assembled
    # run must agree with pulsar_phase1_attn, which gathers the same rows.
    w = W.shrink(W.CONFIGS["tiny"], L=2048, block_size=512, chunk=16, k=4, sink=64, Hq=4, Hkv=1, d=64)
    sel = oracle.maxidf_select(W.needle_ids(w), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    pidx, plen = sel["prefix_idx"], sel["prefix_len"]
    Q, K, V = W.qkv(w)
    Qa, cu = assemble(w, Q, pidx, plen)
    Ka, _ = assemble(w, K, pidx, plen)
    Va, _ = assemble(w, V, pidx, plen)
    assert [b - a for a, b in zip(cu[:-1], cu[1:])] == [w.block_size + int(p) for p in plen]   # n_i of Eq. 14
    O, LSE = binding.pulsar_causal_varlen_attn(Qa.to(DEV), Ka.to(DEV), Va.to(DEV), cu)
    Oref, Lref = oracle.causal_varlen_attn(Qa, Ka, Va, cu)
    print(check_attention(O, LSE, Oref, Lref, "assembled"))
    O1, L1, _, _ = binding.pulsar_phase1_attn(Q.to(DEV), K.to(DEV), V.to(DEV), w.block_size,
                                              torch.from_numpy(pidx).to(DEV), torch.from_numpy(plen).to(DEV))
    torch.cuda.synchronize()
    for i in range(w.n_blocks):
        blk = slice(cu[i + 1] - w.block_size, cu[i + 1])
        own = slice(i * w.block_size, (i + 1) * w.block_size)
        assert (O[blk].float() - O1[own].float()).abs().max().item() <= 2e-2
        assert (LSE[blk] - L1[own]).abs().max().item() <= 1e-3


def test_16k_config_assembled_sampled_sequences():
    w = W.CONFIGS["16k"]
    pidx, plen = W.first_k_prefix(w)
    Q, K, V = W.qkv(w)
    Qa, cu = assemble(w, Q, pidx, plen)
    Ka, _ = assemble(w, K, pidx, plen)
    Va, _ = assemble(w, V, pidx, plen)
    O, LSE = binding.pulsar_causal_varlen_attn(Qa.to(DEV), Ka.to(DEV), Va.to(DEV), cu)
    torch.cuda.synchronize()
    # the oracle on the last (longest) sequence, sampled rows
    a, b = cu[-2], cu[-1]
    rows = np.unique(np.concatenate([np.arange(0, 8), np.arange(b - a - 8, b - a),
                                     np.random.default_rng(0).integers(0, b - a, 48)]))
    Oref, Lref = oracle.phase1_attn(Qa[a:b], Ka[a:b], Va[a:b], b - a, np.zeros(0, np.int32), np.zeros(1, np.int32),
                                    rows=rows)
    idx = torch.from_numpy(rows + a).to(DEV)
    print(check_attention(O[idx], LSE[idx], Oref, Lref, "16k assembled, last sequence"))


def test_bad_offsets_are_rejected_on_the_host():
    z = torch.zeros(64, 2, 64, dtype=torch.bfloat16, device=DEV)
    for cu in ([0, 10, 10, 64], [1, 64], [0, 32]):
        with pytest.raises(binding.PulsarError) as e:
            binding.pulsar_causal_varlen_attn(z, z, z, cu)
        assert e.value.status == 2


def test_kv_discard_keeps_each_blocks_own_rows():
    """Appendix F: after the pass over the assembled inputs only the last block_size rows of each are
    kept -- the same rows a boolean mask that is true on the last block_size positions selects --
    and the retained cache is the original K, V (every context token once)."""
    w = W.CONFIGS["tiny"]
    _, K, V = W.qkv(w)
    pidx, plen = W.first_k_prefix(w)
    rows, cu = [], [0]
    for i in range(w.n_blocks):
        rows += list(pidx[: plen[i]]) + list(range(i * w.block_size, (i + 1) * w.block_size))
        cu.append(len(rows))
    idx = torch.tensor(rows)
    Ka, Va = K[idx].contiguous().to(DEV), V[idx].contiguous().to(DEV)
    Kr, Vr = binding.pulsar_retain_block_kv(Ka, Va, cu, w.block_size)
    torch.cuda.synchronize()
    for i in range(w.n_blocks):
        is_bi = torch.zeros(cu[i + 1] - cu[i], dtype=torch.bool)
        is_bi[-w.block_size:] = True
        seg = Ka[cu[i]: cu[i + 1]].cpu()[is_bi]
        assert torch.equal(Kr[i * w.block_size: (i + 1) * w.block_size].cpu(), seg)
    assert torch.equal(Kr.cpu(), K) and torch.equal(Vr.cpu(), V)
    with pytest.raises(binding.PulsarError):
        binding.pulsar_retain_block_kv(Ka, Va, cu, w.block_size + cu[1] + 1)       # longer than the first input
