"""GPU parity on sequences whose length does not divide into blocks, and blocks that do not divide
into chunks: selection bit-exact, Phase 1 and Phase 2 within tolerance of the oracle.

The paper cuts the tokenised context into blocks of a given size (Appendix B.3) and the blocks into
chunks (Appendix C) without a word on remainders; the reading both sides take: the last block and the
last chunk of a block hold what remains, a block with fewer than k chunks contributes all of them,
prefix_len counts the tokens actually selected.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_attention, to_dev_ids
from paper_2607_20457_b200 import binding, workloads as W
from paper_2607_20457_b200.pipeline import ContextEncoder

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

RAGGED = [
    dict(L=1000, block_size=256, chunk=16, k=3, sink=20, Hq=4, Hkv=2, d=64),      # last block 232 rows, chunks divide
    dict(L=777, block_size=200, chunk=7, k=5, sink=13, Hq=2, Hkv=1, d=128),       # nothing divides; 4-token last chunk
    dict(L=530, block_size=512, chunk=32, k=4, sink=64, Hq=4, Hkv=1, d=64),       # last block of 18 rows: one chunk < k
    dict(L=300, block_size=512, chunk=24, k=3, sink=400, Hq=2, Hkv=2, d=64),      # one block shorter than block and sink
    dict(L=1153, block_size=384, chunk=10, k=6, sink=0, Hq=8, Hkv=2, d=128),      # last block = 1 row; 4-token last chunk
    dict(L=2049, block_size=128, chunk=9, k=2, sink=5, Hq=2, Hkv=1, d=64),        # 17 blocks, 2-token last chunk, 1-row block
    dict(L=4000, block_size=1024, chunk=32, k=8, sink=64, Hq=4, Hkv=1, d=128),    # last block 928 rows: 8 tiles -> 4 pairs
    dict(L=3300, block_size=1024, chunk=32, k=8, sink=64, Hq=4, Hkv=1, d=128),    # last block 228 rows: 2 tiles, one pair
]


def ragged_ids(w, seed=3):
    """Few frequent ids everywhere plus ids unique to a block planted at chunk ends, so that short
    last chunks are selected in some blocks and not in others."""
    rng = np.random.default_rng(seed)
    ids = rng.integers(0, 6, size=w.L).astype(np.uint32)
    nxt = 10
    for b in range(w.n_blocks):
        lo, hi = b * w.block_size, min((b + 1) * w.block_size, w.L)
        spots = [lo + int(x) for x in rng.integers(0, hi - lo, size=2)]
        if b % 2 == 0:
            spots.append(hi - 1)                           # the last token: inside the last (maybe short) chunk
        for p in spots:
            ids[p] = nxt
            nxt += 1
    assert nxt <= w.vocab_size
    return ids


def select_both(w, ids):
    status = binding.new_status(DEV)
    out = binding.pulsar_maxidf_select(to_dev_ids(ids, DEV), w.vocab_size, w.block_size, w.chunk, w.k, w.sink,
                                       want_df=True, status=status)
    ref = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    np.testing.assert_array_equal(out["sel_chunks"].cpu().numpy(), ref["sel_chunks"])
    np.testing.assert_array_equal(out["prefix_idx"].cpu().numpy(), ref["prefix_idx"])
    np.testing.assert_array_equal(out["prefix_len"].cpu().numpy(), ref["prefix_len"])
    np.testing.assert_array_equal(out["df"].cpu().numpy().view(np.uint32), ref["df"])
    return out, ref


@pytest.mark.parametrize("shape", RAGGED)
def test_selection_phase1_phase2(shape):
    w = W.shrink(W.CONFIGS["tiny"], vocab_size=4096, nq=9, **shape)
    ids = ragged_ids(w)
    out, ref = select_both(w, ids)
    for other in (W.zipf_ids(w.L, w.vocab_size, 1.3, 5), np.zeros(w.L, np.uint32)):
        select_both(w, other)                              # spread-out scores; all chunks tie

    Q, K, V = W.qkv(w, q_scale=2.0)
    status = binding.new_status(DEV)
    Kd, Vd = K.to(DEV), V.to(DEV)
    # the workspace arrives full of NaN patterns: prefix entries that no block uses (a short chunk was
    # selected, so the list is shorter than its buffer) must not reach the result through 0 * NaN
    ws = torch.full((binding.phase1_workspace_bytes(w.L, w.Hq, w.Hkv, w.d, w.block_size, out["prefix_idx"].numel()),),
                    0xFF, dtype=torch.uint8, device=DEV)
    O, LSE, Kr, Vr = binding.pulsar_phase1_attn(Q.to(DEV), Kd, Vd, w.block_size, out["prefix_idx"], out["prefix_len"],
                                                status=status, retain_copy=True, workspace=ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(Kr, Kd) and torch.equal(Vr, Vd) and Kr.shape[0] == w.L
    Oref, Lref = oracle.phase1_attn(Q, K, V, w.block_size, ref["prefix_idx"], ref["prefix_len"])
    print(check_attention(O, LSE, Oref, Lref, f"phase 1 {shape}"))

    # Phase 2 over the retained rows: one run of L rows (the parts are the library's, not the blocks')
    Qq = W.phase2_query(w, q_scale=2.0)
    for J in (0, 2):
        O2, L2 = binding.pulsar_phase2_attn(Qq.to(DEV), Kr, Vr, 1, w.L, n_splits=J, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        O2ref, L2ref = oracle.phase2_attn(Qq, K, V, 1, w.L)
        print(check_attention(O2, L2, O2ref, L2ref, f"phase 2 J={J} {shape}"))


def test_short_chunk_selected_shortens_the_prefix_on_the_gpu_too():
    w = W.shrink(W.CONFIGS["tiny"], L=30, block_size=10, chunk=4, k=2, sink=1, vocab_size=8)
    ids = np.zeros(30, np.uint32)
    ids[9] = 7
    out, _ = select_both(w, ids)
    assert out["prefix_len"].cpu().tolist() == [0, 7, 15]
    assert out["prefix_idx"].cpu().tolist()[-2:] == [-1, -1]


def test_131000_tokens_sampled_rows():
    """A sequence of 131,000 tokens in blocks of 8192 (the last block holds 8120 rows: a short last
    row tile, no second tile in its last pair) with the 128K configuration's other parameters."""
    w = W.shrink(W.CONFIGS["128k"], L=131000, nq=64)
    assert w.n_blocks == 16 and w.L - 15 * w.block_size == 8120
    ids = W.needle_ids(W.shrink(w, L=131072))[: w.L]
    out, ref = select_both(w, ids)
    Q, K, V = W.qkv(w)
    status = binding.new_status(DEV)
    Kd, Vd = K.to(DEV), V.to(DEV)
    O, LSE, _, _ = binding.pulsar_phase1_attn(Q.to(DEV), Kd, Vd, w.block_size, out["prefix_idx"], out["prefix_len"],
                                              status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rows = np.unique(np.concatenate([W.sample_rows(w, per_block=10), np.arange(w.L - 130, w.L)]))
    Oref, Lref = oracle.phase1_attn(Q, K, V, w.block_size, ref["prefix_idx"], ref["prefix_len"], rows=rows)
    idx = torch.from_numpy(rows).to(DEV)
    print(check_attention(O[idx], LSE[idx], Oref, Lref, "131000 phase 1"))
    Qq = W.phase2_query(w)
    O2, L2 = binding.pulsar_phase2_attn(Qq.to(DEV), Kd, Vd, 1, w.L, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    pick = [0, 1, 31, 32, 63]
    O2ref, L2ref = oracle.phase2_attn(Qq[pick].contiguous(), K, V, 1, w.L)
    print(check_attention(O2[pick], L2[pick], O2ref, L2ref, "131000 phase 2"))


def test_whole_step_through_the_encoder():
    w = W.shrink(W.CONFIGS["tiny"], L=3000, block_size=1024, chunk=24, k=5, sink=64, nq=16, vocab_size=4096)
    ids = ragged_ids(w)
    Q, K, V = W.qkv(w)
    Qq = W.phase2_query(w)
    enc = ContextEncoder(w, DEV)
    res = enc.step_device(to_dev_ids(ids, DEV), Q.to(DEV), K.to(DEV), V.to(DEV), Qq.to(DEV))
    torch.cuda.synchronize()
    assert int(enc.status.item()) == 0
    ref = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    np.testing.assert_array_equal(res["prefix_idx"].cpu().numpy(), ref["prefix_idx"])
    Oref, Lref = oracle.phase1_attn(Q, K, V, w.block_size, ref["prefix_idx"], ref["prefix_len"])
    check_attention(res["O1"], res["LSE1"], Oref, Lref, "encoder phase 1")
    O2ref, L2ref = oracle.phase2_attn(Qq, K, V, 1, w.L)
    check_attention(res["O2"], res["LSE2"], O2ref, L2ref, "encoder phase 2")
