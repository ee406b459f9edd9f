"""GPU parity: Phase-1 prefix-block attention against the float64 oracle (Eq. 1 over Eq. 4)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_attention
from paper_2607_20457_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_phase1(w, Q, K, V, pidx, plen, rows=None, scale=0.0, what=""):
    status = binding.new_status(DEV)
    pidx_d = torch.from_numpy(np.ascontiguousarray(pidx, dtype=np.int32)).to(DEV)
    plen_d = torch.from_numpy(np.ascontiguousarray(plen, dtype=np.int32)).to(DEV)
    O, LSE, _, _ = binding.pulsar_phase1_attn(Q.to(DEV), K.to(DEV), V.to(DEV), w.block_size, pidx_d, plen_d,
                                              softmax_scale=scale, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, f"device status {int(status.item())}"
    Oref, Lref = oracle.phase1_attn(Q, K, V, w.block_size, pidx, plen, scale=scale, rows=rows)
    if rows is not None:
        idx = torch.from_numpy(np.asarray(rows)).to(DEV)
        O, LSE = O[idx], LSE[idx]
    return check_attention(O, LSE, Oref, Lref, what)


def test_tiny_config_full_output():
    w = W.CONFIGS["tiny"]
    ids = W.token_ids(w)
    sel = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    Q, K, V = W.qkv(w)
    print(run_phase1(w, Q, K, V, sel["prefix_idx"], sel["prefix_len"], what="tiny"))


def test_tiny_config_peaked_logits_and_needle_prefix():
    w = W.CONFIGS["tiny"]
    sel = oracle.maxidf_select(W.needle_ids(w), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    Q, K, V = W.qkv(w, q_scale=4.0)
    print(run_phase1(w, Q, K, V, sel["prefix_idx"], sel["prefix_len"], what="tiny peaked"))


@pytest.mark.parametrize("shape", [
    dict(L=512, block_size=128, chunk=8, k=2, sink=8, Hq=2, Hkv=1, d=64),          # one tile per block
    dict(L=768, block_size=192, chunk=16, k=3, sink=40, Hq=4, Hkv=2, d=128),       # ragged block, ragged prefix
    dict(L=600, block_size=200, chunk=8, k=5, sink=3, Hq=2, Hkv=2, d=128),         # nothing divides 128
    dict(L=1280, block_size=640, chunk=32, k=20, sink=64, Hq=8, Hkv=2, d=64),      # prefix longer than a tile
    dict(L=384, block_size=384, chunk=32, k=2, sink=64, Hq=2, Hkv=1, d=128),       # one block: plain causal
    dict(L=100, block_size=50, chunk=5, k=1, sink=0, Hq=1, Hkv=1, d=64),           # smaller than a tile, no sink
])
def test_small_shapes_full_output(shape):
    w = W.shrink(W.CONFIGS["tiny"], vocab_size=4096, nq=4, **shape)
    sel = oracle.maxidf_select(W.needle_ids(w), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    Q, K, V = W.qkv(w, q_scale=2.0)
    print(run_phase1(w, Q, K, V, sel["prefix_idx"], sel["prefix_len"], what=str(shape)))


def test_empty_prefix_and_custom_scale():
    w = W.shrink(W.CONFIGS["tiny"], L=1024, block_size=256)
    Q, K, V = W.qkv(w)
    print(run_phase1(w, Q, K, V, np.zeros(0, np.int32), np.zeros(w.n_blocks, np.int32), scale=0.3,
                     what="no prefix"))


def test_star_anchor_prefix():
    w = W.shrink(W.CONFIGS["tiny"], L=2048, block_size=512)
    Q, K, V = W.qkv(w)
    pidx, plen = W.star_anchor_prefix(w)
    print(run_phase1(w, Q, K, V, pidx, plen, what="star anchor"))


def test_poisoned_invisible_rows_do_not_leak():
    # rows a block must not see get huge finite values and amplified keys
    w = W.shrink(W.CONFIGS["tiny"], L=2048, block_size=512, chunk=16, k=4, sink=64)
    sel = oracle.maxidf_select(W.needle_ids(w), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    pidx, plen = sel["prefix_idx"], sel["prefix_len"]
    Q, K, V = W.qkv(w)
    blk = 2
    rows = np.arange(blk * w.block_size, blk * w.block_size + 200)
    visible = set(pidx[: plen[blk]].tolist()) | set(rows.tolist())
    K2, V2 = K.clone(), V.clone()
    hidden = torch.tensor([j for j in range(w.L) if j not in visible])
    V2[hidden] = 3.0e4
    K2[hidden] = K2[hidden] * 8
    print(run_phase1(w, Q, K2, V2, pidx, plen, rows=rows, what="poison"))


@pytest.mark.parametrize("name", ["16k", "32k", "64k", "128k"])
def test_full_size_configs_on_sampled_rows(name):
    """Each configuration with the prefix its own token ids select (the 32K ids carry injected rare
    tokens; at 128K the selection leaves "the first k chunks" in some blocks)."""
    w = W.CONFIGS[name]
    sel = oracle.maxidf_select(W.token_ids(w), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    pidx, plen = sel["prefix_idx"], sel["prefix_len"]
    Q, K, V = W.qkv(w)
    rows = W.sample_rows(w, per_block=16 if w.L > 40000 else 32)
    print(run_phase1(w, Q, K, V, pidx, plen, rows=rows, what=name))


def test_twice_the_largest_configuration_on_sampled_rows():
    """262,144 tokens in 32 blocks of 8192: prefixes up to 15,936 rows (125 key tiles before the block's
    own 64), 65,536 work items; the prefix is the one the sequence's own token ids select."""
    w = W.shrink(W.CONFIGS["128k"], L=262144)
    sel = oracle.maxidf_select(W.token_ids(w), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    Q, K, V = W.qkv(w)
    rows = W.sample_rows(w, per_block=10)
    print(run_phase1(w, Q, K, V, sel["prefix_idx"], sel["prefix_len"], rows=rows, what="256k"))


def test_64k_star_anchor_sampled_rows():
    w = W.CONFIGS["64k"]
    pidx, plen = W.star_anchor_prefix(w)
    Q, K, V = W.qkv(w)
    rows = W.sample_rows(w, per_block=12)
    print(run_phase1(w, Q, K, V, pidx, plen, rows=rows, what="64k star"))


def test_bad_prefix_index_is_reported():
    w = W.shrink(W.CONFIGS["tiny"], L=1024, block_size=256)
    Q, K, V = W.qkv(w)
    pidx, plen = W.first_k_prefix(w)
    pidx = pidx.copy()
    pidx[w.sink + 3] = 900                      # a row of block 3 in block 1's prefix
    status = binding.new_status(DEV)
    binding.pulsar_phase1_attn(Q.to(DEV), K.to(DEV), V.to(DEV), w.block_size, torch.from_numpy(pidx).to(DEV),
                               torch.from_numpy(plen).to(DEV), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) & binding.DEV_BAD_PREFIX


def test_retained_kv_is_the_blocks_own_rows_and_runs_repeat_exactly():
    w = W.shrink(W.CONFIGS["tiny"], L=2048, block_size=512)
    Q, K, V = (t.to(DEV) for t in W.qkv(w))
    pidx, plen = (torch.from_numpy(x).to(DEV) for x in W.first_k_prefix(w))
    O1, L1, Kr, Vr = binding.pulsar_phase1_attn(Q, K, V, w.block_size, pidx, plen, retain_copy=True)
    O2, L2, Kv, Vv = binding.pulsar_phase1_attn(Q, K, V, w.block_size, pidx, plen)
    torch.cuda.synchronize()
    assert torch.equal(Kr, K) and torch.equal(Vr, V) and Kr.data_ptr() != K.data_ptr()
    assert Kv.data_ptr() == K.data_ptr() and Kr.shape[0] == w.L        # exactly block_size rows per block, L in total
    assert torch.equal(O1, O2) and torch.equal(L1, L2)


def test_many_small_blocks_long_nested_prefix():
    # 32 blocks of one tile each: the prefix grows to 31 summaries, every item is a single tile pair
    w = W.shrink(W.CONFIGS["tiny"], L=4096, block_size=128, chunk=8, k=3, sink=16, Hq=4, Hkv=2, d=64, vocab_size=4096)
    sel = oracle.maxidf_select(W.needle_ids(w), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    Q, K, V = W.qkv(w, q_scale=2.0)
    print(run_phase1(w, Q, K, V, sel["prefix_idx"], sel["prefix_len"], what="32 blocks"))


def test_prefix_list_present_but_unused():
    # a prefix list exists, yet every block is told to use none of it
    w = W.shrink(W.CONFIGS["tiny"], L=1024, block_size=256)
    Q, K, V = W.qkv(w)
    pidx, _ = W.first_k_prefix(w)
    print(run_phase1(w, Q, K, V, pidx, np.zeros(w.n_blocks, np.int32), what="unused prefix"))


def test_non_monotone_prefix_lengths():
    # the scheduler assumes later blocks are costlier; results must not depend on that
    w = W.shrink(W.CONFIGS["tiny"], L=2048, block_size=512)
    Q, K, V = W.qkv(w)
    pidx, plen = W.first_k_prefix(w)
    plen = np.asarray([0, plen[3], 0, plen[1]], np.int32)      # only indices below 512 are used by block 1
    pidx = pidx.copy()
    pidx[:] = np.arange(len(pidx)) % 512                       # all entries lie in block 0
    print(run_phase1(w, Q, K, V, pidx, plen, what="non-monotone"))


@pytest.mark.parametrize("d", [64, 128])
def test_logits_that_jump_far_above_the_running_maximum(d):
    """Key magnitudes grow along the sequence in steps, some in the first and some in the second
    half of a 128-key tile, so that later tiles hold logits tens of nats above everything seen
    before: the kernel has to move its running maximum in the middle of a row, also after the first
    half of a tile has already gone to the tensor cores."""
    w = W.shrink(W.CONFIGS["tiny"], L=2048, block_size=1024, chunk=16, k=4, sink=64, Hq=4, Hkv=2, d=d)
    Q, K, V = W.qkv(w, seed=31)
    Kf = K.float()
    for start, factor in ((200, 6.0), (330, 14.0), (520, 30.0), (1024 + 150, 8.0), (1024 + 600, 40.0), (1024 + 840, 90.0)):
        Kf[start: start + 40] *= factor
    K = Kf.bfloat16()
    pidx, plen = W.first_k_prefix(w)
    print(run_phase1(w, Q, K, V, pidx, plen, what=f"jumping logits d={d}"))
