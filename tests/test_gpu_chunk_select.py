"""GPU parity: chunk selection under the TF-IDF, BM25, type-token and Max-IDF scores of Appendix C
(Eq. 6-9) against the oracle -- scores bit-identical float64, selection and prefix list exact."""
import numpy as np
import pytest
import torch

import oracle
from helpers import to_dev_ids
from paper_2607_20457_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MODES = ["max_idf", "tf_idf", "bm25", "type_token"]


def run_and_compare(ids, vocab_size, block_size, chunk, k, sink, mode):
    status = binding.new_status(DEV)
    out = binding.pulsar_chunk_select(to_dev_ids(ids, DEV), vocab_size, block_size, chunk, k, sink, mode,
                                      want_score=True, status=status)
    ref = oracle.chunk_select(ids, vocab_size, block_size, chunk, k, sink, mode)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = out["score"].cpu().numpy()
    assert got.tobytes() == ref["score"].tobytes(), np.abs(got - ref["score"]).max()   # same doubles
    np.testing.assert_array_equal(out["sel_chunks"].cpu().numpy(), ref["sel_chunks"])
    np.testing.assert_array_equal(out["prefix_idx"].cpu().numpy(), ref["prefix_idx"])
    np.testing.assert_array_equal(out["prefix_len"].cpu().numpy(), ref["prefix_len"])
    return out, ref


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("name", ["tiny", "16k", "128k"])
def test_configs_bit_exact(name, mode):
    w = W.CONFIGS[name]
    run_and_compare(W.token_ids(w), w.vocab_size, w.block_size, w.chunk, w.k, w.sink, mode)


@pytest.mark.parametrize("mode", MODES)
def test_needle_inputs(mode):
    w = W.CONFIGS["32k"]
    out, ref = run_and_compare(W.needle_ids(w), w.vocab_size, w.block_size, w.chunk, w.k, w.sink, mode)
    if mode != "type_token":
        assert not np.array_equal(ref["sel_chunks"], np.tile(np.arange(w.k), (w.n_blocks, 1)))


def test_max_idf_mode_equals_the_integer_selection():
    w = W.CONFIGS["64k"]
    ids = to_dev_ids(W.needle_ids(w), DEV)
    a = binding.pulsar_maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    b = binding.pulsar_chunk_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink, "max_idf")
    assert torch.equal(a["sel_chunks"], b["sel_chunks"]) and torch.equal(a["prefix_idx"], b["prefix_idx"])


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("shape", [
    dict(L=96, block_size=24, chunk=3, k=2, sink=5, vocab_size=40),          # ragged, many repeated tokens
    dict(L=4096, block_size=4096, chunk=32, k=8, sink=64, vocab_size=1000),  # one block: every IDF is 0
    dict(L=8192, block_size=1024, chunk=1, k=7, sink=0, vocab_size=300),     # chunk of one token, C = 1024
    dict(L=8192, block_size=512, chunk=64, k=8, sink=512, vocab_size=70000), # k = C
    dict(L=2048, block_size=256, chunk=16, k=0, sink=16, vocab_size=5000),   # nothing selected
    dict(L=1 << 15, block_size=32, chunk=8, k=3, sink=8, vocab_size=1 << 18),# 1024 blocks (the table's limit)
    dict(L=1 << 14, block_size=8192, chunk=2, k=300, sink=0, vocab_size=64), # C = 4096, long tie runs
    dict(L=4096, block_size=2048, chunk=1024, k=1, sink=0, vocab_size=30),   # longest chunk
])
def test_edge_shapes(shape, mode):
    rng = np.random.default_rng(5)
    ids = rng.integers(0, shape["vocab_size"], size=shape["L"]).astype(np.uint32)
    run_and_compare(ids, shape["vocab_size"], shape["block_size"], shape["chunk"], shape["k"], shape["sink"], mode)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("shape", [
    dict(L=1000, block_size=256, chunk=16, k=3, sink=20),      # short last block, chunks divide
    dict(L=777, block_size=200, chunk=7, k=5, sink=13),        # nothing divides: 4-token last chunks, BM25's D varies
    dict(L=530, block_size=512, chunk=32, k=4, sink=64),       # last block of 18 tokens: one chunk, fewer than k
    dict(L=300, block_size=512, chunk=24, k=3, sink=400),      # one block shorter than block and sink
    dict(L=2049, block_size=128, chunk=9, k=2, sink=5),        # 17 blocks, 2-token last chunks, 1-token last block
    dict(L=131000, block_size=8192, chunk=32, k=16, sink=64),  # the 128K shape cut short
])
def test_lengths_that_do_not_divide(shape, mode):
    rng = np.random.default_rng(shape["L"])
    ids = rng.integers(0, 9, size=shape["L"]).astype(np.uint32)          # few types: ties and repeated tokens
    ids[rng.integers(0, shape["L"], size=shape["L"] // 50)] = rng.integers(9, 4000, size=shape["L"] // 50)
    run_and_compare(ids, 4096, shape["block_size"], shape["chunk"], shape["k"], shape["sink"], mode)


def test_rejections():
    ids = to_dev_ids(np.zeros(1 << 16, np.uint32), DEV)
    with pytest.raises(binding.PulsarError):                  # 2048 blocks: beyond the per-df table
        binding.pulsar_chunk_select(ids, 100, 32, 8, 1, 0, "bm25")
    with pytest.raises(binding.PulsarError):                  # unknown score
        binding.pulsar_chunk_select(ids, 100, 2048, 16, 8, 16, 7)
