"""GPU parity: Max-IDF selection against the oracle, bit-exact (Section 3.1, Eq. 2-4)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import to_dev_ids
from paper_2607_20457_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_and_compare(ids, w, want_tables=True):
    status = binding.new_status(DEV)
    out = binding.pulsar_maxidf_select(to_dev_ids(ids, DEV), w.vocab_size, w.block_size, w.chunk, w.k, w.sink,
                                       want_df=want_tables, want_idf=want_tables, status=status)
    ref = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    np.testing.assert_array_equal(out["sel_chunks"].cpu().numpy(), ref["sel_chunks"])
    np.testing.assert_array_equal(out["prefix_idx"].cpu().numpy(), ref["prefix_idx"])
    np.testing.assert_array_equal(out["prefix_len"].cpu().numpy(), ref["prefix_len"])
    if want_tables:
        np.testing.assert_array_equal(out["df"].cpu().numpy().view(np.uint32), ref["df"])
        np.testing.assert_allclose(out["idf"].cpu().numpy(), ref["idf"], rtol=0, atol=1e-6)
    return out, ref


@pytest.mark.parametrize("name", W.CONFIG_ORDER)
def test_configs_bit_exact(name):
    w = W.CONFIGS[name]
    run_and_compare(W.token_ids(w), w)


@pytest.mark.parametrize("name", ["tiny", "32k", "128k"])
def test_needle_inputs_exercise_topk(name):
    w = W.CONFIGS[name]
    ids = W.needle_ids(w)
    out, ref = run_and_compare(ids, w)
    first_k = np.tile(np.arange(w.k), (w.n_blocks, 1))
    assert not np.array_equal(ref["sel_chunks"], first_k)          # the input really selects


@pytest.mark.parametrize("s", [1.5, 2.0])
def test_steeper_zipf_spreads_score_levels(s):
    w = W.shrink(W.CONFIGS["128k"], zipf_s=s)
    out, ref = run_and_compare(W.token_ids(w), w)
    assert len(np.unique(ref["score"])) >= 8


@pytest.mark.parametrize("shape", [
    dict(L=96, block_size=24, chunk=3, k=2, sink=5, vocab_size=40),       # ragged everything
    dict(L=4096, block_size=4096, chunk=32, k=8, sink=64, vocab_size=1000),   # one block
    dict(L=8192, block_size=1024, chunk=1, k=7, sink=0, vocab_size=300),      # chunk of one token, C=1024
    dict(L=8192, block_size=512, chunk=64, k=8, sink=512, vocab_size=70000),  # k = C, sink = block
    dict(L=2048, block_size=256, chunk=16, k=0, sink=16, vocab_size=5000),    # nothing selected
    dict(L=1 << 16, block_size=64, chunk=8, k=3, sink=8, vocab_size=1 << 20), # 1024 blocks, large vocabulary
])
def test_edge_shapes(shape):
    w = W.shrink(W.CONFIGS["tiny"], **shape)
    rng = np.random.default_rng(shape["L"])
    ids = rng.integers(0, min(w.vocab_size, 4 * w.block_size), size=w.L).astype(np.uint32)
    run_and_compare(ids, w)
    run_and_compare(W.zipf_ids(w.L, w.vocab_size, 1.3, 5), w, want_tables=False)


def test_token_outside_vocabulary_is_reported_not_fatal():
    w = W.CONFIGS["tiny"]
    ids = W.token_ids(w).copy()
    ids[100] = w.vocab_size + 5
    status = binding.new_status(DEV)
    binding.pulsar_maxidf_select(to_dev_ids(ids, DEV), w.vocab_size, w.block_size, w.chunk, w.k, w.sink,
                                 status=status)
    torch.cuda.synchronize()
    assert int(status.item()) & binding.DEV_BAD_TOKEN


def test_two_runs_are_identical():
    w = W.CONFIGS["128k"]
    ids = to_dev_ids(W.needle_ids(w), DEV)
    a = binding.pulsar_maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    b = binding.pulsar_maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    for key in ("sel_chunks", "prefix_idx", "prefix_len"):
        assert torch.equal(a[key], b[key])


def test_many_blocks():
    """50,000 blocks of one 2-token chunk each: the level histogram of the top-k kernel (one counter per
    possible df value) nearly fills shared memory; beyond that the call is rejected on the host."""
    w = W.shrink(W.CONFIGS["tiny"], L=100000, block_size=2, chunk=2, k=1, sink=1, vocab_size=97)
    rng = np.random.default_rng(1)
    run_and_compare(rng.integers(0, 97, size=w.L).astype(np.uint32), w, want_tables=True)
    ids = to_dev_ids(np.zeros(65533, np.uint32), DEV)
    with pytest.raises(binding.PulsarError) as e:            # 65,533 blocks: within the 16-bit levels, beyond shared memory
        binding.pulsar_maxidf_select(ids, 97, 1, 1, 1, 0)
    assert e.value.status == 2
