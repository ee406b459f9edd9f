"""The workspace-free selection entry point against the regular one (GPU, through the C ABI).

Some callers of the library cannot allocate device memory while they run (their memory was
handed to a pool at start-up, or they are a plug-in inside a process that owns the budget), so
`pulsar_maxidf_select_noalloc` keeps its scratch inside the library.  It must give exactly what
`pulsar_maxidf_select` gives, call after call, because the scratch is reused and never cleared.
This file is collected last so that a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest
import torch

from helpers import to_dev_ids
from paper_2607_20457_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _buffers(w):
    return (torch.full((w.n_blocks * w.k,), -7, dtype=torch.int32, device=DEV),
            torch.full((w.prefix_total,), -7, dtype=torch.int32, device=DEV),
            torch.full((w.n_blocks,), -7, dtype=torch.int32, device=DEV))


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    lib = binding.load_library()
    assert lib.pulsar_maxidf_select_noalloc_max_scratch() == 4 << 20
    # two different problems back to back: the second call sees the first call's leftovers
    cases = [(W.CONFIGS["128k"], W.needle_ids(W.CONFIGS["128k"])),
             (W.CONFIGS["tiny"], W.token_ids(W.shrink(W.CONFIGS["tiny"], zipf_s=2.0)))]
    for w, ids in cases:
        ids_d = to_dev_ids(ids, DEV)
        ref = binding.pulsar_maxidf_select(ids_d, w.vocab_size, w.block_size, w.chunk, w.k, w.sink,
                                           want_df=True, want_idf=True)
        status = binding.new_status(DEV)
        sel, pidx, plen = _buffers(w)
        df = torch.full((w.vocab_size,), -7, dtype=torch.int32, device=DEV)
        idf = torch.full((w.vocab_size,), -7.0, dtype=torch.float32, device=DEV)
        binding.pulsar_maxidf_select_noalloc(ids_d, w.vocab_size, w.block_size, w.chunk, w.k, w.sink,
                                             sel, pidx, plen, status=status, df_out=df, idf_out=idf)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(sel.view(w.n_blocks, w.k), ref["sel_chunks"])
        assert torch.equal(pidx, ref["prefix_idx"])
        assert torch.equal(plen, ref["prefix_len"])
        assert torch.equal(df, ref["df"]) and torch.equal(idf, ref["idf"])      # the optional tables too
    # and the first problem once more, after the smaller one has overwritten part of the scratch
    w, ids = cases[0]
    ids_d = to_dev_ids(ids, DEV)
    ref = binding.pulsar_maxidf_select(ids_d, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    sel, pidx, plen = _buffers(w)
    binding.pulsar_maxidf_select_noalloc(ids_d, w.vocab_size, w.block_size, w.chunk, w.k, w.sink, sel, pidx, plen)
    torch.cuda.synchronize()
    assert torch.equal(sel.view(w.n_blocks, w.k), ref["sel_chunks"]) and torch.equal(pidx, ref["prefix_idx"])


def test_problem_larger_than_the_builtin_scratch_is_rejected():
    # 64 blocks over a 1M-entry vocabulary need 8 MiB of presence bitmaps: more than the 4 MiB built in
    w = W.shrink(W.CONFIGS["tiny"], L=64 * 256, block_size=256, vocab_size=1 << 20)
    assert binding.maxidf_select_workspace_bytes(w.L, w.vocab_size, w.block_size, w.chunk, w.k, w.sink) > (4 << 20)
    ids_d = to_dev_ids(np.zeros(w.L, np.uint32), DEV)
    sel, pidx, plen = _buffers(w)
    with pytest.raises(binding.PulsarError) as e:
        binding.pulsar_maxidf_select_noalloc(ids_d, w.vocab_size, w.block_size, w.chunk, w.k, w.sink, sel, pidx, plen)
    assert e.value.status == 4                      # PULSAR_ERR_WORKSPACE, nothing was launched
    torch.cuda.synchronize()
    assert int(sel[0].item()) == -7
