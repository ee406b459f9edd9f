"""Pins for the selection oracle: brute force, closed forms, the needle property.

Every check here re-derives the expected result by a route that does not go
through the oracle's own code: membership scans, subset enumeration, or a value
the paper fixes (Section 3.1, Appendix C.1/C.5, Eq. 4, Eq. 14).
"""
import itertools
import math

import numpy as np
import pytest

import oracle
from paper_2607_20457_b200 import workloads as W


def brute_df(ids, nb, V):
    B = len(ids) // nb
    df = np.zeros(V, np.int64)
    for t in set(ids.tolist()):
        df[t] = sum(1 for b in range(B) if t in ids[b * nb:(b + 1) * nb])
    return df


def brute_scores(ids, nb, m, V):
    B = len(ids) // nb
    df = brute_df(ids, nb, V)
    sc = np.zeros((B, nb // m))
    for b in range(B):
        for c in range(nb // m):
            toks = ids[b * nb + c * m: b * nb + (c + 1) * m]
            sc[b, c] = max(math.log(B / max(df[t], 1)) for t in toks)
    return df, sc


@pytest.mark.parametrize("seed", range(6))
def test_subset_enumeration_tiny(seed):
    rng = np.random.default_rng(seed)
    B, C, m, k, V = 4, 7, 3, 3, 12
    nb = C * m
    ids = rng.integers(0, V, size=B * nb).astype(np.uint32)
    r = oracle.maxidf_select(ids, V, nb, m, k, sink=2)
    df, sc = brute_scores(ids, nb, m, V)
    np.testing.assert_array_equal(r["df"], df)
    np.testing.assert_allclose(r["score"], sc, rtol=0, atol=1e-15)
    for b in range(B):
        # the best k-subset: largest descending score tuple, then smallest index tuple
        best = max(itertools.combinations(range(C), k),
                   key=lambda S: (tuple(sorted((sc[b, c] for c in S), reverse=True)),
                                  tuple(-c for c in S)))
        assert tuple(r["sel_chunks"][b]) == tuple(sorted(best))


@pytest.mark.parametrize("name", ["tiny"])
def test_defining_property_on_config(name):
    w = W.CONFIGS[name]
    for ids in (W.token_ids(w), W.needle_ids(w)):
        r = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
        df, sc = brute_scores(ids, w.block_size, w.chunk, w.vocab_size)
        np.testing.assert_array_equal(r["df"], df)
        for b in range(w.n_blocks):
            S = r["sel_chunks"][b]
            assert len(S) == w.k and all(S[i] < S[i + 1] for i in range(w.k - 1))
            inside = set(S.tolist())
            for c in inside:
                for c2 in range(w.chunks_per_block):
                    if c2 not in inside:
                        assert sc[b, c] > sc[b, c2] or (sc[b, c] == sc[b, c2] and c < c2)


def test_idf_closed_forms():
    # token 0 in every block, token 1 in one block, token 2 nowhere, token 3 in two of four
    nb, m = 8, 2
    blocks = [[0, 1, 1, 0, 0, 0, 0, 3], [0] * 8, [0, 0, 3, 3, 0, 0, 0, 0], [0] * 8]
    ids = np.asarray(sum(blocks, []), np.uint32)
    r = oracle.maxidf_select(ids, 5, nb, m, 1, 0)
    assert r["df"].tolist() == [4, 1, 0, 2, 0]
    assert r["idf"][0] == 0.0
    assert r["idf"][1] == math.log(4.0)
    assert r["idf"][2] == math.log(4.0)          # max(df, 1) guard
    assert r["idf"][3] == math.log(2.0)
    # block 0: chunk 0 holds the unique token -> wins over chunk 3 (df 2)
    assert r["sel_chunks"][0].tolist() == [0]
    # block 2: chunk 1 holds token 3 twice; a block counts once
    assert r["sel_chunks"][2].tolist() == [1]
    # blocks of identical scores: ties go to the lowest index
    assert r["sel_chunks"][1].tolist() == [0] and r["sel_chunks"][3].tolist() == [0]


def test_needle_chunks_always_selected():
    # Appendix C.5: a chunk holding a token that occurs in one block only is selected,
    # as long as no more than k chunks of the block qualify.
    w = W.shrink(W.CONFIGS["tiny"], k=8)
    rng = np.random.default_rng(5)
    ids = (np.arange(w.L) % 50).astype(np.uint32)          # every id in every block
    planted = {}
    for b in range(w.n_blocks):
        cs = rng.choice(w.chunks_per_block, size=w.k - 1, replace=False)
        planted[b] = set(int(c) for c in cs)
        for j, c in enumerate(cs):
            ids[b * w.block_size + c * w.chunk + rng.integers(0, w.chunk)] = 10000 + b * 100 + j
    r = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    for b in range(w.n_blocks):
        assert planted[b] <= set(r["sel_chunks"][b].tolist())


def test_prefix_list_layout_and_lengths():
    w = W.CONFIGS["tiny"]
    ids = W.needle_ids(w)
    r = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    assert r["prefix_len"].tolist() == [0] + [w.sink + i * w.sigma for i in range(1, w.n_blocks)]
    exp = list(range(w.sink))
    for b in range(w.n_blocks - 1):
        for c in r["sel_chunks"][b]:
            exp += list(range(b * w.block_size + c * w.chunk, b * w.block_size + (c + 1) * w.chunk))
    assert r["prefix_idx"].tolist() == exp
    # Table 6 lengths: block + prefix for the last of four blocks, sigma 512, sink 64
    for L, n in ((16384, 5696), (32768, 9792), (65536, 17984)):
        nb = L // 4
        ids = np.zeros(L, np.uint32)
        rr = oracle.maxidf_select(ids, 8, nb, 32, 16, 64)
        assert nb + rr["prefix_len"][3] == n


def test_integer_and_float_ranking_agree():
    # ranking by score (float) must equal ranking by ascending minimum df (integer)
    w = W.shrink(W.CONFIGS["tiny"], zipf_s=2.0)
    ids = W.token_ids(w)
    r = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    df = r["df"].astype(np.int64)
    mindf = df[ids.astype(np.int64)].reshape(w.n_blocks, w.chunks_per_block, w.chunk).min(-1)
    for b in range(w.n_blocks):
        order = sorted(range(w.chunks_per_block), key=lambda c: (mindf[b, c], c))[: w.k]
        assert sorted(order) == r["sel_chunks"][b].tolist()
    assert len(np.unique(mindf)) >= 3      # the input really has several score levels


def test_rejects_shapes_outside_the_definition():
    ids = np.zeros(64, np.uint32)
    with pytest.raises(ValueError):
        oracle.maxidf_select(ids, 8, 24, 4, 1, 0)       # L not a multiple of the block
    with pytest.raises(ValueError):
        oracle.maxidf_select(ids, 8, 32, 4, 9, 0)       # k above chunks per block
