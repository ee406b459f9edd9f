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
        oracle.maxidf_select(ids, 8, 32, 4, 9, 0)       # k above chunks per block
    with pytest.raises(ValueError):
        oracle.maxidf_select(ids, 8, 32, 4, 2, 33)      # sink longer than a block
    with pytest.raises(ValueError):
        oracle.chunk_select(ids, 8, 32, 4, 9, 0, "bm25")   # k above chunks per block, any score


# ---- lengths that do not divide ---------------------------------------------------------------
def ragged_reference(ids, nb, m, k, sink, V):
    """The selection on a sequence whose length need not divide, by a route of its own: Python
    slices cut the blocks and chunks (a slice simply ends where the data ends), df by set
    membership, the k best chunks by sorting on (-score, index)."""
    L = len(ids)
    blocks = [ids[s: s + nb].tolist() for s in range(0, L, nb)]
    B = len(blocks)
    df = {t: sum(1 for blk in blocks if t in blk) for t in set(ids.tolist())}
    sel, prefix, plen = [], list(range(min(sink, len(blocks[0])))), []
    for b, blk in enumerate(blocks):
        plen.append(0 if b == 0 else len(prefix))
        chunks = [blk[s: s + m] for s in range(0, len(blk), m)]
        score = [max(math.log(B / max(df[t], 1)) for t in ch) for ch in chunks]
        best = sorted(sorted(range(len(chunks)), key=lambda c: (-score[c], c))[:k])
        sel.append(best + [-1] * (k - len(best)))
        if b < B - 1:
            for c in best:
                prefix += list(range(b * nb + c * m, b * nb + c * m + len(chunks[c])))
    cap = sink + (B - 1) * k * m
    return np.asarray(sel), np.asarray(prefix + [-1] * (cap - len(prefix))), np.asarray(plen)


@pytest.mark.parametrize("L,nb,m,k,sink", [
    (50, 16, 5, 2, 3),      # short last block (2 tokens) and a one-token last chunk in every block
    (61, 20, 4, 3, 6),      # chunks divide the block, the last block holds 1 token: fewer chunks than k
    (64, 16, 4, 2, 4),      # everything divides: the reading changes nothing
    (47, 12, 5, 3, 12),     # sink = the whole first block; last block 11 tokens
    (9, 16, 4, 2, 12),      # one block shorter than the block size and than the sink
    (100, 33, 7, 5, 0),     # five chunks per block, all taken; no sink
])
@pytest.mark.parametrize("seed", range(3))
def test_lengths_that_do_not_divide(L, nb, m, k, sink, seed):
    V = 14
    ids = np.random.default_rng(100 + seed).integers(0, V, size=L).astype(np.uint32)
    r = oracle.maxidf_select(ids, V, nb, m, k, sink)
    sel, prefix, plen = ragged_reference(ids, nb, m, k, sink, V)
    np.testing.assert_array_equal(r["sel_chunks"], sel)
    np.testing.assert_array_equal(r["prefix_idx"], prefix)
    np.testing.assert_array_equal(r["prefix_len"], plen)


def test_a_short_last_chunk_can_win_and_shortens_the_prefix():
    # blocks of 10 tokens in chunks of 4: the third chunk of a block has 2 tokens.  Block 0's short
    # chunk holds the only token that is unique to the block, so it is selected (Appendix C.5) and
    # contributes its 2 tokens: block 1's prefix is sink + 4 + 2, not sink + 2*4 (Eq. 14 with whole chunks).
    ids = np.zeros(30, np.uint32)
    ids[9] = 7
    r = oracle.maxidf_select(ids, 8, 10, 4, 2, 1)
    assert r["sel_chunks"].tolist() == [[0, 2], [0, 1], [0, 1]]
    assert r["prefix_len"].tolist() == [0, 1 + 4 + 2, 1 + 6 + 8]
    assert r["prefix_idx"].tolist() == [0, 0, 1, 2, 3, 8, 9, 10, 11, 12, 13, 14, 15, 16, 17, -1, -1]
    assert r["df"][7] == 1 and r["df"][0] == 3
    assert r["score"][0, 2] == math.log(3.0) and r["score"][0, 0] == 0.0


def test_short_last_block_counts_as_a_block():
    # N is the number of blocks, the short one included: 3 blocks of 8, 8 and 2 tokens
    ids = np.asarray([1] * 8 + [1] * 8 + [1, 2], np.uint32)
    r = oracle.maxidf_select(ids, 4, 8, 4, 1, 0)
    assert r["df"].tolist() == [0, 3, 1, 0]
    assert r["idf"][2] == math.log(3.0) and r["idf"][1] == 0.0
    assert r["sel_chunks"].tolist() == [[0], [0], [0]]
    assert r["score"][2].tolist() == [math.log(3.0), -math.inf]


# ---- the other scoring heuristics of Appendix C -------------------------------------------------
def python_scores(ids, nb, m, V, mode):
    """Eq. 6-9 re-derived with Python floats, collections and math.log."""
    from collections import Counter
    B = len(ids) // nb
    df = brute_df(ids, nb, V)
    out = np.zeros((B, nb // m))
    for b in range(B):
        for c in range(nb // m):
            toks = [int(t) for t in ids[b * nb + c * m: b * nb + (c + 1) * m]]
            if mode == "max_idf":
                out[b, c] = max(math.log(B / max(df[t], 1)) for t in toks)
            elif mode == "tf_idf":
                out[b, c] = sum(math.log(B / max(df[t], 1)) for t in toks) / m
            elif mode == "type_token":
                out[b, c] = len(set(toks)) / m
            else:
                cnt = Counter(toks)
                D = 1 - 0.75 + 0.75 * (m / m)                  # every chunk has the mean length
                out[b, c] = sum(math.log((B - df[t] + 0.5) / (df[t] + 0.5) + 1) * tf * 2.2 / (tf + 1.2 * D)
                                for t, tf in cnt.items())
    return out


@pytest.mark.parametrize("mode", ["max_idf", "tf_idf", "bm25", "type_token"])
def test_heuristic_scores_and_selection(mode):
    rng = np.random.default_rng(11)
    B, C, m, k, V = 5, 9, 6, 3, 40
    nb = C * m
    ids = rng.integers(0, V, size=B * nb).astype(np.uint32)
    ids[: nb] = np.arange(nb) % 7                              # a block of few, much repeated types
    r = oracle.chunk_select(ids, V, nb, m, k, 4, mode)
    sc = python_scores(ids, nb, m, V, mode)
    np.testing.assert_allclose(r["score"], sc, rtol=0, atol=1e-12)
    for b in range(B):
        S = r["sel_chunks"][b].tolist()
        assert S == sorted(S) and len(set(S)) == k
        for c in S:
            for c2 in set(range(C)) - set(S):
                a, bb = r["score"][b, c], r["score"][b, c2]
                assert a > bb or (a == bb and c < c2)
    assert r["prefix_len"].tolist() == [0] + [4 + i * k * m for i in range(1, B)]


def test_mode_zero_is_the_max_idf_selection():
    w = W.CONFIGS["tiny"]
    ids = W.needle_ids(w)
    a = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    b = oracle.chunk_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink, "max_idf")
    np.testing.assert_array_equal(a["sel_chunks"], b["sel_chunks"])
    np.testing.assert_array_equal(a["prefix_idx"], b["prefix_idx"])
    np.testing.assert_array_equal(a["score"], b["score"])


def test_heuristic_closed_forms():
    nb, m, B = 16, 4, 4
    ids = np.zeros(B * nb, np.uint32)                         # token 0 everywhere ...
    ids[0:4] = [1, 2, 3, 4]                                   # ... one chunk of four distinct tokens unique to block 0
    ids[4:8] = [5, 5, 5, 5]                                   # ... one chunk of a repeated token unique to block 0
    tt = oracle.chunk_select(ids, 8, nb, m, 1, 0, "type_token")["score"]
    assert tt[0, 0] == 1.0 and tt[0, 1] == 0.25 and tt[1, 0] == 0.25
    tf = oracle.chunk_select(ids, 8, nb, m, 1, 0, "tf_idf")["score"]
    assert tf[1, 0] == 0.0                                    # tokens present in every block carry no IDF
    assert abs(tf[0, 0] - math.log(4.0)) < 1e-15              # four tokens, each in one block of four
    bm = oracle.chunk_select(ids, 8, nb, m, 1, 0, "bm25")["score"]
    idf1 = math.log((4 - 1 + 0.5) / (1 + 0.5) + 1)
    assert abs(bm[0, 1] - idf1 * 4 * 2.2 / (4 + 1.2)) < 1e-15  # one type with tf = 4
    assert abs(bm[0, 0] - 4 * idf1 * 2.2 / (1 + 1.2)) < 1e-14  # four types with tf = 1


def ragged_scores(ids, nb, m, mode):
    """Eq. 6-9 on a sequence cut by Python slices: |C| is whatever the slice holds, the mean chunk
    length is taken over all chunks of the sequence."""
    from collections import Counter
    blocks = [ids[s: s + nb].tolist() for s in range(0, len(ids), nb)]
    B = len(blocks)
    df = Counter(t for blk in blocks for t in set(blk))
    chunks = [[blk[s: s + m] for s in range(0, len(blk), m)] for blk in blocks]
    lbar = len(ids) / sum(len(cs) for cs in chunks)
    out = []
    for cs in chunks:
        row = []
        for ch in cs:
            if mode == "max_idf":
                row.append(max(math.log(B / df[t]) for t in ch))
            elif mode == "tf_idf":
                acc = 0.0
                for t in ch:
                    acc = acc + math.log(B / df[t])
                row.append(acc / len(ch))
            elif mode == "type_token":
                row.append(len(set(ch)) / len(ch))
            else:
                D = (1 - 0.75) + 0.75 * (len(ch) / lbar)
                acc = 0.0
                for t in dict.fromkeys(ch):                    # types in order of first occurrence
                    tf = ch.count(t)
                    acc = acc + (math.log((B - df[t] + 0.5) / (df[t] + 0.5) + 1) * (tf * 2.2)) / (tf + 1.2 * D)
                row.append(acc)
        out.append(row)
    return out


@pytest.mark.parametrize("mode", ["max_idf", "tf_idf", "bm25", "type_token"])
@pytest.mark.parametrize("L,nb,m,k,sink", [(50, 16, 5, 2, 3), (61, 20, 4, 3, 6), (100, 33, 7, 5, 0), (9, 16, 4, 2, 12)])
def test_heuristics_on_lengths_that_do_not_divide(mode, L, nb, m, k, sink):
    ids = np.random.default_rng(L).integers(0, 11, size=L).astype(np.uint32)
    r = oracle.chunk_select(ids, 11, nb, m, k, sink, mode)
    sc = ragged_scores(ids, nb, m, mode)
    B = len(sc)
    prefix, plen, sel = list(range(min(sink, min(nb, L)))), [], []
    for b, row in enumerate(sc):
        for c, v in enumerate(row):
            assert r["score"][b, c] == v or abs(r["score"][b, c] - v) <= 1e-15 * abs(v)
        assert np.isneginf(r["score"][b, len(row):]).all()
        plen.append(0 if b == 0 else len(prefix))
        best = sorted(sorted(range(len(row)), key=lambda c: (-r["score"][b, c], c))[:k])
        sel.append(best + [-1] * (k - len(best)))
        if b < B - 1:
            for c in best:
                prefix += list(range(b * nb + c * m, min(b * nb + (c + 1) * m, (b + 1) * nb)))
    np.testing.assert_array_equal(r["sel_chunks"], np.asarray(sel))
    np.testing.assert_array_equal(r["prefix_len"], np.asarray(plen))
    cap = sink + (B - 1) * k * m
    np.testing.assert_array_equal(r["prefix_idx"], np.asarray(prefix + [-1] * (cap - len(prefix))))


def test_bm25_length_normaliser_by_hand():
    # 10 tokens in chunks of 4: chunks of 4, 4 and 2 tokens, mean length 10/3.  One block, so N = 1 and
    # every token has df = 1: IDF_BM25 = ln((1 - 1 + 0.5)/(1 + 0.5) + 1) = ln(4/3).
    ids = np.asarray([1, 1, 1, 1, 2, 3, 4, 5, 6, 6], np.uint32)
    r = oracle.chunk_select(ids, 8, 10, 4, 1, 0, "bm25")
    idf, lbar = math.log(4.0 / 3.0), 10.0 / 3.0
    D4, D2 = 0.25 + 0.75 * (4 / lbar), 0.25 + 0.75 * (2 / lbar)
    assert abs(r["score"][0, 0] - idf * (4 * 2.2) / (4 + 1.2 * D4)) < 1e-15        # one type, tf = 4
    assert abs(r["score"][0, 1] - 4 * idf * 2.2 / (1 + 1.2 * D4)) < 1e-15          # four types, tf = 1
    assert abs(r["score"][0, 2] - idf * (2 * 2.2) / (2 + 1.2 * D2)) < 1e-15        # the short chunk: smaller D
    assert r["sel_chunks"].tolist() == [[1]]
    tt = oracle.chunk_select(ids, 8, 10, 4, 1, 0, "type_token")["score"]
    assert tt[0].tolist() == [0.25, 1.0, 0.5]                                      # the short chunk divides by 2
