"""Pins for the attention oracles (Phase 1, Phase 2, merge).

Independent formulations: dense attention with a materialised multiplicity
matrix (numpy), a library causal attention routine for block 0, a single softmax
over all keys written with numpy, closed-form log-sum-exp for the merge.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_20457_b200 import workloads as W


def f64(x):
    return x.to(torch.float64).numpy()


def small_workload(**kw):
    base = dict(L=256, block_size=64, chunk=8, k=2, sink=8, vocab_size=64, Hq=4, Hkv=2, d=16, nq=5)
    base.update(kw)
    return W.shrink(W.CONFIGS["tiny"], name="small", **base)


def dense_multiplicity_attention(Q, K, V, w, pidx, plen, scale):
    """Eq. 1 with an explicit L x L multiplicity matrix M[q][j] = number of times key
    j occurs in q's assembled key list (2 when a sink token is also in a summary)."""
    L = w.L
    M = np.zeros((L, L))
    for p in range(L):
        i = p // w.block_size
        for j in pidx[: plen[i]]:
            M[p, j] += 1
        M[p, i * w.block_size: p + 1] += 1
    q, k, v = f64(Q), f64(K), f64(V)
    g = w.Hq // w.Hkv
    O = np.zeros((L, w.Hq, w.d))
    LSE = np.zeros((L, w.Hq))
    for h in range(w.Hq):
        S = q[:, h] @ k[:, h // g].T * scale
        mx = np.where(M > 0, S, -np.inf).max(axis=1, keepdims=True)
        E = M * np.exp(S - mx)
        den = E.sum(1)
        O[:, h] = (E @ v[:, h // g]) / den[:, None]
        LSE[:, h] = mx[:, 0] + np.log(den)
    return O, LSE, M


@pytest.mark.parametrize("q_scale", [1.0, 4.0])
def test_phase1_equals_dense_attention_with_multiplicity_mask(q_scale):
    w = small_workload()
    ids = W.needle_ids(W.shrink(w, vocab_size=4096))
    # force the overlap case: the first summary chunks of block 0 lie inside the sink
    sel = oracle.maxidf_select(np.zeros(w.L, np.uint32), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    Q, K, V = W.qkv(w, q_scale=q_scale)
    scale = 1.0 / np.sqrt(w.d)
    for s in (sel, oracle.maxidf_select(ids, 4096, w.block_size, w.chunk, w.k, w.sink)):
        pidx, plen = s["prefix_idx"], s["prefix_len"]
        O, LSE = oracle.phase1_attn(Q, K, V, w.block_size, pidx, plen)
        Od, Ld, M = dense_multiplicity_attention(Q, K, V, w, pidx, plen, scale)
        np.testing.assert_allclose(O, Od, rtol=0, atol=1e-12)
        np.testing.assert_allclose(LSE, Ld, rtol=0, atol=1e-12)
    # the all-ties selection duplicates sink tokens: multiplicity 2 must occur
    _, _, M = dense_multiplicity_attention(Q, K, V, w, sel["prefix_idx"], sel["prefix_len"], scale)
    assert M.max() == 2


def test_phase1_with_a_short_last_block_and_short_chunks():
    """L = 230 in blocks of 64 (the last one holds 38 tokens) and chunks of 7 (the last chunk of a
    block holds 1 token): the dense multiplicity-matrix attention again, and the short block with an
    empty prefix equals library causal attention over its 38 rows."""
    w = small_workload(L=230, chunk=7, k=3, sink=10)
    assert w.n_blocks == 4 and w.L - 3 * w.block_size == 38
    ids = np.random.default_rng(4).integers(0, 40, size=w.L).astype(np.uint32)
    ids[63] = 41                                              # block 0's one-token chunk holds a unique id
    sel = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    assert 9 in sel["sel_chunks"][0] and sel["prefix_len"][1] == w.sink + 2 * 7 + 1
    Q, K, V = W.qkv(w, q_scale=2.0)
    pidx, plen = sel["prefix_idx"], sel["prefix_len"]
    O, LSE = oracle.phase1_attn(Q, K, V, w.block_size, pidx, plen)
    Od, Ld, _ = dense_multiplicity_attention(Q, K, V, w, pidx, plen, 1.0 / np.sqrt(w.d))
    np.testing.assert_allclose(O, Od, rtol=0, atol=1e-12)
    np.testing.assert_allclose(LSE, Ld, rtol=0, atol=1e-12)
    # the short block alone
    lo = 3 * w.block_size
    Ob, _ = oracle.phase1_attn(Q, K, V, w.block_size, pidx, np.zeros(4, np.int32), rows=np.arange(lo, w.L))
    g = w.Hq // w.Hkv
    q = Q[lo:].to(torch.float64).permute(1, 0, 2)[None]
    k = K[lo:].to(torch.float64).repeat_interleave(g, dim=1).permute(1, 0, 2)[None]
    v = V[lo:].to(torch.float64).repeat_interleave(g, dim=1).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)[0]
    np.testing.assert_allclose(Ob, ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


def test_block0_is_plain_causal_attention_library_routine():
    w = small_workload()
    Q, K, V = W.qkv(w)
    pidx, plen = W.first_k_prefix(w)
    rows = np.arange(w.block_size)
    O, _ = oracle.phase1_attn(Q, K, V, w.block_size, pidx, plen, rows=rows)
    g = w.Hq // w.Hkv
    q = Q[: w.block_size].to(torch.float64).permute(1, 0, 2)[None]
    k = K[: w.block_size].to(torch.float64).repeat_interleave(g, dim=1).permute(1, 0, 2)[None]
    v = V[: w.block_size].to(torch.float64).repeat_interleave(g, dim=1).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)[0]
    np.testing.assert_allclose(O, ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


def test_single_block_or_empty_prefix_is_block_diagonal_causal():
    w = small_workload()
    Q, K, V = W.qkv(w)
    empty = np.zeros(0, np.int32)
    O, LSE = oracle.phase1_attn(Q, K, V, w.block_size, empty, np.zeros(w.n_blocks, np.int32))
    # each block on its own, as a one-block sequence
    for b in range(w.n_blocks):
        sl = slice(b * w.block_size, (b + 1) * w.block_size)
        Ob, Lb = oracle.phase1_attn(Q[sl], K[sl], V[sl], w.block_size, empty, np.zeros(1, np.int32))
        np.testing.assert_array_equal(O[sl], Ob)
        np.testing.assert_array_equal(LSE[sl], Lb)
    # first row of every block sees one key only: output = that value row, LSE = its logit
    g = w.Hq // w.Hkv
    for b in range(w.n_blocks):
        p = b * w.block_size
        for h in range(w.Hq):
            np.testing.assert_allclose(O[p, h], f64(V)[p, h // g], atol=1e-15)
            z = float(f64(Q)[p, h] @ f64(K)[p, h // g]) / np.sqrt(w.d)
            assert abs(LSE[p, h] - z) < 1e-12


def test_row_subset_matches_full_run_and_custom_scale():
    w = small_workload()
    Q, K, V = W.qkv(w)
    pidx, plen = W.first_k_prefix(w)
    O, LSE = oracle.phase1_attn(Q, K, V, w.block_size, pidx, plen, scale=0.37)
    rows = np.asarray([0, 63, 64, 100, 255])
    Or, Lr = oracle.phase1_attn(Q, K, V, w.block_size, pidx, plen, scale=0.37, rows=rows)
    np.testing.assert_array_equal(O[rows], Or)
    np.testing.assert_array_equal(LSE[rows], Lr)
    Od, Ld, _ = dense_multiplicity_attention(Q, K, V, w, pidx, plen, 0.37)
    np.testing.assert_allclose(O, Od, atol=1e-12)


def test_poisoned_invisible_rows_do_not_leak():
    w = small_workload()
    Q, K, V = W.qkv(w)
    pidx, plen = W.first_k_prefix(w)
    O, LSE = oracle.phase1_attn(Q, K, V, w.block_size, pidx, plen)
    rows = np.arange(2 * w.block_size, 2 * w.block_size + 10)       # block 2, rows 0..9
    visible = set(pidx[: plen[2]].tolist()) | set(range(2 * w.block_size, 2 * w.block_size + 10))
    K2, V2 = K.clone(), V.clone()
    for j in range(w.L):
        if j not in visible:
            V2[j] = 3.0e4
            K2[j] = K2[j] * 8
    O2, L2 = oracle.phase1_attn(Q, K2, V2, w.block_size, pidx, plen, rows=rows)
    np.testing.assert_array_equal(O[rows], O2)
    np.testing.assert_array_equal(LSE[rows], L2)


def numpy_global_softmax(Qq, K, V, w, scale):
    q, k, v = f64(Qq), f64(K), f64(V)
    g = w.Hq // w.Hkv
    O = np.zeros((q.shape[0], w.Hq, w.d))
    LSE = np.zeros((q.shape[0], w.Hq))
    for h in range(w.Hq):
        S = q[:, h] @ k[:, h // g].T * scale
        mx = S.max(1, keepdims=True)
        E = np.exp(S - mx)
        O[:, h] = (E / E.sum(1, keepdims=True)) @ v[:, h // g]
        LSE[:, h] = mx[:, 0] + np.log(E.sum(1))
    return O, LSE


@pytest.mark.parametrize("q_scale", [1.0, 6.0])
def test_phase2_is_one_softmax_over_all_retained_keys(q_scale):
    w = small_workload()
    _, K, V = W.qkv(w)
    Qq = W.phase2_query(w, q_scale=q_scale)
    O, LSE, pO, pL = oracle.phase2_attn(Qq, K, V, w.n_blocks, w.block_size, partials=True)
    Oref, Lref = numpy_global_softmax(Qq, K, V, w, 1 / np.sqrt(w.d))
    np.testing.assert_allclose(O, Oref, atol=1e-12)
    np.testing.assert_allclose(LSE, Lref, atol=1e-12)
    # per-block partials are the same routine on one block
    for b in range(w.n_blocks):
        sl = slice(b * w.block_size, (b + 1) * w.block_size)
        Ob, Lb = numpy_global_softmax(Qq, K[sl], V[sl], w, 1 / np.sqrt(w.d))
        np.testing.assert_allclose(pO[b], Ob, atol=1e-12)
        np.testing.assert_allclose(pL[b], Lb, atol=1e-12)


def test_merge_recovers_global_attention_and_is_order_and_split_invariant():
    w = small_workload()
    _, K, V = W.qkv(w)
    Qq = W.phase2_query(w, q_scale=3.0)
    O, LSE, pO, pL = oracle.phase2_attn(Qq, K, V, w.n_blocks, w.block_size, partials=True)
    R = w.nq * w.Hq
    flatO, flatL = pO.reshape(w.n_blocks, R, w.d), pL.reshape(w.n_blocks, R)
    Om, Lm = oracle.lse_merge(flatO, flatL)
    np.testing.assert_allclose(Om, O.reshape(R, w.d), atol=1e-12)
    np.testing.assert_allclose(Lm, LSE.reshape(R), atol=1e-12)
    # closed form: l = m + ln sum exp(l_b - m); o = sum exp(l_b - l) o_b
    m = flatL.max(0)
    lc = m + np.log(np.exp(flatL - m).sum(0))
    oc = (np.exp(flatL - lc)[..., None] * flatO).sum(0)
    np.testing.assert_allclose(Lm, lc, atol=1e-12)
    np.testing.assert_allclose(Om, oc, atol=1e-12)
    # permutation of the parts
    perm = [2, 0, 3, 1]
    Op, Lp = oracle.lse_merge(flatO[perm], flatL[perm])
    np.testing.assert_allclose(Op, Om, atol=1e-12)
    np.testing.assert_allclose(Lp, Lm, atol=1e-12)
    # a different split of the same keys (2 blocks of 128) gives the same merged result
    O2, L2, pO2, pL2 = oracle.phase2_attn(Qq, K, V, 2, 128, partials=True)
    Om2, Lm2 = oracle.lse_merge(pO2.reshape(2, R, w.d), pL2.reshape(2, R))
    np.testing.assert_allclose(Om2, Om, atol=1e-12)
    np.testing.assert_allclose(O2, O, atol=1e-12)
    # one part: the merge is the identity
    O1, L1 = oracle.lse_merge(flatO[:1], flatL[:1])
    np.testing.assert_array_equal(O1, flatO[0])
    np.testing.assert_array_equal(L1, flatL[0])


def test_merge_two_parts_by_hand():
    # l = ln(e^0 + e^ln3) = ln 4 ; weights 1/4 and 3/4
    pO = np.asarray([[[1.0, 0.0]], [[0.0, 2.0]]])
    pL = np.asarray([[0.0], [np.log(3.0)]])
    O, L = oracle.lse_merge(pO, pL)
    np.testing.assert_allclose(L, [np.log(4.0)], atol=1e-15)
    np.testing.assert_allclose(O, [[0.25, 1.5]], atol=1e-15)


def test_uniform_keys_closed_form():
    # identical keys -> uniform weights: O = mean of V, LSE = z + ln n
    w = small_workload()
    Q, K, V = W.qkv(w)
    K[:] = K[0:1]
    Qq = W.phase2_query(w)
    O, LSE = oracle.phase2_attn(Qq, K, V, w.n_blocks, w.block_size)
    g = w.Hq // w.Hkv
    for h in range(w.Hq):
        np.testing.assert_allclose(O[:, h], np.broadcast_to(f64(V)[:, h // g].mean(0), O[:, h].shape), atol=1e-12)
        z = f64(Qq)[:, h] @ f64(K)[0, h // g] / np.sqrt(w.d)
        np.testing.assert_allclose(LSE[:, h], z + np.log(w.L), atol=1e-12)


def _bits_of(t):
    return np.ascontiguousarray(t.contiguous().view(torch.int16).numpy().view(np.uint16))


def test_generate_step_is_one_softmax_over_context_and_causal_shard():
    # Algorithm 1 lines 11-16: query tokens, then generated tokens, are appended to the generation
    # shard and attend to all context keys plus the shard up to themselves.
    w = small_workload()
    _, K, V = W.qkv(w)
    cap, g = 16, w.Hq // w.Hkv
    gen = torch.Generator().manual_seed(9)
    Kgen = np.zeros((cap, w.Hkv, w.d), np.uint16)
    Vgen = np.zeros((cap, w.Hkv, w.d), np.uint16)
    gen_len = 0
    hist_K, hist_V = [], []
    for n_new in (5, 1, 1, 3):                                  # the query first, then single tokens
        Qn = torch.randn(n_new, w.Hq, w.d, generator=gen).to(torch.bfloat16)
        Kn = torch.randn(n_new, w.Hkv, w.d, generator=gen).to(torch.bfloat16)
        Vn = torch.randn(n_new, w.Hkv, w.d, generator=gen).to(torch.bfloat16)
        O, LSE = oracle.generate_step(Qn, Kn, Vn, K, V, Kgen, Vgen, gen_len)
        hist_K.append(Kn); hist_V.append(Vn)
        Kall = torch.cat([K] + hist_K); Vall = torch.cat([V] + hist_V)
        # the shard now holds exactly the appended rows
        np.testing.assert_array_equal(Kgen[: gen_len + n_new], _bits_of(torch.cat(hist_K)))
        np.testing.assert_array_equal(Vgen[: gen_len + n_new], _bits_of(torch.cat(hist_V)))
        for u in range(n_new):
            n_keys = w.L + gen_len + u + 1
            k, v, q = f64(Kall[:n_keys]), f64(Vall[:n_keys]), f64(Qn[u])
            for h in range(w.Hq):
                zz = k[:, h // g] @ q[h] / np.sqrt(w.d)
                e = np.exp(zz - zz.max())
                np.testing.assert_allclose(O[u, h], (e / e.sum()) @ v[:, h // g], atol=1e-12)
                assert abs(LSE[u, h] - (zz.max() + np.log(e.sum()))) < 1e-12
        gen_len += n_new
    # the newest token with an empty history and a one-token step is plain Phase 2 over context + itself
    Kgen2 = np.zeros((4, w.Hkv, w.d), np.uint16); Vgen2 = np.zeros_like(Kgen2)
    Qn, Kn, Vn = hist_K[1].repeat_interleave(g, 1), hist_K[1], hist_V[1]
    O1, L1 = oracle.generate_step(Qn, Kn, Vn, K, V, Kgen2, Vgen2, 0)
    O2, L2 = oracle.phase2_attn(Qn, torch.cat([K, Kn]), torch.cat([V, Vn]), 1, w.L + 1)
    np.testing.assert_allclose(O1, O2, atol=1e-12)
    np.testing.assert_allclose(L1, L2, atol=1e-12)


def test_varlen_causal_is_library_causal_attention_per_sequence():
    w = small_workload()
    Q, K, V = W.qkv(w)
    cu = [0, 37, 101, 256]
    O, LSE = oracle.causal_varlen_attn(Q, K, V, cu)
    g = w.Hq // w.Hkv
    for a, b in zip(cu[:-1], cu[1:]):
        q = Q[a:b].to(torch.float64).permute(1, 0, 2)[None]
        k = K[a:b].to(torch.float64).repeat_interleave(g, dim=1).permute(1, 0, 2)[None]
        v = V[a:b].to(torch.float64).repeat_interleave(g, dim=1).permute(1, 0, 2)[None]
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)[0]
        np.testing.assert_allclose(O[a:b], ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)
