"""GPU parity: position ids of the assembled inputs (exact) and rotary embedding (Appendix E)
against the float64 oracle.  Tolerance: the result is rounded once to bf16 (relative 2^-9) from
float32 products of a float32 sine/cosine whose angle was formed in float64, so
|dY| <= 2^-8 * (|x_j| + |x_{j+d/2}|) + 1e-6 element by element."""
import numpy as np
import pytest
import torch

import oracle
from helpers import to_dev_ids
from paper_2607_20457_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def check_rope(X, pos, theta):
    st = binding.new_status(DEV)
    Y = binding.pulsar_rope_apply(X.to(DEV), torch.from_numpy(pos).to(DEV), theta, status=st)
    ref = oracle.rope_apply(X, pos, theta)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    x = X.double().numpy()
    half = X.shape[-1] // 2
    mag = np.abs(x[..., :half]) + np.abs(x[..., half:])
    bound = 2.0 ** -8 * np.concatenate([mag, mag], axis=-1) + 1e-6
    err = np.abs(Y.double().cpu().numpy() - ref)
    assert (err <= bound).all(), float((err / bound).max())
    return Y


@pytest.mark.parametrize("H,d", [(32, 128), (8, 128), (4, 64), (3, 16), (2, 256)])
def test_rope_matches_oracle(H, d):
    g = torch.Generator().manual_seed(H * 1000 + d)
    rows = 777
    X = torch.randn((rows, H, d), generator=g).bfloat16()
    rng = np.random.default_rng(d)
    pos = rng.integers(0, 131072, size=rows).astype(np.int32)
    pos[:4] = [0, 1, 131071, 2 ** 31 - 1]                  # identity, smallest step, the 128K end, the largest id
    check_rope(X, pos, 500000.0 if d != 64 else 10000.0)


def test_rope_in_place_and_sparse_positions_of_an_assembled_input():
    w = W.CONFIGS["16k"]
    ids = W.needle_ids(w)
    sel = binding.pulsar_maxidf_select(to_dev_ids(ids, DEV), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    ref = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    total = int(ref["prefix_len"].sum()) + w.n_blocks * w.block_size
    for mode in ("sparse", "contiguous"):
        st = binding.new_status(DEV)
        pos = binding.pulsar_assemble_positions(sel["prefix_idx"], sel["prefix_len"], w.n_blocks, w.block_size, total,
                                                mode, status=st)
        want = oracle.assemble_positions(ref["prefix_idx"], ref["prefix_len"], w.block_size, mode)
        assert int(st.item()) == 0
        np.testing.assert_array_equal(pos.cpu().numpy(), want)
    # the last assembled input, rotated in place at its sparse positions
    n_last = int(ref["prefix_len"][-1]) + w.block_size
    pos_last = oracle.assemble_positions(ref["prefix_idx"], ref["prefix_len"], w.block_size, "sparse")[-n_last:]
    g = torch.Generator().manual_seed(5)
    X = torch.randn((n_last, w.Hkv, w.d), generator=g).bfloat16()
    Xd = X.to(DEV)
    Y = check_rope(X, pos_last, 500000.0)
    binding.pulsar_rope_apply(Xd, torch.from_numpy(pos_last).to(DEV), 500000.0, out=Xd)
    assert torch.equal(Xd, Y)


def test_rope_qk_in_one_launch_equals_two():
    g = torch.Generator().manual_seed(21)
    rows = 1003
    Q = torch.randn((rows, 32, 128), generator=g).bfloat16().to(DEV)
    K = torch.randn((rows, 8, 128), generator=g).bfloat16().to(DEV)
    pos = torch.randint(0, 131072, (rows,), generator=g, dtype=torch.int32).to(DEV)
    Qo, Ko = binding.pulsar_rope_apply_qk(Q, K, pos)
    assert torch.equal(Qo, binding.pulsar_rope_apply(Q, pos)) and torch.equal(Ko, binding.pulsar_rope_apply(K, pos))
    binding.pulsar_rope_apply_qk(Q, K, pos, q_out=Q, k_out=K)              # in place
    assert torch.equal(Q, Qo) and torch.equal(K, Ko)


def test_rope_keeps_attention_scores_relative():
    """q at position m against k at position n gives the same logit as at (m+s, n+s): checked on the
    GPU results within bf16 rounding of the rotated vectors."""
    g = torch.Generator().manual_seed(9)
    q = torch.randn((1, 1, 128), generator=g).bfloat16().to(DEV)
    k = torch.randn((1, 1, 128), generator=g).bfloat16().to(DEV)
    def logit(m, n):
        qr = binding.pulsar_rope_apply(q, torch.tensor([m], dtype=torch.int32, device=DEV))
        kr = binding.pulsar_rope_apply(k, torch.tensor([n], dtype=torch.int32, device=DEV))
        return float((qr.float() * kr.float()).sum())
    base = logit(100, 40)
    assert abs(logit(100000, 99940) - base) < 0.25 and abs(logit(8292, 8232) - base) < 0.25


def test_negative_position_and_bad_shapes():
    X = torch.randn((4, 2, 32), device=DEV).bfloat16()
    st = binding.new_status(DEV)
    pos = torch.tensor([0, -5, 2, 3], dtype=torch.int32, device=DEV)
    Y = binding.pulsar_rope_apply(X, pos, 10000.0, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) & binding.DEV_BAD_POSITION and torch.equal(Y[1], X[1])     # counted as position 0
    with pytest.raises(binding.PulsarError):
        binding.pulsar_rope_apply(torch.randn((4, 2, 24), device=DEV).bfloat16(), pos, 10000.0)


def test_rope_full_size_rows_sampled_against_the_oracle():
    """131,072 rows of 32 + 8 heads in one launch (the shape the bench times), 1500 rows checked."""
    rows = 131072
    g = torch.Generator().manual_seed(4)
    Q = torch.randn((rows, 32, 128), generator=g, dtype=torch.bfloat16)
    K = torch.randn((rows, 8, 128), generator=g, dtype=torch.bfloat16)
    pos = np.arange(rows, dtype=np.int32)                       # sparse mode of an unassembled sequence: global positions
    st = binding.new_status(DEV)
    Qo, Ko = binding.pulsar_rope_apply_qk(Q.to(DEV), K.to(DEV), torch.from_numpy(pos).to(DEV), status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    pick = np.unique(np.concatenate([np.arange(8), np.arange(rows - 8, rows),
                                     np.random.default_rng(0).integers(0, rows, size=1500)]))
    for X, Y in ((Q, Qo), (K, Ko)):
        ref = oracle.rope_apply(X[pick], pos[pick], 500000.0)
        x = X[pick].double().numpy()
        mag = np.abs(x[..., :64]) + np.abs(x[..., 64:])
        bound = 2.0 ** -8 * np.concatenate([mag, mag], axis=-1) + 1e-6
        err = np.abs(Y[torch.from_numpy(pick).to(DEV)].double().cpu().numpy() - ref)
        assert (err <= bound).all(), float((err / bound).max())


def test_position_ids_of_a_sequence_with_a_short_last_block():
    """The last assembled input of a sequence that ends inside a block is shorter: the call takes the
    total number of rows, and what lies beyond it is not written.  Expected ids written out directly
    from the definition (sparse: a prefix entry keeps its position, row r of block i is i*n_b + r)."""
    w = W.shrink(W.CONFIGS["tiny"], L=3000, block_size=1024, chunk=24, k=5, sink=64, vocab_size=4096)
    ids = W.zipf_ids(w.L, w.vocab_size, 1.3, 9)
    sel = binding.pulsar_maxidf_select(to_dev_ids(ids, DEV), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    ref = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    lens = [min(w.block_size, w.L - i * w.block_size) for i in range(w.n_blocks)]
    total = int(ref["prefix_len"].sum()) + sum(lens)
    for mode in ("sparse", "contiguous"):
        want = []
        for i, n in enumerate(lens):
            P = int(ref["prefix_len"][i])
            want += (ref["prefix_idx"][:P].tolist() if mode == "sparse" else list(range(P)))
            want += [i * w.block_size + r if mode == "sparse" else P + r for r in range(n)]
        pos = binding.pulsar_assemble_positions(sel["prefix_idx"], sel["prefix_len"], w.n_blocks, w.block_size, total, mode)
        assert pos.cpu().tolist() == want
