"""Pins for the oracle's position-id assembly and rotary embedding (Appendix E), independent of it:
complex-number rotation in numpy, norm preservation, the relative-position property, position 0,
a hand case with d = 2, and the layout of the assembled position ids."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2607_20457_b200 import workloads as W


def rand_bf16(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g).bfloat16()


def test_rope_equals_complex_rotation():
    X = rand_bf16((23, 3, 16), 1)
    pos = np.array([0, 1, 2, 5, 100, 4095, 131071] + list(range(7, 23)), np.int32)
    theta = 500000.0
    Y = oracle.rope_apply(X, pos, theta)
    x = X.double().numpy()
    half = 8
    z = x[..., :half] + 1j * x[..., half:]                      # pair (j, j + d/2) as one complex number
    ang = pos[:, None].astype(np.float64) * theta ** (-np.arange(half) / half)
    zr = z * np.exp(1j * ang)[:, None, :]
    np.testing.assert_allclose(Y[..., :half], zr.real, rtol=0, atol=1e-9)
    np.testing.assert_allclose(Y[..., half:], zr.imag, rtol=0, atol=1e-9)


def test_rope_position_zero_is_identity_and_norms_are_kept():
    X = rand_bf16((9, 2, 32), 2)
    Y0 = oracle.rope_apply(X, np.zeros(9, np.int32))
    np.testing.assert_array_equal(Y0, X.double().numpy())
    Y = oracle.rope_apply(X, np.arange(9, dtype=np.int32) * 1000 + 3)
    np.testing.assert_allclose((Y ** 2).sum(-1), (X.double().numpy() ** 2).sum(-1), rtol=1e-12)


def test_rope_scores_depend_on_relative_position_only():
    q, k = rand_bf16((1, 1, 64), 3), rand_bf16((1, 1, 64), 4)
    dots = []
    for m, n in [(10, 3), (1007, 1000), (50007, 50000)]:
        qr = oracle.rope_apply(q, np.array([m], np.int32), 10000.0)
        kr = oracle.rope_apply(k, np.array([n], np.int32), 10000.0)
        dots.append(float((qr * kr).sum()))
    assert abs(dots[0] - dots[1]) < 1e-9 and abs(dots[0] - dots[2]) < 1e-8
    other = float((oracle.rope_apply(q, np.array([11], np.int32), 10000.0) *
                   oracle.rope_apply(k, np.array([3], np.int32), 10000.0)).sum())
    assert abs(other - dots[0]) > 1e-3                             # a different distance does change it


def test_rope_by_hand_d2_and_frequency_of_the_last_pair():
    X = torch.tensor([[[1.0, 0.0]], [[0.0, 2.0]]]).bfloat16()      # d = 2: one pair, frequency theta^0 = 1
    Y = oracle.rope_apply(X, np.array([1, 3], np.int32), 10000.0)
    np.testing.assert_allclose(Y[0, 0], [math.cos(1), math.sin(1)], atol=1e-15)
    np.testing.assert_allclose(Y[1, 0], [-2 * math.sin(3), 2 * math.cos(3)], atol=1e-15)
    X = torch.zeros(1, 1, 4).bfloat16(); X[0, 0, 1] = 1.0            # d = 4, pair j = 1: frequency theta^(-1/2)
    Y = oracle.rope_apply(X, np.array([50], np.int32), 10000.0)
    np.testing.assert_allclose(Y[0, 0], [0, math.cos(0.5), 0, math.sin(0.5)], atol=1e-15)


@pytest.mark.parametrize("mode", ["sparse", "contiguous"])
def test_assembled_position_ids(mode):
    w = W.CONFIGS["tiny"]
    ref = oracle.maxidf_select(W.needle_ids(w), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    pos = oracle.assemble_positions(ref["prefix_idx"], ref["prefix_len"], w.block_size, mode)
    at = 0
    for i in range(w.n_blocks):
        P = int(ref["prefix_len"][i])
        seg = pos[at: at + P + w.block_size]
        if mode == "sparse":
            assert seg[:P].tolist() == ref["prefix_idx"][:P].tolist()
            assert seg[P:].tolist() == list(range(i * w.block_size, (i + 1) * w.block_size))
            assert (np.diff(seg) > 0).all()                      # gaps, but still increasing
            if i > 0:
                assert seg[: w.sink].tolist() == list(range(w.sink))
        else:
            assert seg.tolist() == list(range(P + w.block_size))
        at += P + w.block_size
    assert at == len(pos)
