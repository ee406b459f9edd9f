"""GPU parity on seeded random shapes: selection, Phase 1, Phase 2, the generation step and the
assembled-input attention against the oracle, with block sizes, prefix lengths and query counts that
divide nothing in particular."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_attention, to_dev_ids
from paper_2607_20457_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def random_workload(seed):
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3]))
    g = int(rng.choice([1, 2, 4, 8]))
    chunk = int(rng.choice([1, 3, 8, 16, 25]))
    C = int(rng.integers(2, 40))
    block_size = chunk * C
    B = int(rng.integers(1, 7))
    k = int(rng.integers(0, min(C, 6) + 1))
    sink = int(rng.integers(0, min(block_size, 70) + 1))
    return W.shrink(W.CONFIGS["tiny"], L=B * block_size, block_size=block_size, chunk=chunk, k=k, sink=sink,
                    vocab_size=int(rng.choice([50, 1000, 40000])), Hq=Hkv * g, Hkv=Hkv, d=d,
                    nq=int(rng.integers(1, 150)), ids_seed=seed)


@pytest.mark.parametrize("seed", range(16))
def test_whole_path_on_a_random_shape(seed):
    w = random_workload(seed)
    ids = W.token_ids(w)
    Q, K, V = W.qkv(w, seed=seed + 3)
    Qq = W.phase2_query(w, seed=seed + 5)
    st = binding.new_status(DEV)
    sel = binding.pulsar_maxidf_select(to_dev_ids(ids, DEV), w.vocab_size, w.block_size, w.chunk, w.k, w.sink, status=st)
    ref = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    np.testing.assert_array_equal(sel["sel_chunks"].cpu().numpy(), ref["sel_chunks"])
    np.testing.assert_array_equal(sel["prefix_idx"].cpu().numpy(), ref["prefix_idx"])
    np.testing.assert_array_equal(sel["prefix_len"].cpu().numpy(), ref["prefix_len"])
    Qd, Kd, Vd = Q.to(DEV), K.to(DEV), V.to(DEV)
    O, LSE, _, _ = binding.pulsar_phase1_attn(Qd, Kd, Vd, w.block_size, sel["prefix_idx"], sel["prefix_len"], status=st)
    O_ref, L_ref = oracle.phase1_attn(Q, K, V, w.block_size, ref["prefix_idx"], ref["prefix_len"])
    check_attention(O, LSE, O_ref, L_ref, f"phase 1 {w}")
    O2, LSE2 = binding.pulsar_phase2_attn(Qq.to(DEV), Kd, Vd, w.n_blocks, w.block_size, status=st)
    O2_ref, L2_ref = oracle.phase2_attn(Qq, K, V, w.n_blocks, w.block_size)
    check_attention(O2, LSE2, O2_ref, L2_ref, f"phase 2 {w}")
    torch.cuda.synchronize()
    assert int(st.item()) == 0


@pytest.mark.parametrize("seed", range(6))
def test_assembled_inputs_and_generation_on_a_random_shape(seed):
    w = random_workload(100 + seed)
    rng = np.random.default_rng(seed)
    Q, K, V = W.qkv(w, seed=seed + 11)
    # assembled inputs: cut the rows into sequences of random lengths
    cuts = sorted(set(rng.integers(1, w.L, size=min(5, w.L - 1)).tolist()))
    cu = [0] + cuts + [w.L]
    O, LSE = binding.pulsar_causal_varlen_attn(Q.to(DEV), K.to(DEV), V.to(DEV), cu)
    O_ref, L_ref = oracle.causal_varlen_attn(Q, K, V, np.asarray(cu, np.int32))
    check_attention(O, LSE, O_ref, L_ref, f"assembled {cu}")
    # two generation steps: n_new tokens, then one
    n_new = int(rng.integers(1, 20))
    cap = 64
    Kg = torch.zeros(cap, w.Hkv, w.d, dtype=torch.bfloat16, device=DEV)
    Vg = torch.zeros_like(Kg)
    Kg_o, Vg_o = np.zeros((cap, w.Hkv, w.d), np.uint16), np.zeros((cap, w.Hkv, w.d), np.uint16)
    gen_len = 0
    for n in (n_new, 1):
        g = torch.Generator().manual_seed(seed * 7 + n)
        Qn = torch.randn((n, w.Hq, w.d), generator=g).bfloat16()
        Kn = torch.randn((n, w.Hkv, w.d), generator=g).bfloat16()
        Vn = torch.randn((n, w.Hkv, w.d), generator=g).bfloat16()
        Og, Lg = binding.pulsar_phase2_generate_step(Qn.to(DEV), Kn.to(DEV), Vn.to(DEV), K.to(DEV), V.to(DEV),
                                                     w.n_blocks, w.block_size, Kg, Vg, gen_len)
        Og_ref, Lg_ref = oracle.generate_step(Qn, Kn, Vn, K, V, Kg_o, Vg_o, gen_len)
        check_attention(Og, Lg, Og_ref, Lg_ref, f"generation step n={n} gen_len={gen_len}")
        gen_len += n
