"""GPU parity: Phase-2 split-KV attention and the LSE merge against the oracle (Section 3.2, App. H)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_attention, TOL_LSE_ABS
from paper_2607_20457_b200 import binding, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_phase2(w, Qq, K, V, n_splits=0, what="", scale=0.0, rows=None):
    """The GPU always runs the whole query; ``rows`` limits the oracle (and the comparison) to some
    query rows -- every query row is an independent softmax, so a subset is a query of its own."""
    status = binding.new_status(DEV)
    O, LSE = binding.pulsar_phase2_attn(Qq.to(DEV), K.to(DEV), V.to(DEV), w.n_blocks, w.block_size,
                                        softmax_scale=scale, n_splits=n_splits, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    if rows is not None:
        idx = torch.as_tensor(np.asarray(rows))
        Qq, O, LSE = Qq[idx].contiguous(), O[idx.to(DEV)], LSE[idx.to(DEV)]
    Oref, Lref = oracle.phase2_attn(Qq, K, V, w.n_blocks, w.block_size, scale=scale)
    return check_attention(O, LSE, Oref, Lref, what)


def tile_edge_rows(nq, g, per_tile=2):
    """Query tokens at the first and last row of row tiles (128 rows = 128/g tokens x g heads) and of
    tile pairs, spread over the query, plus the last token."""
    tok = 128 // g
    tiles = -(-nq // tok)
    pick = sorted(set([0, 1, tiles // 2, tiles - 2, tiles - 1]) & set(range(tiles)))
    rows = []
    for t in pick:
        rows += [t * tok, min(nq, (t + 1) * tok) - 1]
    return sorted(set(rows + [nq - 1]))


@pytest.mark.parametrize("n_splits", [0, 1, 4, 32])
def test_tiny_config(n_splits):
    w = W.CONFIGS["tiny"]
    _, K, V = W.qkv(w)
    print(run_phase2(w, W.phase2_query(w), K, V, n_splits, what=f"tiny J={n_splits}"))


def test_tiny_peaked():
    w = W.CONFIGS["tiny"]
    _, K, V = W.qkv(w)
    print(run_phase2(w, W.phase2_query(w, q_scale=6.0), K, V, 4, what="tiny peaked"))


@pytest.mark.parametrize("shape", [
    dict(L=1000, block_size=250, Hq=4, Hkv=2, d=128, nq=1),       # decode shape, ragged keys
    dict(L=768, block_size=192, Hq=8, Hkv=1, d=64, nq=17),        # g = 8, ragged rows
    dict(L=512, block_size=128, Hq=2, Hkv=2, d=128, nq=130),      # g = 1, more than one row tile
    dict(L=640, block_size=320, Hq=16, Hkv=1, d=64, nq=9),        # g = 16
    # decode shapes: at most 32 query rows per KV head, each softmax warp takes a quarter of the keys
    dict(L=640, block_size=320, Hq=16, Hkv=1, d=64, nq=2),        # g = 16, 32 rows
    dict(L=900, block_size=300, Hq=8, Hkv=1, d=128, nq=3),        # g = 8, 24 rows, ragged keys
    dict(L=512, block_size=256, Hq=2, Hkv=2, d=128, nq=32),       # g = 1, 32 rows
    dict(L=512, block_size=256, Hq=2, Hkv=2, d=64, nq=33),        # g = 1, one row too many for that mode
    dict(L=1152, block_size=384, Hq=4, Hkv=2, d=128, nq=16),      # g = 2, 32 rows
    dict(L=90, block_size=45, Hq=4, Hkv=1, d=64, nq=5),           # fewer keys than one tile
    # one or two query tiles per KV head and several parts
    dict(L=1280, block_size=640, Hq=8, Hkv=2, d=128, nq=40),      # g = 4, 160 rows: two query tiles, the second ragged
    dict(L=1280, block_size=640, Hq=8, Hkv=2, d=64, nq=64),       # 256 rows exactly
    dict(L=256, block_size=128, Hq=4, Hkv=1, d=128, nq=20),       # two parts of one key tile
    dict(L=1000, block_size=500, Hq=16, Hkv=4, d=128, nq=33),     # odd key-tile counts per part, ragged last tile
])
@pytest.mark.parametrize("n_splits", [1, 2])
def test_small_shapes(shape, n_splits):
    w = W.shrink(W.CONFIGS["tiny"], **shape)
    _, K, V = W.qkv(w)
    print(run_phase2(w, W.phase2_query(w, q_scale=2.0), K, V, n_splits, what=f"{shape} J={n_splits}", scale=0.2))


@pytest.mark.parametrize("nq", [1, 8, 20, 32, 40, 64, 70])
@pytest.mark.parametrize("n_splits", [1, 2])
def test_row_maximum_jumps_at_late_key_tiles(nq, n_splits):
    """One query row's logits jump by far more than the kernel's lazy-rescale threshold at two later
    key tiles, so the accumulated output is rescaled there while the other rows of the same warp --
    near-uniform attention, every key tile counts -- pass through the same rescale step with factor 1.
    Covers the decode mode (nq * g <= 32), the one-tile schedule (<= 128 rows) and two and three query
    tiles per KV head."""
    L, Hq, Hkv, d, tile = 6 * 128 + 40, 8, 2, 128, 128
    w = W.shrink(W.CONFIGS["tiny"], L=L, block_size=L, Hq=Hq, Hkv=Hkv, d=d, nq=nq)
    gen = torch.Generator().manual_seed(1234 + nq)
    u = torch.zeros(d)
    u[::2] = 1.0 / (d // 2) ** 0.5                                   # unit direction
    Qq = 0.05 * torch.randn(nq, Hq, d, generator=gen)
    K = 0.05 * torch.randn(L, Hkv, d, generator=gen)
    V = torch.randn(L, Hkv, d, generator=gen)
    for h in (0, Hq - 1):                                            # one row in each KV head's group
        Qq[nq // 2, h] = 12.0 * u
    K[3 * tile:, :, :] += 3.0 * u                                    # logit + 36 * scale from key tile 3 on
    K[5 * tile + 7:, :, :] += 4.0 * u                                # and + 48 * scale more inside key tile 5
    Qq, K, V = Qq.bfloat16(), K.bfloat16(), V.bfloat16()
    print(run_phase2(w, Qq, K, V, n_splits, what=f"late maximum nq={nq} J={n_splits}", scale=0.5))


def test_per_block_partials_match_oracle_partials():
    w = W.CONFIGS["tiny"]
    _, K, V = W.qkv(w)
    Qq = W.phase2_query(w)
    O, LSE, pO, pL = binding.pulsar_phase2_attn(Qq.to(DEV), K.to(DEV), V.to(DEV), w.n_blocks, w.block_size,
                                                n_splits=w.n_blocks, want_partials=True)
    Oref, Lref, pOref, pLref = oracle.phase2_attn(Qq, K, V, w.n_blocks, w.block_size, partials=True)
    for b in range(w.n_blocks):
        check_attention(pO[b], pL[b], pOref[b], pLref[b], f"block {b} partial")
    check_attention(O, LSE, Oref, Lref, "merged")


@pytest.mark.parametrize("name,nq", [("16k", None), ("32k", None), ("64k", None), ("128k", 64), ("128k", 1)])
def test_full_size_kv(name, nq):
    """Each configuration's own query (16K and 32K: 64 rows, 64K: 128 rows) and decode-sized
    queries at 128K, library-chosen split, every query row checked."""
    w = W.CONFIGS[name]
    _, K, V = W.qkv(w)
    Qq = W.phase2_query(w, nq=nq)
    print(run_phase2(w, Qq, K, V, 0, what=f"{name} nq={Qq.shape[0]}"))


@pytest.mark.parametrize("nq", [1, 24])
def test_twice_the_largest_configuration_and_a_ragged_end(nq):
    """262,181 keys (2049 key tiles, the last one of 37 keys) as one block: twice the KV of the largest
    configuration, through the decode mode (1 token) and the one-tile schedule (24 tokens = 96 rows per
    KV head), with the split the library picks."""
    L = 2 * 131072 + 37
    w = W.shrink(W.CONFIGS["128k"], L=L, block_size=L)
    gen = torch.Generator().manual_seed(99)
    K = torch.randn(L, w.Hkv, w.d, generator=gen).to(torch.bfloat16)
    V = torch.randn(L, w.Hkv, w.d, generator=gen).to(torch.bfloat16)
    Qq = W.phase2_query(w, nq=nq, seed=17)
    rows = None if nq == 1 else [0, nq // 2, nq - 1]
    print(run_phase2(w, Qq, K, V, 0, what=f"256K+37 keys nq={nq}", rows=rows))


@pytest.mark.parametrize("n_splits", [0, 9])
def test_128k_config_own_query(n_splits):
    """The 128K configuration's own Phase-2 call -- 8 queries x 64 tokens = 512 rows, i.e. 16 row
    tiles (8 pairs) per KV head -- with the split the library picks (the launch the benchmark
    times) and with 9 parts (1024 key tiles in runs of 114, the last one shorter).  The oracle runs
    on the first and last tokens of several row tiles."""
    w = W.CONFIGS["128k"]
    assert w.nq == 512
    J = n_splits or binding.phase2_choose_splits(w.nq, w.n_blocks, w.block_size, w.Hq, w.Hkv, w.d)
    assert J > 1
    _, K, V = W.qkv(w)
    rows = tile_edge_rows(w.nq, w.Hq // w.Hkv)
    print(run_phase2(w, W.phase2_query(w), K, V, n_splits, what=f"128k nq=512 J={J} rows={rows}", rows=rows))


def test_merge_entry_point_against_oracle_merge():
    rng = np.random.default_rng(0)
    J, rows, d = 5, 333, 128
    pO = rng.standard_normal((J, rows, d))
    pL = rng.standard_normal((J, rows)) * 4
    pL[2, :7] = -np.inf                                   # an empty part has weight zero
    Oref, Lref = oracle.lse_merge(pO.astype(np.float32).astype(np.float64),
                                  np.where(np.isinf(pL), -1e30, pL.astype(np.float32).astype(np.float64)))
    O, LSE = binding.pulsar_lse_merge(torch.from_numpy(pO.astype(np.float32)).to(DEV),
                                      torch.from_numpy(pL.astype(np.float32)).to(DEV))
    torch.cuda.synchronize()
    assert np.abs(O.float().cpu().numpy() - Oref).max() <= 1e-2
    assert np.abs(LSE.cpu().numpy() - Lref).max() <= TOL_LSE_ABS
    # one part: identity up to the bf16 rounding of the output
    O1, L1 = binding.pulsar_lse_merge(torch.from_numpy(pO[:1].astype(np.float32)).to(DEV),
                                      torch.from_numpy(pL[:1].astype(np.float32)).to(DEV))
    assert torch.equal(O1, torch.from_numpy(pO[0].astype(np.float32)).to(DEV).to(torch.bfloat16))


@pytest.mark.parametrize("J,rows,d", [(16, 32, 128), (72, 32, 128), (77, 5, 64), (23, 250, 128)])
def test_merge_of_many_parts_into_few_rows(J, rows, d):
    """Decode shapes take the merge that spreads the parts of an output over lanes."""
    rng = np.random.default_rng(J)
    pO = rng.standard_normal((J, rows, d)).astype(np.float32)
    pL = (rng.standard_normal((J, rows)) * 4).astype(np.float32)
    pL[J // 2, : rows // 2] = -np.inf
    pL[:, -1] = -np.inf                                   # a row with no keys at all
    Oref, Lref = oracle.lse_merge(pO.astype(np.float64), np.where(np.isinf(pL), -1e30, pL.astype(np.float64)))
    out = torch.empty((rows, d), dtype=torch.float32, device=DEV)
    lse = torch.empty(rows, dtype=torch.float32, device=DEV)
    tO, tL = torch.from_numpy(pO).to(DEV), torch.from_numpy(pL).to(DEV)
    binding.pulsar_lse_merge_strided(tO.view(-1), tL.view(-1), J, rows * d, rows, rows, d, out, lse)
    torch.cuda.synchronize()
    got, gl = out.cpu().numpy(), lse.cpu().numpy()
    assert np.abs(got[:-1] - Oref[:-1]).max() < 5e-6 * max(1.0, np.abs(Oref).max())
    assert np.abs(gl[:-1] - Lref[:-1]).max() < 1e-5
    assert np.isneginf(gl[-1]) and (got[-1] == 0).all()
    again = torch.empty_like(out)
    binding.pulsar_lse_merge_strided(tO.view(-1), tL.view(-1), J, rows * d, rows, rows, d, again, lse)
    assert torch.equal(again, out)                        # fixed combination order


def test_phase1_then_phase2_chain_on_retained_kv():
    w = W.CONFIGS["tiny"]
    Q, K, V = W.qkv(w)
    pidx, plen = W.first_k_prefix(w)
    _, _, Kr, Vr = binding.pulsar_phase1_attn(Q.to(DEV), K.to(DEV), V.to(DEV), w.block_size,
                                              torch.from_numpy(pidx).to(DEV), torch.from_numpy(plen).to(DEV))
    Qq = W.phase2_query(w)
    O, LSE = binding.pulsar_phase2_attn(Qq.to(DEV), Kr, Vr, w.n_blocks, w.block_size)
    Oref, Lref = oracle.phase2_attn(Qq, K, V, w.n_blocks, w.block_size)
    check_attention(O, LSE, Oref, Lref, "chain")


def test_two_runs_are_bit_identical():
    w = W.CONFIGS["16k"]
    _, K, V = W.qkv(w)
    Qq = W.phase2_query(w).to(DEV)
    Kd, Vd = K.to(DEV), V.to(DEV)
    a = binding.pulsar_phase2_attn(Qq, Kd, Vd, w.n_blocks, w.block_size)
    b = binding.pulsar_phase2_attn(Qq, Kd, Vd, w.n_blocks, w.block_size)
    torch.cuda.synchronize()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


@pytest.mark.parametrize("n_splits", [3, 6])
def test_uneven_parts(n_splits):
    # 2048 keys = 16 key tiles cut into runs of whole tiles, the last run shorter: 6+6+4, 3*5+1
    w = W.shrink(W.CONFIGS["tiny"], L=2048, block_size=512, Hq=8, Hkv=2, d=128, nq=40)
    _, K, V = W.qkv(w)
    print(run_phase2(w, W.phase2_query(w, q_scale=2.0), K, V, n_splits, what=f"uneven J={n_splits}"))


def test_part_count_that_leaves_a_part_empty_is_rejected():
    # 16 key tiles in 5 parts would be runs of 4 tiles: only 4 parts are non-empty
    w = W.shrink(W.CONFIGS["tiny"], L=2048, block_size=512, Hq=8, Hkv=2, d=128, nq=8)
    _, K, V = W.qkv(w)
    with pytest.raises(binding.PulsarError) as e:
        binding.pulsar_phase2_attn(W.phase2_query(w).to(DEV), K.to(DEV), V.to(DEV), w.n_blocks, w.block_size, n_splits=5)
    assert e.value.status == 2
