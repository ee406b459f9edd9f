"""Host logic of the sharded path: the block-to-host mapping (Appendix J, Eq. 15), the layout of
the two exchanges, and -- as two gloo ranks on the CPU with the oracle standing in for the
kernels -- that gathering per-rank results and merging them reproduces the unsharded result."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import oracle
from paper_2607_20457_b200 import cost_model as cm, workloads as W
from paper_2607_20457_b200.sharding import ShardLayout, TorchCollective


@pytest.mark.parametrize("kind", cm.MAPPINGS)
@pytest.mark.parametrize("B,H", [(8, 4), (16, 8), (16, 2), (4, 4), (6, 1)])
def test_mapping_is_balanced_in_count(kind, B, H):
    pi = cm.block_to_host(B, H, kind)
    assert len(pi) == B and sorted(set(pi)) == list(range(H))
    assert all(pi.count(h) == B // H for h in range(H))


def test_critical_path_eq15():
    # the paper's 128K setting: B = 8 blocks on H = 4 hosts, two blocks each, sink 64, sigma 512
    L, B, H, sink, sigma = 131072, 8, 4, 64, 512
    cost = lambda i: cm.paper_flops(cm.paper_input_len(L, B, sink, sigma, i))
    by_hand = {}
    for kind in cm.MAPPINGS:
        pi = cm.block_to_host(B, H, kind)
        hosts = [sum(cost(i) for i in range(B) if pi[i] == h) for h in range(H)]
        assert cm.host_costs(pi, cost) == hosts
        by_hand[kind] = max(hosts)
        assert cm.critical_path(pi, cost) == max(hosts)
    # contiguous puts the two costliest blocks (6, 7) on one host; zigzag pairs i with 7 - i
    assert by_hand["contiguous"] == cost(6) + cost(7)
    assert by_hand["zigzag"] == max(cost(i) + cost(7 - i) for i in range(4))
    assert by_hand["zigzag"] <= by_hand["round_robin"] <= by_hand["contiguous"]
    assert sum(cm.host_costs(cm.block_to_host(B, H, "zigzag"), cost)) == sum(cost(i) for i in range(B))
    with pytest.raises(ValueError):
        cm.block_to_host(7, 4)


def numpy_pack(lay, h, K, sel):
    """What pulsar_pack_summary_kv writes for rank h, from the unsharded K [L, ...] (numpy)."""
    blocks = lay.local_blocks(h)
    Kl = K[lay.local_token_rows(h)]
    rows = [np.arange(lay.sink)]
    for s, i in enumerate(blocks):
        for c in sel[i]:
            rows.append(s * lay.block_size + c * lay.chunk + np.arange(lay.chunk))
    return Kl[np.concatenate(rows)] if rows else Kl[:0]


@pytest.mark.parametrize("kind", cm.MAPPINGS)
@pytest.mark.parametrize("H", [1, 2, 4])
def test_prefix_exchange_layout_reproduces_the_prefix_list(kind, H):
    w = W.CONFIGS["tiny"]
    lay = ShardLayout.make(w.n_blocks, H, w.block_size, w.chunk, w.k, w.sink, kind)
    ids = W.needle_ids(w)
    ref = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    K = np.arange(w.L, dtype=np.int64) * 10 + 1                 # "rows" that name their position
    V = -K
    gathered = np.concatenate([np.concatenate([numpy_pack(lay, h, K, ref["sel_chunks"]),
                                               numpy_pack(lay, h, V, ref["sel_chunks"])]) for h in range(H)])
    order = lay.prefix_order()
    np.testing.assert_array_equal(gathered[order], K[ref["prefix_idx"]])
    np.testing.assert_array_equal(gathered[order + lay.send_rows], V[ref["prefix_idx"]])
    assert lay.prefix_total == len(ref["prefix_idx"])
    for h in range(H):
        np.testing.assert_array_equal(lay.prefix_len_local(h), ref["prefix_len"][lay.local_blocks(h)])
    assert sorted(np.concatenate([lay.local_token_rows(h) for h in range(H)]).tolist()) == list(range(w.L))


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    coll = TorchCollective()
    w = W.CONFIGS["tiny"]
    lay = ShardLayout.make(w.n_blocks, world, w.block_size, w.chunk, w.k, w.sink, "zigzag")
    Q, K, V = W.qkv(w)
    Qq = W.phase2_query(w)[:5]
    rows = lay.local_token_rows(rank)
    # Phase 2: every rank attends the query to its own KV, the (o_h, l_h) are all-gathered as one
    # float buffer per rank laid out [rows*d | rows], and the merge runs over the gathered set
    o_h, l_h = oracle.phase2_attn(Qq, K[rows], V[rows], lay.n_local, w.block_size)
    n = Qq.shape[0] * w.Hq
    stride = (n * (w.d + 1) + 3) // 4 * 4
    send = torch.zeros(stride, dtype=torch.float64)
    send[: n * w.d] = torch.from_numpy(o_h.reshape(-1))
    send[n * w.d: n * w.d + n] = torch.from_numpy(l_h.reshape(-1))
    g = coll.all_gather(send).numpy()
    assert g.shape == (world, stride)
    pO = g[:, : n * w.d].reshape(world, n, w.d)
    pL = g[:, n * w.d: n * w.d + n]
    O, LSE = oracle.lse_merge(pO, pL)
    O_ref, LSE_ref = oracle.phase2_attn(Qq, K, V, w.n_blocks, w.block_size)
    # Phase 1 exchange: pack, all-gather, reorder -> the rows the prefix list names
    ref = oracle.maxidf_select(W.token_ids(w), w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    Kb = K.view(torch.int16).reshape(w.L, -1).long()          # the bf16 bit patterns, row by row
    mine = numpy_pack(lay, rank, Kb.numpy(), ref["sel_chunks"])
    gk = coll.all_gather(torch.from_numpy(np.concatenate([mine, mine]))).numpy().reshape(-1, Kb.shape[1])
    ok_prefix = bool(np.array_equal(gk[lay.prefix_order()], Kb.numpy()[ref["prefix_idx"]]))
    np.savez(os.path.join(out_dir, f"r{rank}.npz"), dO=np.abs(O.reshape(O_ref.shape) - O_ref).max(),
             dL=np.abs(LSE.reshape(LSE_ref.shape) - LSE_ref).max(), ok_prefix=ok_prefix)
    dist.destroy_process_group()


def test_two_gloo_ranks_exchange_and_merge(tmp_path):
    port = 31500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        z = np.load(tmp_path / f"r{r}.npz")
        assert z["dO"] < 1e-12 and z["dL"] < 1e-12 and bool(z["ok_prefix"])


@pytest.mark.parametrize("H", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("rows", [1, 4, 15, 20, 21, 128, 2048 + 5])
def test_row_slices_of_the_fused_exchange_tile_the_rows(H, rows):
    lay = ShardLayout.make(8 * H, H, 64, 8, 2, 8, "zigzag")
    slices = [lay.row_slice(h, rows) for h in range(H)]
    per = -(-rows // H)
    covered = []
    for begin, n in slices:
        assert 0 <= n <= per and 0 <= begin <= rows
        covered += list(range(begin, begin + n))
    assert covered == list(range(rows))                       # in rank order, no gap, no overlap


def _worker_fused(rank, world, port, out_dir, Hq, Hkv, nq):
    """The fused Phase-2 exchange and the Phase-1 prefix exchange on `world` gloo ranks with several
    blocks per rank, the oracle standing in for the kernels."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    coll = TorchCollective()
    w = W.shrink(W.CONFIGS["tiny"], L=6 * 128, block_size=128, chunk=8, k=3, sink=8, vocab_size=4096, Hq=Hq, Hkv=Hkv,
                 d=16, nq=nq)
    ids = W.needle_ids(w)
    ref = oracle.maxidf_select(ids, w.vocab_size, w.block_size, w.chunk, w.k, w.sink)
    Q, K, V = W.qkv(w)
    Qq = W.phase2_query(w)
    ok_prefix = {}
    res = {}
    for kind in cm.MAPPINGS:
        lay = ShardLayout.make(w.n_blocks, world, w.block_size, w.chunk, w.k, w.sink, kind)
        assert lay.n_local == 6 // world > 1
        rows_local = lay.local_token_rows(rank)
        # Phase-1 exchange: pack, all-gather, reorder -> the rows the prefix list names
        Kb = K.view(torch.int16).reshape(w.L, -1).long().numpy()
        mine = numpy_pack(lay, rank, Kb, ref["sel_chunks"])
        gk = coll.all_gather(torch.from_numpy(np.concatenate([mine, -mine]))).numpy().reshape(-1, Kb.shape[1])
        ok_prefix[kind] = bool(np.array_equal(gk[lay.prefix_order()], Kb[ref["prefix_idx"]]) and
                               np.array_equal(gk[lay.prefix_order() + lay.send_rows], -Kb[ref["prefix_idx"]]))
        # Phase 2, exchange fused into the merge: every rank's partial is visible to all (here: gathered),
        # rank r merges only its slice of the rows, the merged slices are gathered
        o_h, l_h = oracle.phase2_attn(Qq, K[rows_local], V[rows_local], lay.n_local, w.block_size)
        n = nq * Hq
        pO = coll.all_gather(torch.from_numpy(o_h.reshape(n, w.d))).numpy()
        pL = coll.all_gather(torch.from_numpy(l_h.reshape(n))).numpy()
        begin, cnt = lay.row_slice(rank, n)
        per = -(-n // world)
        o_pad, l_pad = np.zeros((per, w.d)), np.zeros(per)
        if cnt:
            o_pad[:cnt], l_pad[:cnt] = oracle.lse_merge(pO[:, begin: begin + cnt], pL[:, begin: begin + cnt])
        O = coll.all_gather(torch.from_numpy(o_pad)).numpy().reshape(-1, w.d)[:n]
        LSE = coll.all_gather(torch.from_numpy(l_pad)).numpy().reshape(-1)[:n]
        O_ref, LSE_ref = oracle.phase2_attn(Qq, K, V, w.n_blocks, w.block_size)
        res[kind] = (float(np.abs(O - O_ref.reshape(n, w.d)).max()), float(np.abs(LSE - LSE_ref.reshape(n)).max()), cnt)
    np.savez(os.path.join(out_dir, f"r{rank}.npz"), ok=np.array([ok_prefix[k] for k in cm.MAPPINGS]),
             dO=np.array([res[k][0] for k in cm.MAPPINGS]), dL=np.array([res[k][1] for k in cm.MAPPINGS]),
             cnt=np.array([res[k][2] for k in cm.MAPPINGS]))
    dist.destroy_process_group()


@pytest.mark.parametrize("world,Hq,Hkv,nq", [(2, 3, 1, 5), (3, 4, 2, 5)])
def test_gloo_ranks_fused_exchange_rows_that_do_not_divide(tmp_path, world, Hq, Hkv, nq):
    assert (nq * Hq) % world != 0
    port = 33500 + os.getpid() % 2000 + world
    mp.spawn(_worker_fused, args=(world, port, str(tmp_path), Hq, Hkv, nq), nprocs=world, join=True)
    counts = np.zeros(len(cm.MAPPINGS), int)
    for r in range(world):
        z = np.load(tmp_path / f"r{r}.npz")
        assert z["ok"].all() and (z["dO"] < 1e-12).all() and (z["dL"] < 1e-12).all()
        counts += z["cnt"]
    assert (counts == nq * Hq).all()
