"""The analytical cost model against the cells the paper prints (Table 6, Eq. 14)."""
import os

from paper_2607_20457_b200 import cost_model as cm
from paper_2607_20457_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table6_phase1_cost.txt")


def _rows():
    cells, ratios = [], []
    for line in open(GOLDEN):
        f = line.split()
        if not f or f[0].startswith("#") or f[0] == "method":
            continue
        (ratios if f[0] == "ratio" else cells).append(f)
    return cells, ratios


def test_table6_lengths_follow_eq14():
    cells, _ = _rows()
    for method, ctx, n, *_ in cells:
        L, n = int(ctx), int(n)
        if method == "dense":
            assert n == L
        elif method == "star":
            assert n == 2 * (L // 4)
        else:
            assert n == cm.paper_input_len(L, 4, 64, 512, 3)
    assert cm.paper_input_len(16384, 4, 64, 512, 0) == 4096
    # "fixed 1,600-token prefix": sink + 3 summaries of 512
    assert cm.paper_input_len(65536, 4, 64, 512, 3) - 65536 // 4 == 1600


def test_table6_flops_and_memory_cells():
    cells, _ = _rows()
    assert len(cells) == 9
    for _m, _ctx, n, flops_g, mem, unit in cells:
        n = int(n)
        # one cell (43,981) is printed one above the rounded value: allow the last digit
        assert abs(cm.paper_flops(n) / 1e9 - int(flops_g)) <= 0.6
        b = cm.paper_activation_bytes(n)
        if unit == "GB":
            assert abs(b / 2**30 - float(mem)) < 0.005
        else:
            assert int(mem) in (round(b / 2**20), round(b / 1e6))


def test_table6_reduction_rows():
    cells, ratios = _rows()
    n = {(m, int(c)): int(nn) for m, c, nn, *_ in cells}
    for _r, ctx, p_vs_s, p_vs_d, s_vs_d in ratios:
        c = int(ctx)
        fp, fs, fd = (cm.paper_flops(n[(m, c)]) for m in ("pulsar", "star", "dense"))
        assert round(fs / fp, 1) == float(p_vs_s)
        assert round(fd / fp, 1) == float(p_vs_d)
        assert round(fd / fs, 1) == float(s_vs_d)


def test_algorithmic_pair_counts_by_enumeration():
    # small shape: count (row, key) pairs one at a time
    nb, plen = 8, [0, 3, 5]
    brute = 0
    for i, p in enumerate(plen):
        for r in range(nb):
            brute += p + (r + 1)
    assert cm.phase1_pairs(nb, plen) == brute
    assert cm.phase1_flops(nb, plen, Hq=4, d=16) == 4 * 16 * 4 * brute


def test_config_sizes():
    w = W.CONFIGS["128k"]
    plen = cm.prefix_lens(w.n_blocks, w.sink, w.sigma)
    assert plen[-1] == 7744 and w.prefix_total == 7744
    # 17.17 TFLOP per layer at the 128K configuration
    assert abs(cm.phase1_flops(w.block_size, plen, w.Hq, w.d) / 1e12 - 17.17) < 0.01
    w4 = W.CONFIGS["64k"]
    pl4 = cm.prefix_lens(w4.n_blocks, w4.sink, w4.sigma)
    star = [0] + [w4.block_size] * (w4.n_blocks - 1)
    ratio = cm.phase1_pairs(w4.block_size, star) / cm.phase1_pairs(w4.block_size, pl4)
    assert abs(ratio - 1.895) < 0.001


def test_phase2_query_positions():
    # the paper's 128K setting: B = 8 blocks of 16K, sink 64, sigma 512 -> longest input 16384 + 64 + 7*512
    assert cm.phase2_query_position_start(131072, 8, 64, 512, "sparse") == 131072
    assert cm.phase2_query_position_start(131072, 8, 64, 512, "contiguous") == 16384 + 64 + 3584
    assert cm.phase2_query_position_start(4096, 1, 64, 512, "contiguous") == 4096      # one block: no prefix at all
