"""Seeded random configurations (row size, R, L, alpha, P, c, k_repair, expansion cap, element type, mode, delete
variant, snapshot mode, batch sizes, id reuse, clustered or uniform or heavily duplicated data): the CUDA library must
leave the oracle's graph after every batch and return its search results, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import grand_oracle as go
from tests.helpers import INV, assert_same_graph

pytestmark = pytest.mark.gpu


def run_config(seed, wide=False):
    from paper_2608_21163_b200 import binding as gb
    rng = np.random.default_rng(seed)
    dtype = int(rng.choice([go.U8, go.U8, go.I8]))
    dim = int(rng.choice([3, 8, 16, 17, 31, 32, 48, 64, 96, 100, 127, 128, 129, 160, 200, 256, 300]))
    if wide:                                           # rows of 257..4000 bytes: the whole-warp distance layouts
        dim = int(rng.choice([257, 384, 512, 513, 700, 1024, 1500, 2048, 3000, 4000]))
    R = int(rng.choice([4, 7, 8, 13, 16, 24, 32, 33, 48, 64, 65, 96]))
    L = max(int(rng.choice([R, R + 3, 2 * R, 40, 64, 100, 128])), 4)
    alpha = float(rng.choice([1.0, 1.1, 1.2, 1.5, 2.0]))
    P = int(rng.choice([0, 0, 3, 16, 64, 100]))
    c = int(rng.choice([0, 1, 2, 3, 5]))
    kr = int(rng.choice([0, 0, 5, 20, 56, 57, 100]))
    vmax = int(rng.choice([0, 0, L, 3 * L]))
    visited = int(rng.random() < 0.25)
    mode = int(rng.random() < 0.3)
    snap = int(rng.random() < 0.3)
    if mode or snap:
        visited = 0
    if mode:
        L = max(L, R)
    kr = min(kr, L)
    n = int(rng.choice([600, 1500, 3000]))
    nb = int(rng.choice([100, 250, 500]))
    if wide:
        n, nb = int(rng.choice([400, 800])), int(rng.choice([50, 100, 200]))
    if dtype == go.U8:
        if rng.random() < 0.5:
            cen = rng.integers(0, 256, (8, dim))
            base = np.clip(cen[rng.integers(0, 8, n)] + rng.normal(0, 12, (n, dim)), 0, 255).astype(np.uint8)
        else:
            base = rng.integers(0, 256, (n, dim)).astype(np.uint8)
    else:
        base = rng.integers(-128, 128, (n, dim)).astype(np.int8)
    if rng.random() < 0.3:
        base[: n // 10] = base[0]                      # many identical vectors: ties everywhere
    kw = dict(P=P, c=c, k_repair=kr, vmax=vmax, mode=mode)
    what = f"seed {seed}: dim {dim} dtype {dtype} R {R} L {L} alpha {alpha} {kw} visited {visited} snapshot {snap} n {n} batch {nb}"
    o = go.Oracle(dim, dtype, go.L2, R, L, alpha, n, approx_delete=visited, **kw)
    g = gb.GrandIndex(dim, dtype, gb.L2, R, L, alpha, capacity=n, max_batch=nb, visited_set_delete=visited,
                      snapshot_search=snap, **kw)
    alive = np.zeros(n, bool)
    t = torch.from_numpy
    for step in range(12):
        free = np.flatnonzero(~alive)
        if len(free) and (rng.random() < 0.6 or alive.sum() < nb):
            ids = rng.permutation(free)[: min(nb, len(free))].astype(np.uint32)
            o.insert_batch(ids, base[ids]); g.insert_batch(t(ids), t(base[ids]))
            alive[ids] = True
        else:
            live = np.flatnonzero(alive)
            ids = rng.permutation(live)[: int(min(len(live), rng.choice([1, nb // 4, nb])))].astype(np.uint32)
            o.delete_batch(ids); g.delete_batch(t(ids))
            alive[ids] = False
        assert_same_graph(o, g, f"{what}, step {step}")
        if step % 4 == 3 and alive.any():
            q = base[rng.integers(0, n, 50)]
            Ls = int(rng.choice([10, L, 2 * L]))
            k = min(10, Ls)
            oi, od = o.search(q, k, Ls)
            gi, gd = g.search(t(q), k, Ls)
            gi = gi.cpu().numpy()
            have = oi != INV
            assert (oi == gi).all() and (od[have] == gd.cpu().numpy()[have]).all(), f"{what}, search at step {step}"


@pytest.mark.parametrize("block", range(4))
def test_random_configurations_bit_exact(block):
    for seed in range(5000 + 25 * block, 5000 + 25 * (block + 1)):
        run_config(seed)


def test_random_configurations_wide_rows_bit_exact():
    for seed in range(6000, 6030):
        run_config(seed, wide=True)
