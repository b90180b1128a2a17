"""Seeded random configurations (row size, R, L, alpha, P, c, k_repair, expansion cap, element type, mode, delete
variant, snapshot mode, batch sizes, id reuse, clustered or uniform or heavily duplicated data): the CUDA library must
leave the oracle's graph after every batch and return its search results, bit for bit.  A second family aims at the
paths that only hubs and fp32 rows reach: a few targets that collect thousands of requests (segments far longer
than shared memory, with small and large P), fixed-degree graphs under inner product whose large-norm rows gather
thousands of in-neighbours and are then deleted, and fp32 rows with small integer coordinates, on which fp32
arithmetic is exact in any order so that the fp32 kernels can be held to the oracle bit for bit as well."""
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


def run_hub_config(seed):
    """Returns False when the configuration had to be skipped: the first batch's medoid is the row closest to a mean
    that is not an integer vector, the one place where fp32 and fp64 may order two rows differently."""
    from paper_2608_21163_b200 import binding as gb
    rng = np.random.default_rng(seed)
    kind = str(rng.choice(["f32int", "f32int_wide", "hub", "fixed_ip"]))
    metric = go.L2
    dtype = int(rng.choice([go.U8, go.I8]))
    dim = int(rng.choice([3, 8, 16, 17, 32, 48, 64, 96, 100, 128, 160, 256]))
    R = int(rng.choice([4, 8, 13, 16, 24, 32, 48, 64]))
    L = max(int(rng.choice([R, R + 3, 2 * R, 40, 64, 100, 128])), 4)
    alpha = float(rng.choice([1.0, 1.25, 1.5, 2.0]))           # exact in binary: the fp32 prune test is then exact too
    P = int(rng.choice([0, 3, 16, 64, 100]))
    c = int(rng.choice([0, 1, 2, 3, 4, 5]))
    kr = int(rng.choice([0, 5, 20, 56, 57, 100, 128]))
    mode = 0
    n, nb = int(rng.choice([1500, 3000, 6000])), int(rng.choice([250, 500, 1000]))
    if kind == "f32int":
        dtype, dim = go.F32, int(rng.choice([4, 16, 24, 64, 96, 100, 128]))
    if kind == "f32int_wide":
        dtype, dim = go.F32, int(rng.choice([130, 192, 300, 512, 768, 960]))
        n, nb = int(rng.choice([600, 1200])), int(rng.choice([100, 200]))
    if kind == "hub":
        alpha, R = float(rng.choice([1000.0, 2.0])), int(rng.choice([4, 8, 16]))
        L, nb = max(L, R), int(rng.choice([1000, 2000]))
        n = 3 * nb
    if kind == "fixed_ip":
        mode, metric, dtype, L = 1, go.IP, go.U8, max(L, R)
    kr = min(kr, L)
    if dtype == go.F32:
        base = rng.integers(0, 8, (n, dim)).astype(np.float32)
    elif dtype == go.U8:
        cen = rng.integers(0, 256, (8, dim))
        base = np.clip(cen[rng.integers(0, 8, n)] + rng.normal(0, 12, (n, dim)), 0, 255).astype(np.uint8)
        if kind == "hub":
            base = (base // 8 + 100).astype(np.uint8)
            base[:4] = rng.integers(0, 256, (4, dim)).astype(np.uint8)
        if kind == "fixed_ip":
            base = (base // 2).astype(np.uint8)
            base[:6] = 255                                    # large-norm rows attract everyone under inner product
            base[:6, 0] = np.arange(6)
    else:
        base = rng.integers(-128, 128, (n, dim)).astype(np.int8)
    kw = dict(P=P, c=c, k_repair=kr, mode=mode)
    what = f"seed {seed} {kind}: dim {dim} dtype {dtype} metric {metric} R {R} L {L} alpha {alpha} {kw} n {n} batch {nb}"
    o = go.Oracle(dim, dtype, metric, R, L, alpha, n, **kw)
    g = gb.GrandIndex(dim, dtype, metric, R, L, alpha, capacity=n, max_batch=nb, max_delete_edges=n * R, **kw)
    alive = np.zeros(n, bool)
    t = torch.from_numpy
    hubs = kind in ("hub", "fixed_ip")
    order = np.concatenate([np.arange(8), rng.permutation(np.arange(8, n))]) if hubs else np.arange(n)
    for step in range(10):
        free = order[~alive[order]]
        if len(free) and (rng.random() < 0.6 or alive.sum() < nb):
            # (hub families: a first batch of 8 rows, so that the whole second batch links to those 8)
            ids = free[: min(8 if hubs and step == 0 else nb, len(free))].astype(np.uint32)
            o.insert_batch(ids, base[ids]); g.insert_batch(t(ids), t(base[ids]))
            alive[ids] = True
        else:
            live = np.flatnonzero(alive)
            ids = rng.permutation(live)[: int(min(len(live), rng.choice([1, nb // 4, nb])))].astype(np.uint32)
            if hubs and rng.random() < 0.7:
                ids = np.unique(np.concatenate([ids, live[live < 6]])).astype(np.uint32)[:nb]   # the hubs go
            o.delete_batch(ids); g.delete_batch(t(ids))
            alive[ids] = False
        if step == 0 and dtype == go.F32 and o.entry != g.entry:
            return False
        assert_same_graph(o, g, f"{what}, step {step}")
        if step % 3 == 2 and alive.any():
            q = base[rng.integers(0, n, 40)]
            Ls = int(rng.choice([10, L, 2 * L]))
            k = min(10, Ls)
            oi, od = o.search(q, k, Ls)
            gi, gd = g.search(t(q), k, Ls)
            gi = gi.cpu().numpy()
            have = oi != INV
            assert (oi == gi).all() and (od[have] == gd.cpu().numpy().astype(np.float64)[have]).all(), f"{what}, search at step {step}"
    return True


def test_random_configurations_hubs_and_exact_fp32_bit_exact():
    ran = sum(run_hub_config(seed) for seed in range(7000, 7120))
    assert ran >= 110
