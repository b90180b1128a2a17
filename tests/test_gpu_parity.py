"""GPU parity: the CUDA library against the CPU oracle on the same seeded inputs, through the
C-ABI.  Integer vectors must match bit for bit (adjacency rows, degrees, live bitmap, medoid,
search ids and distances); fp32 vectors are held to 1e-5 relative distance error and a recall@10
within 0.005 of the oracle's."""
import numpy as np
import pytest

from oracle import grand_oracle as go
from paper_2608_21163_b200 import synth
from tests.helpers import (INV, assert_same_graph, brute_force_topk, gpu_graph, make_pair, recall_at_k, run_stream)

pytestmark = pytest.mark.gpu


def torch_():
    import torch
    return torch


def gpu_search(g, q, k, L):
    torch = torch_()
    ids, d = g.search(torch.from_numpy(q), k, L)
    torch.cuda.synchronize()
    return ids.cpu().numpy(), d.cpu().numpy()


def import_from_oracle(o, g, base_full):
    torch = torch_()
    adj, deg, live, entry = o.export_graph()
    R = adj.shape[1]
    adj = adj.copy()
    adj[np.arange(R)[None, :] >= deg[:, None]] = INV
    g.import_graph(torch.from_numpy(adj), torch.from_numpy(deg), torch.from_numpy(live), entry, torch.from_numpy(base_full))


def small_cfg(name, scale, **over):
    c = synth.scaled(synth.CONFIGS[name], scale)
    c.update(over)
    return c


# ------------------------------------------------------------------ search on an imported graph
@pytest.mark.parametrize("dim,dtype", [(32, go.U8), (33, go.U8), (128, go.U8), (20, go.I8), (200, go.U8)])
def test_search_bit_exact_on_oracle_graph(dim, dtype):
    n, R, L = 3000, 24, 48
    rng = np.random.default_rng(dim)
    if dtype == go.U8:
        base = synth.uniform_u8(1, "base", 0, n, dim)
        q = synth.uniform_u8(1, "query", 0, 300, dim)
    else:
        base = rng.integers(-128, 128, (n, dim)).astype(np.int8)
        q = rng.integers(-128, 128, (300, dim)).astype(np.int8)
        base[0] = -128; base[1] = 127           # extreme differences: |a-b| = 255 per coordinate
        q[0] = 127; q[1] = -128
    cfg = dict(dim=dim, dtype=dtype, metric=go.L2, R=R, L=L, alpha=1.2, mode=go.VAMANA, max_build_batch=500, ins=1, dele=1)
    o, g = make_pair(cfg, n)
    for lo in range(0, n, 500):
        o.insert_batch(np.arange(lo, lo + 500, dtype=np.uint32), base[lo:lo + 500])
    import_from_oracle(o, g, base)
    assert g.live_count == n
    for k, Ls in [(10, 48), (1, 1), (10, 10), (48, 48), (5, 200), (10, 512)]:
        oi, od = o.search(q, k, Ls)
        gi, gd = gpu_search(g, q, k, Ls)
        assert (oi == gi).all(), (k, Ls, np.flatnonzero((oi != gi).any(1))[:5])
        assert (od == gd.astype(np.float64)).all()


def test_updates_continue_bit_exact_on_an_imported_graph():
    """An imported graph carries no cached distances and no pruned-run lengths: every row entry is of unknown
    standing when its node is next rebuilt.  Inserts, deletes and re-inserts then have to match the oracle, which
    kept the same graph all along."""
    torch = torch_()
    n, dim, R, L = 6000, 32, 16, 32
    base = synth.uniform_u8(7, "base", 0, n, dim)
    cfg = dict(dim=dim, dtype=go.U8, metric=go.L2, R=R, L=L, alpha=1.2, mode=go.VAMANA, max_build_batch=500, ins=500, dele=500)
    o, g = make_pair(cfg, n)
    for lo in range(0, 4000, 500):
        o.insert_batch(np.arange(lo, lo + 500, dtype=np.uint32), base[lo:lo + 500])
    import_from_oracle(o, g, base)
    assert_same_graph(o, g, "import")
    alive = np.zeros(n, bool); alive[:4000] = True
    for r in range(4):
        ids = np.arange(4000 + 500 * r, 4500 + 500 * r, dtype=np.uint32)
        o.insert_batch(ids, base[ids]); g.insert_batch(torch.from_numpy(ids), torch.from_numpy(base[ids]))
        alive[ids] = True
        assert_same_graph(o, g, f"insert {r} after import")
        dele = synth.choose_ids(7, f"del/{r}", np.flatnonzero(alive).astype(np.uint32), 500)
        o.delete_batch(dele); g.delete_batch(torch.from_numpy(dele))
        alive[dele] = False
        assert_same_graph(o, g, f"delete {r} after import")


def test_search_fp32_tolerance_and_ip():
    n, dim, R, L = 4000, 96, 24, 64
    base = synth.gaussian_unit_f32(2, "base", 0, n, dim)
    q = synth.gaussian_unit_f32(2, "query", 0, 200, dim)
    for metric, mode in [(go.L2, go.VAMANA), (go.IP, go.FIXED_DEGREE)]:
        cfg = dict(dim=dim, dtype=go.F32, metric=metric, R=R, L=L, alpha=1.2, mode=mode, max_build_batch=500, ins=1, dele=1)
        o, g = make_pair(cfg, n)
        for lo in range(0, n, 500):
            o.insert_batch(np.arange(lo, lo + 500, dtype=np.uint32), base[lo:lo + 500])
        import_from_oracle(o, g, base)
        oi, od = o.search(q, 10, L)
        gi, gd = gpu_search(g, q, 10, L)
        # returned distances against a float64 recomputation
        for i in range(len(q)):
            b = base[gi[i]].astype(np.float64)
            exact = ((b - q[i].astype(np.float64)) ** 2).sum(1) if metric == go.L2 else -(b @ q[i].astype(np.float64))
            scale = np.abs(exact) if metric == go.L2 else np.linalg.norm(b, axis=1) * np.linalg.norm(q[i])
            assert (np.abs(gd[i] - exact) <= 1e-5 * scale).all()
            assert (np.diff(gd[i]) >= 0).all()
        # near-ties may reorder; the result sets must agree almost everywhere
        same = np.mean([len(set(a.tolist()) & set(b.tolist())) / 10 for a, b in zip(oi, gi)])
        assert same > 0.99


def test_search_padding_and_empty_index():
    torch = torch_()
    cfg = dict(dim=8, dtype=go.U8, metric=go.L2, R=4, L=8, alpha=1.2, mode=go.VAMANA, max_build_batch=8, ins=1, dele=1)
    o, g = make_pair(cfg, 16)
    q = np.zeros((3, 8), np.uint8)
    gi, gd = gpu_search(g, q, 4, 8)
    assert (gi == INV).all() and (gd == np.iinfo(np.int32).max).all()
    v = np.arange(24, dtype=np.uint8).reshape(3, 8)
    ids = np.array([5, 2, 9], np.uint32)
    o.insert_batch(ids, v)
    g.insert_batch(torch.from_numpy(ids), torch.from_numpy(v))
    assert_same_graph(o, g, "3-point bootstrap")
    oi, od = o.search(q, 4, 8)
    gi, gd = gpu_search(g, q, 4, 8)
    assert (oi == gi).all() and gi[0, 3] == INV and gd[0, 3] == np.iinfo(np.int32).max
    assert (od[:, :3] == gd[:, :3]).all()


# ------------------------------------------------------------------ whole streams, bit exact
def check_search(o, g, wl, cfg, k=10):
    q = wl.queries()
    oi, od = o.search(q, k, cfg["L"])
    gi, gd = gpu_search(g, q, k, cfg["L"])
    assert (oi == gi).all() and (od == gd.astype(np.float64)).all()


def test_tiny_config_stream_bit_exact():
    """The tiny config at full size: 8 x 1,000 build, +2,000, -1,000, 1,000 queries."""
    cfg = synth.CONFIGS["tiny_u8_d32"]
    o, g, wl, st = run_stream(cfg, seed=0)
    check_search(o, g, wl, cfg)
    assert o.stats()["dead_edges_seen"] == 0
    # exact reverse graph
    ooff, osrc = o.reverse_graph()
    goff, gsrc = g.reverse_graph()
    assert (ooff == goff.cpu().numpy().astype(np.uint64)).all() and (osrc == gsrc.cpu().numpy()).all()
    # recall sanity
    base = wl.vectors(0, cfg["n"])
    live = np.flatnonzero(st.live).astype(np.uint32)
    q = wl.queries()[:200]
    gi, _ = gpu_search(g, q, 10, cfg["L"])
    assert recall_at_k(gi, brute_force_topk(base, live, q, 10, go.L2)) > 0.9


def test_sift_shaped_shrink_bit_exact():
    """SIFT-shaped bytes (d=128, R=64, L=128) shrunk to 20k points: several insert/delete rounds, the graph compared
    after every batch."""
    cfg = small_cfg("sift_u8_d128", 0.02, rounds=3)
    o, g, wl, st = run_stream(cfg, seed=0)
    check_search(o, g, wl, cfg)
    q = wl.queries()
    for L in (10, 32, 200):
        oi, od = o.search(q, 10, L)
        gi, gd = gpu_search(g, q, 10, L)
        assert (oi == gi).all() and (od == gd.astype(np.float64)).all()


def test_sift_shaped_100k_points_bit_exact():
    """The same stream at 100,000 points (90,000 built in batches of up to 1,000, then three rounds of insert 1,000 +
    delete 1,000): the graph after the build and after every round, then 1,000 searches, all bit for bit."""
    cfg = small_cfg("sift_u8_d128", 0.1, rounds=3)
    checked = []

    def on_round(r, o, g, wl, st):
        assert_same_graph(o, g, f"round {r}")
        checked.append(r)

    o, g, wl, st = run_stream(cfg, seed=0, check_each=False, on_round=on_round)
    assert checked == [0, 1, 2] and o.live_count == 90_000
    check_search(o, g, wl, cfg)
    assert o.stats()["dead_edges_seen"] == 0


def test_ids_above_the_tag_range_of_the_visited_cache_bit_exact():
    """A capacity above 2^(hash_bits + 14) ids no longer fits the 16-bit tags of the visited cache: the search falls
    back to a direct-mapped table of full ids.  A few thousand live ids spread over a capacity just above 2^22
    (hash_bits = 8) take that path through inserts, a delete and searches."""
    torch = torch_()
    from paper_2608_21163_b200 import binding as gb
    cap, dim, R, L, n = (1 << 22) + 4096, 16, 8, 24, 4000
    ids_all = np.unique(np.linspace(0, cap - 1, n).astype(np.uint32))
    assert ids_all[-1] >= (1 << 22) and len(ids_all) == n
    vecs = synth.uniform_u8(41, "base", 0, n, dim)
    o = go.Oracle(dim, go.U8, go.L2, R, L, 1.2, cap)
    g = gb.GrandIndex(dim, gb.U8, gb.L2, R, L, 1.2, capacity=cap, max_batch=500, hash_bits=8)
    for lo in range(0, n, 500):
        o.insert_batch(ids_all[lo:lo + 500], vecs[lo:lo + 500])
        g.insert_batch(torch.from_numpy(ids_all[lo:lo + 500]), torch.from_numpy(vecs[lo:lo + 500]))
    assert_same_graph(o, g, "sparse ids, build")
    dele = synth.choose_ids(41, "del", ids_all, 400)
    o.delete_batch(dele); g.delete_batch(torch.from_numpy(dele))
    assert_same_graph(o, g, "sparse ids, delete")
    q = synth.uniform_u8(41, "query", 0, 300, dim)
    for k, Ls in [(10, 24), (5, 100)]:
        oi, od = o.search(q, k, Ls)
        gi, gd = gpu_search(g, q, k, Ls)
        assert (oi == gi).all() and (od == gd.astype(np.float64)).all()


def test_ragged_dim_int8_and_small_params_bit_exact():
    """Odd dimension (tail chunk), int8 data, R/L not multiples of 32, tiny P and c=3."""
    rng = np.random.default_rng(9)
    torch = torch_()
    n, dim = 2500, 45
    base = rng.integers(-128, 128, (n, dim)).astype(np.int8)
    cfg = dict(dim=dim, dtype=go.I8, metric=go.L2, R=13, L=21, alpha=1.1, mode=go.VAMANA, max_build_batch=400, ins=1, dele=300)
    o, g = make_pair(cfg, n, P=3, c=3, k_repair=7, vmax=30)
    for lo in range(0, n, 357):
        ids = np.arange(lo, min(n, lo + 357), dtype=np.uint32)
        o.insert_batch(ids, base[ids]); g.insert_batch(torch.from_numpy(ids), torch.from_numpy(base[ids]))
        assert_same_graph(o, g, f"insert at {lo}")
    dele = synth.choose_ids(3, "del", np.arange(n, dtype=np.uint32), 300)
    o.delete_batch(dele); g.delete_batch(torch.from_numpy(dele))
    assert_same_graph(o, g, "delete")
    # id reuse
    o.insert_batch(dele[:100], base[dele[:100]]); g.insert_batch(torch.from_numpy(dele[:100]), torch.from_numpy(base[dele[:100]]))
    assert_same_graph(o, g, "reinsert")


@pytest.mark.parametrize("dim,dtype", [(16, go.U8), (100, go.U8), (200, go.U8), (250, go.U8), (33, go.I8), (256, go.I8)])
def test_delete_repair_bit_exact_across_row_sizes(dim, dtype):
    """The delete repair's neighbour-by-candidate distance block on integer rows of every padding class (row
    bytes a multiple of 32 or not, one to eight 32-byte steps), extreme values included."""
    torch = torch_()
    n = 3000
    rng = np.random.default_rng(100 + dim)
    if dtype == go.U8:
        base = synth.uniform_u8(11, f"base{dim}", 0, n, dim)
        base[:5] = 255; base[5:10] = 0
    else:
        base = rng.integers(-128, 128, (n, dim)).astype(np.int8)
        base[:5] = -128; base[5:10] = 127
    base[:10, 0] = np.arange(10).astype(base.dtype)         # keep the extreme rows distinct
    cfg = dict(dim=dim, dtype=dtype, metric=go.L2, R=20, L=40, alpha=1.2, mode=go.VAMANA, max_build_batch=600, ins=1, dele=600)
    o, g = make_pair(cfg, n)
    for lo in range(0, n, 600):
        ids = np.arange(lo, lo + 600, dtype=np.uint32)
        o.insert_batch(ids, base[ids]); g.insert_batch(torch.from_numpy(ids), torch.from_numpy(base[ids]))
    assert_same_graph(o, g, "build")
    alive = np.ones(n, bool)
    for r in range(3):
        dele = synth.choose_ids(dim, f"del/{r}", np.flatnonzero(alive).astype(np.uint32), 600)
        if r == 0:
            dele[:10] = np.arange(10)                        # the extreme rows go first (ids 0..9 are still live)
            dele = np.unique(dele).astype(np.uint32)
        o.delete_batch(dele); g.delete_batch(torch.from_numpy(dele))
        alive[dele] = False
        assert_same_graph(o, g, f"delete {r}")


@pytest.mark.parametrize("dim", [16, 96, 100, 300, 960])
def test_fp32_rows_with_small_integer_coordinates_bit_exact(dim):
    """fp32 vectors whose coordinates are small integers: every partial sum of a squared distance is exact in
    fp32, whatever the order, and alpha = 1.25 makes the prune test exact as well - so the fp32 kernels (register
    and warp tiles of the delete repair, the prunes, the rebuild, the search; one row size per layout class) must
    reproduce the fp64 oracle bit for bit, not only within the tolerance."""
    torch = torch_()
    n = 2400
    base = (synth.uniform_u8(21, f"intf32/{dim}", 0, n, dim) % 8).astype(np.float32)
    cfg = dict(dim=dim, dtype=go.F32, metric=go.L2, R=16, L=32, alpha=1.25, mode=go.VAMANA, max_build_batch=600, ins=1, dele=500)
    o, g = make_pair(cfg, n)
    for lo in range(0, n, 600):
        ids = np.arange(lo, lo + 600, dtype=np.uint32)
        o.insert_batch(ids, base[ids]); g.insert_batch(torch.from_numpy(ids), torch.from_numpy(base[ids]))
        assert_same_graph(o, g, f"build {lo}")
    alive = np.ones(n, bool)
    for r in range(2):
        dele = synth.choose_ids(dim, f"intdel/{r}", np.flatnonzero(alive).astype(np.uint32), 500)
        o.delete_batch(dele); g.delete_batch(torch.from_numpy(dele))
        alive[dele] = False
        assert_same_graph(o, g, f"delete {r}")
    q = (synth.uniform_u8(22, f"intq/{dim}", 0, 100, dim) % 8).astype(np.float32)
    oi, od = o.search(q, 10, 32)
    gi, gd = gpu_search(g, q, 10, 32)
    assert (oi == gi).all() and (od == gd.astype(np.float64)).all()


def test_hub_segment_longer_than_shared_memory_cap():
    """Every point of a large batch links to the same few hubs: request segments far above the
    in-kernel shared-memory cap take the in-place global-memory sort."""
    torch = torch_()
    dim = 4
    hubs = np.array([[0, 0, 0, 0], [255, 255, 255, 255], [0, 255, 0, 255]], np.uint8)
    pts = synth.uniform_u8(4, "hubpts", 0, 3000, dim) // 8 + 100          # clustered away from the hubs
    cfg = dict(dim=dim, dtype=go.U8, metric=go.L2, R=8, L=16, alpha=1000.0, mode=go.VAMANA, max_build_batch=3000, ins=1, dele=1)
    o, g = make_pair(cfg, 4000)
    ids = np.arange(3, dtype=np.uint32)
    o.insert_batch(ids, hubs); g.insert_batch(torch.from_numpy(ids), torch.from_numpy(hubs))
    ids = np.arange(3, 3003, dtype=np.uint32)
    o.insert_batch(ids, pts); g.insert_batch(torch.from_numpy(ids), torch.from_numpy(pts))
    assert_same_graph(o, g, "hub insert")


def test_delete_everything_and_reinsert():
    torch = torch_()
    cfg = small_cfg("tiny_u8_d32", 0.05)
    n = cfg["n"]
    base = synth.uniform_u8(0, "base", 0, n, 32)
    o, g = make_pair(dict(cfg, max_build_batch=n, ins=n, dele=n), n)
    ids = np.arange(n, dtype=np.uint32)
    for lo in range(0, n, 100):
        o.insert_batch(ids[lo:lo + 100], base[lo:lo + 100]); g.insert_batch(torch.from_numpy(ids[lo:lo + 100]), torch.from_numpy(base[lo:lo + 100]))
    o.delete_batch(ids); g.delete_batch(torch.from_numpy(ids))
    assert_same_graph(o, g, "all deleted")
    assert g.entry == INV and g.live_count == 0
    o.insert_batch(ids[::-1].copy(), base[::-1].copy()); g.insert_batch(torch.from_numpy(ids[::-1].copy()), torch.from_numpy(base[::-1].copy()))
    assert_same_graph(o, g, "rebuilt in one bootstrap batch")


def test_medoid_deletion_paths():
    torch = torch_()
    cfg = small_cfg("tiny_u8_d32", 0.1)
    o, g, wl, st = run_stream(dict(cfg, rounds=0), seed=1)
    m = np.array([o.entry], np.uint32)
    o.delete_batch(m); g.delete_batch(torch.from_numpy(m))
    assert_same_graph(o, g, "medoid deleted")
    assert g.entry != m[0]


# ------------------------------------------------------------------ fixed-degree mode
def test_fixed_degree_mode_bit_exact_on_bytes():
    """Alg. 7 / Alg. 8 logic is integer-only; with uint8 vectors and IP the whole state must match."""
    cfg = dict(gen="uniform_u8", dim=24, dtype=go.U8, metric=go.IP, mode=go.FIXED_DEGREE, R=16, L=40, alpha=1.2,
               n=6000, build=4000, first_batch=500, max_build_batch=1000, rounds=3, ins=500, dele=400, nq=200, reuse_ids=False)
    o, g, wl, st = run_stream(cfg, seed=5)
    check_search(o, g, wl, cfg)
    cfg2 = dict(cfg, metric=go.L2, rounds=2)
    o, g, wl, st = run_stream(cfg2, seed=6)
    check_search(o, g, wl, cfg2)


def test_fixed_degree_delete_of_hubs_bit_exact():
    """Alg. 8 on a graph whose deleted nodes have very long in-neighbour rows: the round-robin
    offset (rank of u among the in-neighbours) is then taken from a sorted row, in shared memory
    (node 1: a few thousand in-neighbours) or in place in global memory (node 0: more than 49,152)."""
    torch = torch_()
    n, R, dim = 60000, 6, 8
    rng = np.random.default_rng(11)
    vecs = synth.uniform_u8(9, "hubgraph", 0, n, dim)
    adj = np.full((n, R), INV, np.uint32)
    adj[2:, 0] = 0                                           # everyone names hub 0 ...
    some = rng.permutation(np.arange(2, n))[:3000]
    adj[some, 1] = 1                                         # ... 3000 nodes name hub 1 ...
    for s in range(2, R):                                    # ... and the rest is a seeded random graph
        cand = rng.integers(2, n, size=n).astype(np.uint32)
        adj[:, s] = cand
    adj[some[:10], 2] = 40                                   # a short row as well
    # rows must not name a node twice, nor the node itself: repair by blanking, then pack to the front
    for s in range(1, R):
        dup = np.zeros(n, bool)
        for t in range(s):
            dup |= adj[:, s] == adj[:, t]
        dup |= adj[:, s] == np.arange(n)
        adj[dup, s] = INV
    order = np.argsort(adj == INV, axis=1, kind="stable")
    adj = np.take_along_axis(adj, order, axis=1)
    deg = (adj != INV).sum(1).astype(np.uint32)
    live = go.pack_bitmap(np.ones(n, bool))
    cfg = dict(dim=dim, dtype=go.U8, metric=go.L2, R=R, L=16, alpha=1.2, mode=go.FIXED_DEGREE, max_build_batch=64, ins=1, dele=64)
    o, g = make_pair(cfg, n, max_delete_edges=n * R)
    o.import_graph(adj, deg, live, 5, vecs)
    g.import_graph(torch.from_numpy(adj), torch.from_numpy(deg), torch.from_numpy(live), 5, torch.from_numpy(vecs))
    assert_same_graph(o, g, "imported")
    ids = np.array([0, 1, 40, 41, 77], np.uint32)
    o.delete_batch(ids); g.delete_batch(torch.from_numpy(ids))
    assert_same_graph(o, g, "hubs deleted")


# ------------------------------------------------------------------ fp32 streams: tolerance + recall
# Sizes: the largest shrinks whose oracle build finishes in about a minute on the test box's host cores
# (Deep-shaped 100,000 points, GIST-shaped 30,000, embedding-shaped 165,000).
@pytest.mark.parametrize("name,scale", [("deep_f32_d96", 0.01), ("gist_f32_d960", 0.025), ("embed_f32_d768_ip", 0.03)])
def test_fp32_streams_recall_matches_oracle(name, scale):
    cfg = small_cfg(name, scale, rounds=2, nq=200)
    cfg["first_batch"] = min(cfg["first_batch"], 500)
    cfg["max_build_batch"] = max(cfg["max_build_batch"], 500)
    o, _, wl, st = run_stream(cfg, seed=0, check_each=False, oracle=True, gpu=False)
    _, g, _, st2 = run_stream(cfg, seed=0, check_each=False, oracle=False, gpu=True)
    assert (st.live == st2.live).all() and (st.row_of == st2.row_of).all()
    # structural invariants of the GPU graph
    adj, deg, live, entry = gpu_graph(g)
    mask = go.live_mask(live, len(deg))
    assert (mask == st.live).all() and (deg <= cfg["R"]).all() and (deg[~mask] == 0).all() and mask[entry]
    for v in np.flatnonzero(mask)[:2000]:
        r = adj[v, :deg[v]]
        assert mask[r].all() and v not in r and len(set(r.tolist())) == len(r)
    # the vector every live id holds now (ids are reused in the GIST-shaped stream: the row map says which)
    live_ids = np.flatnonzero(st.live).astype(np.uint32)
    gen = wl.vectors(0, st.next_row)
    base = np.zeros((wl.capacity(), cfg["dim"]), np.float32)
    base[live_ids] = gen[st.row_of[live_ids]]
    q = wl.queries()
    truth = brute_force_topk(base, live_ids, q, 10, cfg["metric"])
    oi, _ = o.search(q, 10, cfg["L"])
    gi, gd = gpu_search(g, q, 10, cfg["L"])
    r_o, r_g = recall_at_k(oi, truth), recall_at_k(gi, truth)
    print(f"{name} x{scale}: {len(live_ids)} live points, recall@10 oracle {r_o:.4f} gpu {r_g:.4f}")
    assert abs(r_o - r_g) <= 0.005, (r_o, r_g)
    assert r_g > 0.6
    for i in range(0, len(q), 3):
        b = base[gi[i]].astype(np.float64)
        qq = q[i].astype(np.float64)
        exact = ((b - qq) ** 2).sum(1) if cfg["metric"] == go.L2 else -(b @ qq)
        scale_ = np.abs(exact) if cfg["metric"] == go.L2 else np.linalg.norm(b, axis=1) * np.linalg.norm(qq)
        assert (np.abs(gd[i] - exact) <= 1e-5 * scale_).all()


# ------------------------------------------------------------------ errors, host API, determinism
def test_errors_leave_index_unchanged():
    torch = torch_()
    from paper_2608_21163_b200.binding import GrandError
    cfg = small_cfg("tiny_u8_d32", 0.05)
    o, g, wl, st = run_stream(dict(cfg, rounds=0), seed=2)
    n = cfg["n"]
    before = gpu_graph(g)
    v = wl.vectors(0, 4)
    cases = [(np.array([n + 7, 1], np.uint32), -2), (np.array([0, 1], np.uint32), -4)]
    for ids, code in cases:
        with pytest.raises(GrandError) as e:
            g.insert_batch(torch.from_numpy(ids), torch.from_numpy(v[:len(ids)]))
        assert e.value.code == code
    d = np.array([3], np.uint32)
    o.delete_batch(d); g.delete_batch(torch.from_numpy(d))
    with pytest.raises(GrandError) as e:
        g.insert_batch(torch.from_numpy(np.array([3, 3], np.uint32)), torch.from_numpy(v[:2]))
    assert e.value.code == -3
    with pytest.raises(GrandError) as e:
        g.delete_batch(torch.from_numpy(d))
    assert e.value.code == -5
    with pytest.raises(GrandError) as e:
        g.delete_batch(torch.from_numpy(np.array([5, 5], np.uint32)))
    assert e.value.code == -3
    assert_same_graph(o, g, "after failed calls")
    with pytest.raises(GrandError):
        g.search(torch.from_numpy(v), 20, 10)
    # the index still works
    o.insert_batch(d, v[:1]); g.insert_batch(torch.from_numpy(d), torch.from_numpy(v[:1]))
    assert_same_graph(o, g, "after recovery")


def test_fixed_degree_mode_rejects_a_row_longer_than_the_search_list():
    from paper_2608_21163_b200 import binding as gb
    with pytest.raises(gb.GrandError):
        gb.GrandIndex(8, gb.U8, gb.L2, 33, 32, 1.2, capacity=100, max_batch=10, mode=gb.FIXED_DEGREE)
    gb.GrandIndex(8, gb.U8, gb.L2, 32, 32, 1.2, capacity=100, max_batch=10, mode=gb.FIXED_DEGREE)


def test_host_entry_points_match_device_entry_points():
    torch = torch_()
    cfg = small_cfg("tiny_u8_d32", 0.1, rounds=0)
    wl = synth.Workload(cfg, 3)
    n = cfg["n"]
    base = wl.vectors(0, n)
    o, g = make_pair(dict(cfg, max_build_batch=500, ins=500, dele=500), n)
    for lo in range(0, n, 250):
        ids = np.arange(lo, lo + 250, dtype=np.uint32)
        o.insert_batch(ids, base[ids])
        g.insert_batch_host(torch.from_numpy(ids).pin_memory(), torch.from_numpy(base[ids]).pin_memory())
    dele = synth.choose_ids(3, "del", np.arange(n, dtype=np.uint32), 100)
    o.delete_batch(dele)
    g.delete_batch_host(torch.from_numpy(dele).pin_memory())
    assert_same_graph(o, g, "host calls")
    q = wl.queries()
    out_i = torch.empty((len(q), 10), dtype=torch.uint32).pin_memory()
    out_d = torch.empty((len(q), 10), dtype=torch.int32).pin_memory()
    g.search_host(torch.from_numpy(q).pin_memory(), 10, cfg["L"], out_i, out_d)
    oi, od = o.search(q, 10, cfg["L"])
    assert (oi == out_i.numpy()).all() and (od == out_d.numpy().astype(np.float64)).all()


def test_run_twice_is_deterministic_and_counters_move():
    cfg = small_cfg("sift_u8_d128", 0.005, rounds=1)
    _, g1, wl, _ = run_stream(cfg, seed=7, oracle=False)
    _, g2, _, _ = run_stream(cfg, seed=7, oracle=False)
    a, b = gpu_graph(g1), gpu_graph(g2)
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all() and a[3] == b[3]
    s = g1.stats()
    assert s["expansions"] > 0 and s["dist_evals"] > s["expansions"] and s["pair_dists"] > 0
    assert s["dirty_nodes"] > 0 and s["prunes"] > 0 and s["kernel_launches"] > 0


def test_maximum_parameters_bit_exact():
    """Limits of the kernels' fast paths: R = 128 (four id chunks per row), L beyond 256, a visited-list cap
    of 600, P = 200 (candidate lists longer than the rank-merge buffer: full-sort path, 11-word bit
    matrix rows), c = 8 and k_repair = 128."""
    torch = torch_()
    n, dim = 3000, 16
    base = synth.uniform_u8(21, "base", 0, n, dim)
    cfg = dict(dim=dim, dtype=go.U8, metric=go.L2, R=128, L=300, alpha=1.2, mode=go.VAMANA, max_build_batch=1000, ins=1, dele=600)
    o, g = make_pair(cfg, n, P=200, c=8, k_repair=128, vmax=600)
    for lo in range(0, n, 750):
        ids = np.arange(lo, lo + 750, dtype=np.uint32)
        o.insert_batch(ids, base[ids]); g.insert_batch(torch.from_numpy(ids), torch.from_numpy(base[ids]))
        assert_same_graph(o, g, f"insert at {lo}")
    dele = synth.choose_ids(21, "del", np.arange(n, dtype=np.uint32), 600)
    o.delete_batch(dele); g.delete_batch(torch.from_numpy(dele))
    assert_same_graph(o, g, "delete")
    q = synth.uniform_u8(21, "query", 0, 100, dim)
    for k, L in [(10, 300), (100, 512), (1, 257)]:
        oi, od = o.search(q, k, L)
        gi, gd = gpu_search(g, q, k, L)
        assert (oi == gi).all() and (od == gd.astype(np.float64)).all()


def test_small_degree_bound_and_alpha_one():
    """R = 4 with alpha = 1.0: heavy pruning on every dirty node, rows shorter than a warp chunk."""
    torch = torch_()
    n, dim = 4000, 8
    base = synth.uniform_u8(22, "base", 0, n, dim)
    cfg = dict(dim=dim, dtype=go.U8, metric=go.L2, R=4, L=12, alpha=1.0, mode=go.VAMANA, max_build_batch=500, ins=1, dele=500)
    o, g = make_pair(cfg, n)
    for lo in range(0, n, 500):
        ids = np.arange(lo, lo + 500, dtype=np.uint32)
        o.insert_batch(ids, base[ids]); g.insert_batch(torch.from_numpy(ids), torch.from_numpy(base[ids]))
        assert_same_graph(o, g, f"insert at {lo}")
    for r in range(2):
        live = np.flatnonzero(go.live_mask(o.export_graph()[2], n)).astype(np.uint32)
        dele = synth.choose_ids(22, f"del{r}", live, 500)
        o.delete_batch(dele); g.delete_batch(torch.from_numpy(dele))
        assert_same_graph(o, g, f"delete {r}")
        o.insert_batch(dele[:250], base[dele[:250]]); g.insert_batch(torch.from_numpy(dele[:250]), torch.from_numpy(base[dele[:250]]))
        assert_same_graph(o, g, f"reinsert {r}")


def test_mips_reduction_vamana_ip_matches_oracle():
    """Vamana mode on the IP metric through the MIPS -> L2 reduction (Sec. 5.3): fp32, so the comparison is
    recall against brute-force maximum inner product (within 0.005 of the oracle's), negated inner products
    within 1e-5 of a float64 recomputation, and the graph invariants; a norm above the bound is refused."""
    torch = torch_()
    from paper_2608_21163_b200 import binding as gb
    n, d, R, L = 6000, 48, 24, 64
    scale = np.linspace(0.4, 1.0, n, dtype=np.float32)[:, None]
    base = (synth.aniso_unit_f32(5, "base", 0, n, d) * scale).astype(np.float32)
    q = synth.aniso_unit_f32(5, "query", 0, 300, d)
    o = go.Oracle(d, go.F32, go.IP, R, L, 1.2, n, max_norm=1.0)
    g = gb.GrandIndex(d, gb.F32, gb.IP, R, L, 1.2, capacity=n, max_batch=1000, mips_max_norm=1.0)
    for lo in range(0, n, 750):
        ids = np.arange(lo, lo + 750, dtype=np.uint32)
        o.insert_batch(ids, base[ids]); g.insert_batch(torch.from_numpy(ids), torch.from_numpy(base[ids]))
    dele = synth.choose_ids(5, "del", np.arange(n, dtype=np.uint32), 600)
    o.delete_batch(dele); g.delete_batch(torch.from_numpy(dele))
    adj, deg, live, entry = gpu_graph(g)
    mask = go.live_mask(live, n)
    assert mask.sum() == n - 600 == g.live_count and (deg <= R).all() and (deg[~mask] == 0).all() and mask[entry]
    for v in np.flatnonzero(mask)[:1500]:
        r = adj[v, :deg[v]]
        assert mask[r].all() and v not in r and len(set(r.tolist())) == len(r)
    live_ids = np.flatnonzero(mask).astype(np.uint32)
    truth = brute_force_topk(base, live_ids, q, 10, go.IP)
    oi, od = o.search(q, 10, L)
    gi, gd = gpu_search(g, q, 10, L)
    r_o, r_g = recall_at_k(oi, truth), recall_at_k(gi, truth)
    assert abs(r_o - r_g) <= 0.005 and r_g > 0.85, (r_o, r_g)
    for i in range(len(q)):
        b = base[gi[i]].astype(np.float64)
        exact = -(b @ q[i].astype(np.float64))
        # the reduction reports (d - |q|^2 - M^2) / 2 with d the squared L2 distance of the augmented rows: the
        # rounding error of d is relative to d <= |q|^2 + M^2 + 2 |q.x|, not to |q||x|, so that is the scale
        # 1e-5 applies to here (M = 1)
        assert (np.abs(gd[i] - exact) <= 1e-5 * 0.5 * ((q[i].astype(np.float64) ** 2).sum() + 1.0 + 2 * np.abs(exact))).all()
        assert (np.diff(gd[i]) >= -1e-6).all()
    with pytest.raises(gb.GrandError) as e:
        g.insert_batch(torch.from_numpy(dele[:2]), torch.from_numpy((base[:2] * 9).astype(np.float32)))
    assert e.value.code == -1
    g.insert_batch(torch.from_numpy(dele[:2]), torch.from_numpy(base[dele[:2]]))   # the index is still usable
    with pytest.raises(gb.GrandError):
        gb.GrandIndex(d, gb.U8, gb.IP, R, L, 1.2, capacity=n, mips_max_norm=1.0)  # fp32 only


# ------------------------------------------------------------------ hand-worked cases, straight from tests/golden/
from tests import golden_cases as gc


@pytest.mark.parametrize("fname,case", gc.all_cases(), ids=lambda x: x["name"] if isinstance(x, dict) else x.split(".")[0])
def test_hand_worked_graph_cases_on_the_gpu(fname, case):
    """The CUDA library against the hand-worked expected rows and medoids themselves (no oracle in between):
    Alg. 7 slot choice and forward row, Alg. 8 rewire and medoid replacement, the scratch bound of Alg. 6,
    the rounding of the initial medoid."""
    torch = torch_()
    from paper_2608_21163_b200 import binding as gb
    g = gb.GrandIndex(case["dim"], case["dtype"], case["metric"], case["R"], case["L"], case["alpha"], capacity=case["cap"],
                      max_batch=8, mode=case["mode"], **case["opts"])
    s = case["start"]
    if s is not None:
        g.import_graph(torch.from_numpy(s["adj"]), torch.from_numpy(s["deg"]), torch.from_numpy(go.pack_bitmap(s["live"])),
                       s["entry"], torch.from_numpy(s["vecs"]))
    for kind, ids, v in case["ops"]:
        if kind == "insert":
            g.insert_batch(torch.from_numpy(ids), torch.from_numpy(v))
        else:
            g.delete_batch(torch.from_numpy(ids))
    adj, deg, live, entry = gpu_graph(g)
    for v, want in case["expect_rows"].items():
        assert adj[v, :deg[v]].tolist() == want, (case["name"], v, adj[v, :deg[v]].tolist(), want)
    if case["expect_entry"] is not None:
        assert entry == case["expect_entry"]
