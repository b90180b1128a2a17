"""Properties of the C-ABI boundary itself, through the C-ABI: the update path allocates nothing after the index is
created, a delete batch beyond the configured edge bound is refused whole, a caller-supplied graph is checked before
it replaces anything, launches are counted per handle, and more asynchronous searches than the library has work
counters still return the oracle's answers."""
import ctypes as C

import numpy as np
import pytest

from oracle import grand_oracle as go
from paper_2608_21163_b200 import synth
from tests.helpers import INV, assert_same_graph, gpu_graph, make_pair

pytestmark = pytest.mark.gpu


def _hooks(log):
    """dev_alloc / dev_free hooks that route through torch's caching allocator and log every call."""
    import torch
    ALLOC = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
    FREE = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)

    def alloc(nbytes, _user):
        p = torch.cuda.caching_allocator_alloc(max(int(nbytes), 1))
        log.append(("alloc", int(nbytes)))
        return p

    def free(p, _user):
        log.append(("free", 0))
        if p:
            torch.cuda.caching_allocator_delete(p)

    return ALLOC(alloc), FREE(free)


def test_update_path_allocates_nothing_after_creation():
    import torch
    from paper_2608_21163_b200 import binding as gb
    n, dim, R, L, B = 6000, 32, 16, 32, 500
    base = synth.uniform_u8(31, "base", 0, n, dim)
    q = synth.uniform_u8(31, "query", 0, 200, dim)
    log = []
    a, f = _hooks(log)
    g = gb.GrandIndex(dim, gb.U8, gb.L2, R, L, 1.2, capacity=n, max_batch=B, dev_alloc=a, dev_free=f)
    o = go.Oracle(dim, go.U8, go.L2, R, L, 1.2, n)
    assert len(log) > 10 and all(k == "alloc" for k, _ in log)      # the whole pool comes from the hook
    created = len(log)
    alive = np.zeros(n, bool)
    out_i = torch.empty((len(q), 10), dtype=torch.uint32, device="cuda")
    out_d = torch.empty((len(q), 10), dtype=torch.int32, device="cuda")
    pin_i = torch.empty((B,), dtype=torch.uint32).pin_memory()
    for step in range(8):
        ids = np.arange(step * B, (step + 1) * B, dtype=np.uint32)
        o.insert_batch(ids, base[ids])
        if step % 2:
            g.insert_batch_host(torch.from_numpy(ids).pin_memory(), torch.from_numpy(base[ids]).pin_memory())
        else:
            g.insert_batch(torch.from_numpy(ids), torch.from_numpy(base[ids]))
        alive[ids] = True
        if step >= 2:
            dele = synth.choose_ids(31, f"del/{step}", np.flatnonzero(alive).astype(np.uint32), B // 2)
            o.delete_batch(dele)
            if step % 2:
                pin_i[:len(dele)] = torch.from_numpy(dele)
                g.delete_batch_host(pin_i[:len(dele)])
            else:
                g.delete_batch(torch.from_numpy(dele))
            alive[dele] = False
        g.search(torch.from_numpy(q), 10, L, out_i, out_d)
    torch.cuda.synchronize()
    assert len(log) == created, log[created:]                        # inserts, deletes, searches: no allocator call
    assert_same_graph(o, g, "stream through the hooked allocator")
    g.close()
    assert sum(k == "free" for k, _ in log) == created               # and everything goes back through the hook


def test_delete_batch_beyond_the_edge_bound_is_refused_whole():
    import torch
    from paper_2608_21163_b200 import binding as gb
    n, dim, R, L = 3000, 16, 12, 24
    base = synth.uniform_u8(32, "base", 0, n, dim)
    cfg = dict(dim=dim, dtype=go.U8, metric=go.L2, R=R, L=L, alpha=1.2, mode=go.VAMANA, max_build_batch=600, ins=600, dele=600)
    o = go.Oracle(dim, go.U8, go.L2, R, L, 1.2, n)
    g = gb.GrandIndex(dim, gb.U8, gb.L2, R, L, 1.2, capacity=n, max_batch=600, max_delete_edges=2000)
    for lo in range(0, n, 600):
        ids = np.arange(lo, lo + 600, dtype=np.uint32)
        o.insert_batch(ids, base[ids]); g.insert_batch(torch.from_numpy(ids), torch.from_numpy(base[ids]))
    before = gpu_graph(g)
    big = synth.choose_ids(32, "del/big", np.arange(n, dtype=np.uint32), 600)        # ~600 * in-degree entries > 2000
    with pytest.raises(gb.GrandError) as e:
        g.delete_batch(torch.from_numpy(big))
    assert e.value.code == -2 and "max_delete_edges" in str(e.value)
    after = gpu_graph(g)
    assert all((a == b).all() for a, b in zip(before[:3], after[:3])) and before[3] == after[3]
    # the refused batch left no marks behind: the same ids go through in pieces that fit
    small = big[:100]
    o.delete_batch(small); g.delete_batch(torch.from_numpy(small))
    assert_same_graph(o, g, "after a refused batch")
    o.insert_batch(small, base[small]); g.insert_batch(torch.from_numpy(small), torch.from_numpy(base[small]))
    assert_same_graph(o, g, "re-insert after a refused batch")


def test_import_graph_checks_the_callers_graph():
    import torch
    from paper_2608_21163_b200 import binding as gb
    n, dim, R = 64, 8, 4
    g = gb.GrandIndex(dim, gb.U8, gb.L2, R, 8, 1.2, capacity=n, max_batch=16)
    vecs = synth.uniform_u8(33, "base", 0, n, dim)
    ids = np.arange(16, dtype=np.uint32)
    g.insert_batch(torch.from_numpy(ids), torch.from_numpy(vecs[:16]))
    before = gpu_graph(g)
    adj = np.full((n, R), INV, np.uint32)
    deg = np.zeros(n, np.uint32)
    adj[0, :2] = [1, 2]; deg[0] = 2
    live = go.pack_bitmap(np.arange(n) < 3)
    for bad_adj, bad_deg in [((0, 1, n + 5), None), (None, (1, R + 1))]:
        a2, d2 = adj.copy(), deg.copy()
        if bad_adj:
            a2[bad_adj[0], bad_adj[1]] = bad_adj[2]
        if bad_deg:
            d2[bad_deg[0]] = bad_deg[1]
        with pytest.raises(gb.GrandError) as e:
            g.import_graph(torch.from_numpy(a2), torch.from_numpy(d2), torch.from_numpy(live), 0, torch.from_numpy(vecs))
        assert e.value.code == -1
        after = gpu_graph(g)
        assert all((x == y).all() for x, y in zip(before[:3], after[:3])) and before[3] == after[3] and g.live_count == 16
    g.import_graph(torch.from_numpy(adj), torch.from_numpy(deg), torch.from_numpy(live), 0, torch.from_numpy(vecs))
    assert g.live_count == 3


def test_kernel_launches_are_counted_per_handle():
    import torch
    from paper_2608_21163_b200 import binding as gb
    v = synth.uniform_u8(34, "base", 0, 64, 8)
    g1 = gb.GrandIndex(8, gb.U8, gb.L2, 4, 8, 1.2, capacity=64, max_batch=32)
    g2 = gb.GrandIndex(8, gb.U8, gb.L2, 4, 8, 1.2, capacity=64, max_batch=32)
    g1.insert_batch(torch.from_numpy(np.arange(32, dtype=np.uint32)), torch.from_numpy(v[:32]))
    a1, a2 = g1.stats()["kernel_launches"], g2.stats()["kernel_launches"]
    assert a1 > 0 and a2 == 0
    g2.search(torch.from_numpy(v[:4]), 2, 8)
    assert g1.stats()["kernel_launches"] == a1 and g2.stats()["kernel_launches"] == 1


def test_more_asynchronous_searches_than_work_counters():
    """grand_search hands its queries out through a per-launch counter; the library keeps 64 of them.  150 launches
    queued on four streams without a synchronisation in between must each still answer every query once."""
    import torch
    n, dim, R, L = 4000, 32, 16, 32
    base = synth.uniform_u8(35, "base", 0, n, dim)
    q = synth.uniform_u8(35, "query", 0, 1500, dim)
    cfg = dict(dim=dim, dtype=go.U8, metric=go.L2, R=R, L=L, alpha=1.2, mode=go.VAMANA, max_build_batch=500, ins=1, dele=1)
    o, g = make_pair(cfg, n)
    for lo in range(0, n, 500):
        ids = np.arange(lo, lo + 500, dtype=np.uint32)
        o.insert_batch(ids, base[ids]); g.insert_batch(torch.from_numpy(ids), torch.from_numpy(base[ids]))
    want_i, want_d = o.search(q, 10, L)
    qd = torch.from_numpy(q).cuda()
    streams = [torch.cuda.Stream() for _ in range(4)]
    outs = []
    torch.cuda.synchronize()
    for k in range(150):
        oi = torch.full((len(q), 10), 7, dtype=torch.int32, device="cuda").view(torch.uint32)
        od = torch.full((len(q), 10), -7, dtype=torch.int32, device="cuda")
        outs.append((oi, od))
    torch.cuda.synchronize()
    for k in range(150):
        with torch.cuda.stream(streams[k % 4]):
            g.search(qd, 10, L, outs[k][0], outs[k][1])
    torch.cuda.synchronize()
    for k in (0, 1, 63, 64, 65, 100, 149):
        assert (outs[k][0].cpu().numpy() == want_i).all(), k
        assert (outs[k][1].cpu().numpy().astype(np.float64) == want_d).all(), k
    same = torch.stack([o_[0].view(torch.int32) for o_ in outs])
    assert (same == same[0]).all()
