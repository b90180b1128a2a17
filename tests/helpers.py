"""Shared helpers of the parity tests: drive the CPU oracle and the CUDA library with the same
seeded op stream and compare their states."""
import numpy as np

from oracle import grand_oracle as go
from paper_2608_21163_b200 import synth

INV = 0xFFFFFFFF


def oracle_opts(opts):
    """The library's option names, translated to the oracle's constructor arguments."""
    o = dict(opts)
    if "visited_set_delete" in o:
        o["approx_delete"] = o.pop("visited_set_delete")
    o.pop("snapshot_search", None)     # a property of the library's memory management, not of the method
    o.pop("max_delete_edges", None)    # workspace sizing of the library
    return o


def make_pair(cfg, capacity, **opts):
    """(oracle, gpu index) with identical parameters."""
    from paper_2608_21163_b200 import binding as gb
    o = go.Oracle(cfg["dim"], cfg["dtype"], cfg["metric"], cfg["R"], cfg["L"], cfg["alpha"], capacity,
                  mode=cfg["mode"], **oracle_opts(opts))
    g = gb.GrandIndex(cfg["dim"], cfg["dtype"], cfg["metric"], cfg["R"], cfg["L"], cfg["alpha"], capacity=capacity,
                      max_batch=max(cfg.get("first_batch", 1), cfg["max_build_batch"], cfg["ins"], cfg["dele"], 1), mode=cfg["mode"], **opts)
    return o, g


def gpu_graph(g):
    adj, deg, live, entry = g.export_graph()
    return adj.cpu().numpy(), deg.cpu().numpy(), live.cpu().numpy(), entry


def assert_same_graph(o, g, what=""):
    oa, od, ol, oe = o.export_graph()
    ga, gd, gl, ge = gpu_graph(g)
    assert (ol == gl).all(), f"{what}: live bitmaps differ"
    assert oe == ge, f"{what}: medoid differs {oe} vs {ge}"
    bad = np.flatnonzero(od != gd)
    assert len(bad) == 0, f"{what}: degrees differ at {bad[:10]} oracle {od[bad[:10]]} gpu {gd[bad[:10]]}"
    R = oa.shape[1]
    valid = np.arange(R)[None, :] < od[:, None]
    diff = (oa != ga) & valid
    rows = np.flatnonzero(diff.any(1))
    assert len(rows) == 0, (f"{what}: {len(rows)} adjacency rows differ, first {rows[0]}: "
                            f"oracle {oa[rows[0], :od[rows[0]]]} gpu {ga[rows[0], :gd[rows[0]]]}")
    assert (ga[~valid] == INV).all(), f"{what}: unused slots must hold the invalid id"
    assert o.live_count == g.live_count


def run_stream(cfg, seed=0, check_each=True, oracle=True, gpu=True, opts=None, on_round=None):
    """Build + rounds of (insert, delete) as the config says.  Returns (oracle, gpu, workload, state)."""
    import torch
    from paper_2608_21163_b200 import binding as gb
    wl = synth.Workload(cfg, seed)
    st = synth.StreamState(wl)
    cap = wl.capacity()
    opts = opts or {}
    o = g = None
    if oracle and gpu:
        o, g = make_pair(cfg, cap, **opts)
    elif oracle:
        o = go.Oracle(cfg["dim"], cfg["dtype"], cfg["metric"], cfg["R"], cfg["L"], cfg["alpha"], cap, mode=cfg["mode"], **oracle_opts(opts))
    else:
        g = gb.GrandIndex(cfg["dim"], cfg["dtype"], cfg["metric"], cfg["R"], cfg["L"], cfg["alpha"], capacity=cap,
                          max_batch=max(cfg.get("first_batch", 1), cfg["max_build_batch"], cfg["ins"], cfg["dele"], 1), mode=cfg["mode"], **opts)

    st.row_of = np.full(cap, -1, np.int64)     # id -> row of the generated base array that the id holds now

    def ins(ids, rows, what):
        v = wl.vectors(*rows)
        st.row_of[ids] = np.arange(rows[0], rows[0] + rows[1])
        if o:
            o.insert_batch(ids, v)
        if g:
            g.insert_batch(torch.from_numpy(ids), torch.from_numpy(v))
        if o and g and check_each:
            assert_same_graph(o, g, what)

    def dele(ids, what):
        if o:
            o.delete_batch(ids)
        if g:
            g.delete_batch(torch.from_numpy(ids))
        if o and g and check_each:
            assert_same_graph(o, g, what)

    for bi, (ids, rows) in enumerate(st.build_batches()):
        ins(ids, rows, f"build batch {bi}")
    for r in range(cfg["rounds"]):
        if cfg.get("delete_first"):
            dele(st.delete_ids(), f"round {r} delete")
            ids, rows = st.insert_ids()
            ins(ids, rows, f"round {r} insert")
        else:
            ids, rows = st.insert_ids()
            ins(ids, rows, f"round {r} insert")
            dele(st.delete_ids(), f"round {r} delete")
        st.end_round()
        if on_round:
            on_round(r, o, g, wl, st)
    if o and g and not check_each:
        assert_same_graph(o, g, "final")
    return o, g, wl, st


def brute_force_topk(base, live_ids, queries, k, metric):
    """Exact top-k over the live set, ties by id (float64 on the host)."""
    b = base[live_ids].astype(np.float64)
    out = np.empty((len(queries), k), np.uint32)
    for i, q in enumerate(queries.astype(np.float64)):
        d = ((b - q[None, :]) ** 2).sum(1) if metric == 0 else -(b @ q)
        order = np.lexsort((live_ids, d))[:k]
        out[i] = live_ids[order]
    return out


def recall_at_k(found, truth):
    hit = sum(len(set(f.tolist()) & set(t.tolist())) for f, t in zip(found, truth))
    return hit / truth.size
