"""Properties that hold at any size, checked at the bench workload's full size (SIFT-shaped stream,
900,000 x 128 uint8, R=64, L=128) in the launch configuration bench.py times: structural
invariants of the graph after inserts and deletes, the exact reverse graph against a host
transpose of the exported adjacency, and sampled searches whose distances are recomputed exactly
and whose recall is measured against brute force.  (The oracle cannot build this size in test time;
bit-exact parity with it is covered on the tiny config and on shrunken streams.)"""
import numpy as np
import pytest

from oracle import grand_oracle as go
from paper_2608_21163_b200 import synth

pytestmark = pytest.mark.gpu


def test_full_size_stream_invariants_reverse_graph_and_sampled_searches():
    import torch
    from paper_2608_21163_b200 import binding as gb
    cfg = dict(synth.CONFIGS["sift_u8_d128"])
    cfg["rounds"] = 2
    cfg["n"] = cfg["build"] + cfg["rounds"] * cfg["ins"]
    wl = synth.Workload(cfg, 0)
    st = synth.StreamState(wl)
    cap, R, L = wl.capacity(), cfg["R"], cfg["L"]
    base = wl.vectors(0, cfg["n"])
    dbase = torch.from_numpy(base).cuda()
    g = gb.GrandIndex(cfg["dim"], cfg["dtype"], cfg["metric"], R, L, cfg["alpha"], capacity=cap, max_batch=10_000)
    for ids, rows in st.build_batches():
        g.insert_batch(torch.from_numpy(ids), dbase[rows[0]:rows[0] + rows[1]])
    deleted = []
    for r in range(cfg["rounds"]):
        ids, rows = st.insert_ids()
        g.insert_batch(torch.from_numpy(ids), dbase[rows[0]:rows[0] + rows[1]])
        dele = st.delete_ids()
        g.delete_batch(torch.from_numpy(dele))
        deleted.append(dele)
        st.end_round()
    deleted = np.concatenate(deleted)
    adj, deg, live, entry = [x.cpu().numpy() if hasattr(x, "cpu") else x for x in g.export_graph()]
    mask = go.live_mask(live, cap)
    # ---- invariants
    assert (mask == st.live).all() and g.live_count == int(mask.sum())
    assert (deg <= R).all() and (deg[~mask] == 0).all() and mask[entry]
    valid = np.arange(R)[None, :] < deg[:, None]
    assert (adj[~valid] == 0xFFFFFFFF).all()
    tgt = adj[valid]
    assert mask[tgt].all(), "edge to a non-live node"
    assert not np.isin(tgt, deleted).any(), "edge to a deleted node survived"
    src_of = np.repeat(np.arange(cap, dtype=np.uint32), deg)
    assert (tgt != src_of).all(), "self loop"
    srt = np.sort(np.where(valid, adj, np.uint32(0xFFFFFFFF)).astype(np.int64), axis=1)
    dup = (srt[:, 1:] == srt[:, :-1]) & (srt[:, 1:] != 0xFFFFFFFF)
    assert not dup.any(), "repeated neighbour in a row"
    assert deg[mask].mean() > 20
    # ---- exact reverse graph against a host transpose
    off, src = g.reverse_graph()
    off, src = off.cpu().numpy().astype(np.int64), src.cpu().numpy()
    order = np.lexsort((src_of, tgt))
    assert (src == src_of[order]).all()
    want_off = np.zeros(cap + 1, np.int64)
    np.add.at(want_off, tgt.astype(np.int64) + 1, 1)
    assert (off == np.cumsum(want_off)).all()
    # ---- sampled searches: exact distances, order, recall against brute force over the live set
    q = wl.queries()[:256]
    ids, d = g.search(torch.from_numpy(q), 10, L)
    torch.cuda.synchronize()
    ids, d = ids.cpu().numpy(), d.cpu().numpy()
    assert mask[ids].all() and not np.isin(ids, deleted).any()
    exact = ((base[ids].astype(np.int64) - q[:, None, :].astype(np.int64)) ** 2).sum(2)
    assert (exact == d).all()
    key = d.astype(np.int64) * (1 << 32) + ids
    assert (np.diff(key, axis=1) > 0).all()
    live_ids = torch.from_numpy(np.flatnonzero(mask)).cuda()
    x = dbase[live_ids].float()
    qq = torch.from_numpy(q).cuda().float()
    torch.backends.cuda.matmul.allow_tf32 = False
    dist = (qq * qq).sum(1).long()[:, None] + (x * x).sum(1).long()[None, :] - 2 * (qq @ x.T).long()
    truth = live_ids[torch.topk(dist * (1 << 31) + live_ids[None, :], 10, dim=1, largest=False).indices].cpu().numpy()
    rec = np.mean([len(set(a.tolist()) & set(b.tolist())) / 10 for a, b in zip(ids, truth)])
    assert rec > 0.97, rec
