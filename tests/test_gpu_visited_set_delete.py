"""Parity of the visited-set delete variant (Alg. 6 as printed: in-neighbours of a deleted node are
looked for among the nodes its search visited, other edges to it stay behind as dangling edges and
every traversal checks liveness) between the CUDA library and the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import grand_oracle as go
from paper_2608_21163_b200 import synth
from tests.helpers import INV, assert_same_graph, brute_force_topk, recall_at_k, run_stream

pytestmark = pytest.mark.gpu


def test_hand_case_leaves_the_same_dangling_edge():
    from paper_2608_21163_b200 import binding as gb
    base = (10 * np.arange(6))[:, None].astype(np.uint8)
    rows = {0: [1], 1: [0, 2], 2: [1, 3], 3: [2, 4], 4: [3], 5: [2]}
    adj = np.full((6, 2), INV, np.uint32)
    deg = np.zeros(6, np.uint32)
    for v, r in rows.items():
        adj[v, :len(r)] = r
        deg[v] = len(r)
    live = go.pack_bitmap(np.ones(6, bool))
    o = go.Oracle(1, go.U8, go.L2, 2, 8, 1.2, 6, c=2, k_repair=4, approx_delete=1)
    g = gb.GrandIndex(1, gb.U8, gb.L2, 2, 8, 1.2, capacity=6, max_batch=4, c=2, k_repair=4, visited_set_delete=1)
    o.import_graph(adj, deg, live, 0, base)
    g.import_graph(torch.from_numpy(adj), torch.from_numpy(deg), torch.from_numpy(live), 0, torch.from_numpy(base))
    o.delete_batch(np.array([2], np.uint32))
    g.delete_batch(torch.tensor([2], dtype=torch.int64).to(torch.uint32))
    assert_same_graph(o, g, "delete of node 2")
    ga = g.export_graph()[0].cpu().numpy()
    assert ga[5, 0] == 2                                    # the edge nobody visited is still there
    q = np.array([[50]], np.uint8)
    oi, _ = o.search(q, 3, 8)
    gi, _ = g.search(torch.from_numpy(q), 3, 8)
    assert (oi == gi.cpu().numpy()).all() and 2 not in oi[0].tolist()
    back = np.array([2], np.uint32)
    o.insert_batch(back, np.array([[55]], np.uint8))
    g.insert_batch(torch.from_numpy(back), torch.tensor([[55]], dtype=torch.uint8))
    assert_same_graph(o, g, "id 2 comes back")


@pytest.mark.parametrize("name,scale,reuse", [("tiny_u8_d32", 1.0, False), ("sift_u8_d128", 0.02, False),
                                              ("tiny_u8_d32", 1.0, True)])
def test_stream_bit_exact_with_dangling_edges(name, scale, reuse):
    cfg = synth.scaled(synth.CONFIGS[name], scale)
    cfg["nq"] = 200
    if reuse:   # freed ids come back with new vectors, so an old dangling edge turns into an edge to the new node
        cfg.update(reuse_ids=True, delete_first=True, ins=600, dele=1000, rounds=4)
    seen = {"dangling": 0}

    def on_round(r, o, g, wl, st):
        adj, deg, live, _ = o.export_graph()
        mask = go.live_mask(live, len(deg))
        valid = np.arange(adj.shape[1])[None, :] < deg[:, None]
        seen["dangling"] += int((~mask[adj[valid]]).sum())
        q = wl.queries()
        oi, od = o.search(q, 10, cfg["L"])
        gi, gd = g.search(torch.from_numpy(q), 10, cfg["L"])
        gi = gi.cpu().numpy()
        assert (oi == gi).all() and (od == gd.cpu().numpy().astype(np.float64)).all()
        assert mask[gi[gi != INV]].all()                     # a search never returns a deleted id

    run_stream(cfg, seed=3, opts={"visited_set_delete": 1}, on_round=on_round)
    assert seen["dangling"] > 0                              # the stream really exercises the liveness checks


def test_stream_fp32_recall_matches_oracle():
    cfg = synth.scaled(synth.CONFIGS["deep_f32_d96"], 0.002)
    cfg.update(rounds=2, nq=200)
    cfg["first_batch"] = min(cfg["first_batch"], 500)
    cfg["max_build_batch"] = max(cfg["max_build_batch"], 500)
    opts = {"visited_set_delete": 1}
    o, _, wl, st = run_stream(cfg, seed=0, check_each=False, oracle=True, gpu=False, opts=opts)
    _, g, _, st2 = run_stream(cfg, seed=0, check_each=False, oracle=False, gpu=True, opts=opts)
    assert (st.live == st2.live).all()
    adj, deg, live, entry = (t.cpu().numpy() if hasattr(t, "cpu") else t for t in g.export_graph())
    mask = go.live_mask(live, len(deg))
    assert (mask == st.live).all() and (deg <= cfg["R"]).all() and (deg[~mask] == 0).all() and mask[entry]
    base = np.zeros((wl.capacity(), cfg["dim"]), np.float32)
    base[:st.next_row] = wl.vectors(0, st.next_row)
    live_ids = np.flatnonzero(st.live).astype(np.uint32)
    q = wl.queries()
    truth = brute_force_topk(base, live_ids, q, 10, cfg["metric"])
    oi, _ = o.search(q, 10, cfg["L"])
    gi, _ = g.search(torch.from_numpy(q), 10, cfg["L"])
    gi = gi.cpu().numpy()
    r_o, r_g = recall_at_k(oi, truth), recall_at_k(gi, truth)
    assert abs(r_o - r_g) <= 0.005 and r_g > 0.8, (r_o, r_g)
    assert mask[gi[gi != INV]].all()
