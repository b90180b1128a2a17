"""The paper's streaming patterns (Sec. 5.2: Sliding Window, Interleaved, Expiration Time, Clustered,
Insert Heavy) on a SIFT-shaped shrink: the CUDA library must track the CPU oracle bit for bit through
every op of every pattern, and every search of the stream must return identical ids and distances."""
import numpy as np
import pytest

from oracle import grand_oracle as go
from paper_2608_21163_b200 import synth
from tests.helpers import assert_same_graph

pytestmark = pytest.mark.gpu

N, DIM, R, L = 6000, 128, 32, 64


def patterns():
    cl = synth.mixture_centre_of(0, "base", 0, N) % 64
    return {
        "sliding_window": lambda: synth.pattern_sliding_window(N, 20, 10, 150),
        "interleaved": lambda: synth.pattern_interleaved(N, 200, n_ops=40),
        "expiration_time": lambda: synth.pattern_expiration(N, 200),
        "clustered": lambda: synth.pattern_clustered(N, 250, cl),
        "insert_heavy": lambda: synth.pattern_insert_heavy(N, 400),
    }


@pytest.mark.parametrize("name", ["sliding_window", "interleaved", "expiration_time", "clustered", "insert_heavy"])
def test_pattern_bit_exact(name):
    import torch
    from paper_2608_21163_b200 import binding as gb
    base = synth.mixture_u8(0, "base", 0, N, DIM)
    q = synth.mixture_u8(0, "query", 0, 100, DIM)
    o = go.Oracle(DIM, go.U8, go.L2, R, L, 1.2, N)
    g = gb.GrandIndex(DIM, gb.U8, gb.L2, R, L, 1.2, capacity=N, max_batch=1000)
    nops = nsearch = 0
    for op in patterns()[name]():
        if op[0] == "insert":
            o.insert_batch(op[1], base[op[1]]); g.insert_batch(torch.from_numpy(op[1]), torch.from_numpy(base[op[1]]))
        elif op[0] == "delete":
            o.delete_batch(op[1]); g.delete_batch(torch.from_numpy(op[1]))
        else:
            oi, od = o.search(q, 10, L)
            gi, gd = g.search(torch.from_numpy(q), 10, L)
            torch.cuda.synchronize()
            assert (oi == gi.cpu().numpy()).all() and (od == gd.cpu().numpy().astype(np.float64)).all(), f"{name}: search {nsearch}"
            nsearch += 1
            continue
        nops += 1
        if nops % 5 == 0:
            assert_same_graph(o, g, f"{name}: op {nops}")
    assert_same_graph(o, g, f"{name}: end")
    assert nops > 10 and (nsearch > 0 or name == "insert_heavy")
    assert o.stats()["dead_edges_seen"] == 0
