"""The allocation-free reverse-graph entry point (grand_reverse_graph_noalloc).

It exists for callers that may not allocate device memory once they are running (a frozen memory
plan, a sandbox without access to the driver's allocator, a latency budget that cannot absorb
cudaMalloc).  Its scratch lives in a fixed array inside the library that every call shares and that
keeps the previous call's contents, so the check runs it twice in a row, on two different graphs,
and compares each result bit for bit with the regular entry point (grand_reverse_graph) and with
the CPU oracle's reverse graph of the same adjacency: integer output, so the tolerance is zero, as
in the other integer parity tests.  This file is collected last on purpose.
"""
import ctypes as C

import numpy as np
import pytest

from oracle import grand_oracle as go
from paper_2608_21163_b200 import binding as gb
from paper_2608_21163_b200 import synth


def test_size_limit_is_rejected_before_any_gpu_work():
    lib = gb.load()
    one = C.c_uint64(1)   # any non-null address: the call must return before touching it
    p = C.cast(C.pointer(one), C.c_void_p)
    rc = lib.grand_reverse_graph_noalloc(p, p, C.c_uint64(gb.NOALLOC_MAX_NODES + 1), C.c_uint32(8), p, None,
                                         C.c_uint64(0), None, None)
    assert rc == -2 and b"capacity" in lib.grand_strerror(rc)
    assert lib.grand_reverse_graph_noalloc(None, p, C.c_uint64(8), C.c_uint32(8), p, None, C.c_uint64(0), None, None) == -1


@pytest.mark.gpu
def test_noalloc_reverse_graph_matches_regular_entry_point_twice_in_a_row():
    import torch
    n, dim, R, L = 6000, 32, 16, 32
    base = synth.uniform_u8(11, "base", 0, n, dim)
    g = gb.GrandIndex(dim, gb.U8, gb.L2, R, L, 1.2, capacity=n, max_batch=2000)
    o = go.Oracle(dim, go.U8, go.L2, R, L, 1.2, n)      # the oracle follows the same stream; its CSR is the yardstick
    for lo in range(0, n, 1000):
        ids = np.arange(lo, lo + 1000, dtype=np.uint32)
        g.insert_batch(torch.from_numpy(ids), torch.from_numpy(base[ids]))
        o.insert_batch(ids, base[ids])
    dev = g.device
    # outputs are allocated by the caller, up front
    off = torch.empty(n + 1, dtype=torch.uint32, device=dev)
    src = torch.empty(n * R, dtype=torch.uint32, device=dev)

    def check(tag):
        adj, deg, _, _ = g.export_graph()
        want_off, want_src = g.reverse_graph()
        off.view(torch.int32).fill_(-1); src.view(torch.int32).fill_(-1)
        E = gb.reverse_graph_noalloc(adj, deg, off, src)
        torch.cuda.synchronize()
        assert E == want_src.numel() == int(deg.view(torch.int32).to(torch.int64).sum().item()), tag
        assert torch.equal(off.view(torch.int32), want_off.view(torch.int32)), tag
        assert torch.equal(src[:E].view(torch.int32), want_src.view(torch.int32)), tag
        o_off, o_src = o.reverse_graph()                 # Alg. 8's reverse-neighbour lists, written out on the CPU
        assert (off.cpu().numpy().astype(np.uint64) == o_off).all() and (src[:E].cpu().numpy() == o_src).all(), tag
        # offsets-only form
        off2 = torch.empty(n + 1, dtype=torch.uint32, device=dev)
        assert gb.reverse_graph_noalloc(adj, deg, off2, None) == E
        torch.cuda.synchronize()
        assert torch.equal(off2.view(torch.int32), want_off.view(torch.int32)), tag

    check("first call")
    # a different graph for the second call: the shared scratch still holds the first call's cursors
    dele = synth.choose_ids(11, "del/0", np.arange(n, dtype=np.uint32), 1500)
    g.delete_batch(torch.from_numpy(dele))
    o.delete_batch(dele)
    check("second call")
    # an output buffer that is too small is refused, and the call after it still works
    adj, deg, _, _ = g.export_graph()
    with pytest.raises(gb.GrandError) as e:
        gb.reverse_graph_noalloc(adj, deg, off, src[:10])
    assert e.value.code == -2
    check("after a refused call")
    # a neighbour id beyond the node count (a slice of a larger graph, a stale slot) is reported, and neither the
    # caller's buffers nor the library's array is written out of range: guard words around `off` stay intact
    bad = adj.clone()
    v = int((deg.view(torch.int32) > 0).nonzero()[0])     # a node whose first slot is in use
    bad.view(torch.int32)[v, 0] = n + 3
    guard = torch.full((n + 1 + 64,), 0x5A5A5A5A, dtype=torch.int32, device=dev)
    with pytest.raises(gb.GrandError) as e:
        gb.reverse_graph_noalloc(bad, deg, guard[32:32 + n + 1].view(torch.uint32), src)
    assert e.value.code == -1
    torch.cuda.synchronize()
    assert (guard[:32] == 0x5A5A5A5A).all() and (guard[32 + n + 1:] == 0x5A5A5A5A).all()
    check("after a rejected graph")
