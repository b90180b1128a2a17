"""ctypes access to the CPU oracle (oracle/grand_oracle.cpp) -- TEST INFRASTRUCTURE.

Only the test-suite, the smoke check and the CPU-baseline leg of the benchmark may import this
module; the CUDA product path never does.  The oracle restates GrAND's Alg. 1 (BeamSearch),
Alg. 4 (RobustPrune), Alg. 5/6 (Vamana batch insert/delete, in-neighbours from the exact reverse
graph of Alg. 8) and Alg. 7/8 (fixed-degree mode) under deterministic batch semantics.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "grand_oracle.cpp")
_LIB = os.path.join(_HERE, "libgrand_oracle.so")

U8, I8, F32 = 0, 1, 2
L2, IP = 0, 1
VAMANA, FIXED_DEGREE = 0, 1
INVALID = 0xFFFFFFFF
_NP = {U8: np.uint8, I8: np.int8, F32: np.float32}


def build(force=False):
    """Compile the oracle with plain g++ -O2 (no fast-math, no contraction)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
           "-o", _LIB, _SRC]
    subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.grand_oracle_dist.restype = C.c_double
        _lib.grand_oracle_get_entry.restype = C.c_uint32
        _lib.grand_oracle_live_count.restype = C.c_uint64
        _lib.grand_oracle_destroy.restype = None
        _lib.grand_oracle_set_entry.restype = None
        _lib.grand_oracle_get_stats.restype = None
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle error {code}")
        self.code = code


class Oracle:
    def __init__(self, dim, dtype, metric, R, L, alpha, capacity, P=0, c=0, k_repair=0, vmax=0,
                 mode=VAMANA, nthreads=0, max_norm=0.0, approx_delete=0):
        self.dim, self.dtype, self.metric, self.R, self.L = dim, dtype, metric, R, L
        self.capacity = int(capacity)
        self.np_dtype = _NP[dtype]
        if nthreads == 0:
            nthreads = min(len(os.sched_getaffinity(0)), 64)
        self.nthreads = nthreads
        h = C.c_void_p()
        rc = lib().grand_oracle_create(C.c_uint32(dim), C.c_uint32(dtype), C.c_uint32(metric), C.c_uint32(R),
                                       C.c_uint32(L), C.c_float(alpha), C.c_uint64(capacity), C.c_uint32(P),
                                       C.c_uint32(c), C.c_uint32(k_repair), C.c_uint32(vmax), C.c_uint32(mode),
                                       C.c_uint32(nthreads), C.c_float(max_norm), C.c_uint32(approx_delete), C.byref(h))
        if rc != 0:
            raise OracleError(rc)
        self.h = h

    def __del__(self):
        if getattr(self, "h", None):
            lib().grand_oracle_destroy(self.h)
            self.h = None

    def _vec(self, a):
        a = np.ascontiguousarray(a, dtype=self.np_dtype)
        assert a.shape[-1] == self.dim
        return a

    def insert_batch(self, ids, vecs):
        ids = np.ascontiguousarray(ids, dtype=np.uint32)
        vecs = self._vec(vecs)
        rc = lib().grand_oracle_insert_batch(self.h, _p(ids), _p(vecs), C.c_uint64(len(ids)))
        if rc != 0:
            raise OracleError(rc)

    def delete_batch(self, ids):
        ids = np.ascontiguousarray(ids, dtype=np.uint32)
        rc = lib().grand_oracle_delete_batch(self.h, _p(ids), C.c_uint64(len(ids)))
        if rc != 0:
            raise OracleError(rc)

    def search(self, queries, k, L, use_seen_set=False):
        q = self._vec(queries)
        nq = q.shape[0]
        ids = np.empty((nq, k), np.uint32)
        d = np.empty((nq, k), np.float64)
        rc = lib().grand_oracle_search(self.h, _p(q), C.c_uint64(nq), C.c_uint32(k), C.c_uint32(L),
                                       C.c_uint32(int(use_seen_set)), _p(ids), _p(d))
        if rc != 0:
            raise OracleError(rc)
        return ids, d

    def greedy(self, q, L, vmax, use_seen_set=False):
        q = self._vec(q)
        bi = np.empty(L, np.uint32); bd = np.empty(L, np.float64)
        vi = np.empty(vmax, np.uint32); vd = np.empty(vmax, np.float64)
        nb = C.c_uint32(); nv = C.c_uint32()
        lib().grand_oracle_greedy(self.h, _p(q), C.c_uint32(L), C.c_uint32(vmax), C.c_uint32(int(use_seen_set)),
                                  _p(bi), _p(bd), C.byref(nb), _p(vi), _p(vd), C.byref(nv))
        return (bi[:nb.value], bd[:nb.value]), (vi[:nv.value], vd[:nv.value])

    def dist(self, a, b):
        a = self._vec(a); b = self._vec(b)
        return lib().grand_oracle_dist(self.h, _p(a), _p(b))

    def prune(self, p, cand_ids, cand_d, R):
        ci = np.ascontiguousarray(cand_ids, dtype=np.uint32)
        cd = np.ascontiguousarray(cand_d, dtype=np.float64)
        out = np.empty(max(R, 1), np.uint32)
        n = C.c_uint32()
        lib().grand_oracle_prune(self.h, C.c_uint32(p), _p(ci), _p(cd), C.c_uint32(len(ci)), C.c_uint32(R),
                                 _p(out), C.byref(n))
        return out[:n.value].copy()

    def export_graph(self):
        adj = np.empty((self.capacity, self.R), np.uint32)
        deg = np.empty(self.capacity, np.uint32)
        live = np.empty((self.capacity + 31) // 32, np.uint32)
        e = C.c_uint32()
        lib().grand_oracle_export_graph(self.h, _p(adj), _p(deg), _p(live), C.byref(e))
        return adj, deg, live, e.value

    def import_graph(self, adj, deg, live_bitmap, entry, vecs):
        adj = np.ascontiguousarray(adj, dtype=np.uint32).reshape(self.capacity, self.R)
        deg = np.ascontiguousarray(deg, dtype=np.uint32)
        live = np.ascontiguousarray(live_bitmap, dtype=np.uint32)
        vecs = self._vec(vecs)
        assert vecs.shape[0] == self.capacity and len(deg) == self.capacity
        lib().grand_oracle_import_graph(self.h, _p(adj), _p(deg), _p(live), C.c_uint32(entry), _p(vecs))

    def reverse_graph(self):
        E = C.c_uint64()
        off = np.empty(self.capacity + 1, np.uint64)
        lib().grand_oracle_reverse_graph(self.h, _p(off), None, C.byref(E))
        src = np.empty(max(E.value, 1), np.uint32)
        lib().grand_oracle_reverse_graph(self.h, _p(off), _p(src), C.byref(E))
        return off, src[:E.value]

    @property
    def entry(self):
        return lib().grand_oracle_get_entry(self.h)

    @entry.setter
    def entry(self, e):
        lib().grand_oracle_set_entry(self.h, C.c_uint32(e))

    @property
    def live_count(self):
        return lib().grand_oracle_live_count(self.h)

    def stats(self):
        s = np.zeros(5, np.uint64)
        lib().grand_oracle_get_stats(self.h, _p(s))
        return dict(zip(["expansions", "dist_evals", "dead_edges_seen", "prunes", "dirty"], s.tolist()))


def live_mask(live_bitmap, capacity):
    """Expand a uint32 bitmap into a boolean mask of length capacity."""
    bits = np.unpackbits(live_bitmap.view(np.uint8), bitorder="little")
    return bits[:capacity].astype(bool)


def pack_bitmap(mask):
    n = len(mask)
    pad = (-n) % 32
    b = np.concatenate([np.asarray(mask, np.uint8), np.zeros(pad, np.uint8)])
    return np.packbits(b, bitorder="little").view(np.uint32)
