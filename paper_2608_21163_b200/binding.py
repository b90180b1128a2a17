"""Thin ctypes binding of the C-ABI library (include/grand.h).

Argument marshalling only: every step of the batched insert / delete / search path runs inside
the CUDA library.  torch is used for device memory and streams, nothing else.  There is no CPU
fallback: if the shared library is missing or cannot be loaded this module raises.
"""
import ctypes as C
import os

import torch

from . import build as _build

U8, I8, F32 = 0, 1, 2
L2, IP = 0, 1
VAMANA, FIXED_DEGREE = 0, 1
INVALID = 0xFFFFFFFF
_TORCH_DTYPE = {U8: torch.uint8, I8: torch.int8, F32: torch.float32}

EXPORTS = [
    "grand_create", "grand_create_ex", "grand_destroy", "grand_insert_batch", "grand_delete_batch", "grand_search",
    "grand_insert_batch_host", "grand_delete_batch_host", "grand_search_host", "grand_export_graph",
    "grand_import_graph", "grand_reverse_graph", "grand_reverse_graph_noalloc", "grand_get_entry", "grand_set_entry", "grand_live_count",
    "grand_row_bytes", "grand_get_stats", "grand_reset_stats", "grand_set_profiling", "grand_strerror",
    "grand_last_error",
]


class GrandOptions(C.Structure):
    _fields_ = [("capacity", C.c_uint64), ("max_batch", C.c_uint64), ("P", C.c_uint32), ("c", C.c_uint32),
                ("k_repair", C.c_uint32), ("vmax", C.c_uint32), ("mode", C.c_uint32), ("hash_bits", C.c_uint32),
                ("full_transpose", C.c_uint32), ("mips_max_norm", C.c_float),
                ("visited_set_delete", C.c_uint32), ("max_delete_edges", C.c_uint64), ("snapshot_search", C.c_uint32),
                ("dev_alloc", C.c_void_p), ("dev_free", C.c_void_p), ("user", C.c_void_p)]


class GrandStats(C.Structure):
    _fields_ = [("expansions", C.c_uint64), ("dist_evals", C.c_uint64), ("pair_dists", C.c_uint64),
                ("dirty_nodes", C.c_uint64), ("prunes", C.c_uint64), ("requests", C.c_uint64),
                ("kernel_launches", C.c_uint64), ("rebuild_bytes", C.c_uint64), ("picks_bytes", C.c_uint64),
                ("prune_bytes", C.c_uint64), ("rebuild_prunes", C.c_uint64),
                ("ms_search", C.c_double), ("ms_prune", C.c_double), ("ms_group", C.c_double),
                ("ms_rebuild", C.c_double), ("ms_transpose", C.c_double), ("ms_picks", C.c_double),
                ("ms_other", C.c_double), ("n_search_launches", C.c_uint64), ("n_prune_launches", C.c_uint64),
                ("n_rebuild_launches", C.c_uint64), ("n_picks_launches", C.c_uint64), ("n_transpose_launches", C.c_uint64),
                ("picks_pair_dists", C.c_uint64), ("prune_pair_dists", C.c_uint64)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


_lib = None


def lib_path():
    return _build.LIB


def load():
    """Load the CUDA library built in-tree (build it with paper_2608_21163_b200/build.py)."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run `python -m paper_2608_21163_b200.build` (needs nvcc); "
                               "there is no fallback path")
        _lib = C.CDLL(path)
        _lib.grand_strerror.restype = C.c_char_p
        _lib.grand_last_error.restype = C.c_char_p
        _lib.grand_last_error.argtypes = [C.c_void_p]
    return _lib


class GrandError(RuntimeError):
    def __init__(self, code, msg=""):
        super().__init__(f"grand error {code}: {msg}")
        self.code = code


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dp(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


NOALLOC_MAX_NODES = 1 << 20


def reverse_graph_noalloc(adj, deg, off_out, src_out):
    """CSR reverse graph of a caller-supplied adjacency array without any device allocation inside
    the library (grand_reverse_graph_noalloc).  For callers whose memory plan is frozen: adj [n x R]
    and deg [n] are device inputs, off_out [n + 1] and src_out (or None) device outputs that the
    caller allocated beforehand.  Calls on one device share a fixed scratch array inside the
    library and must not overlap.  Returns the number of edges."""
    lib = load()
    n, R = adj.shape
    E = C.c_uint64()
    rc = lib.grand_reverse_graph_noalloc(_dp(adj), _dp(deg), C.c_uint64(n), C.c_uint32(R), _dp(off_out), _dp(src_out),
                                         C.c_uint64(src_out.numel() if src_out is not None else 0), C.byref(E), _stream())
    if rc != 0:
        raise GrandError(rc, lib.grand_strerror(rc).decode())
    return E.value


class GrandIndex:
    """One index on the current CUDA device.  Methods mirror the C entry points one to one."""

    def __init__(self, dim, dtype, metric, R, L, alpha, capacity=0, max_batch=0, P=0, c=0, k_repair=0, vmax=0,
                 mode=VAMANA, hash_bits=0, full_transpose=0, mips_max_norm=0.0, visited_set_delete=0,
                 snapshot_search=0, max_delete_edges=0, dev_alloc=None, dev_free=None):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (no CPU fallback)")
        self.lib = load()
        self.dim, self.dtype, self.metric, self.R, self.L = dim, dtype, metric, R, L
        self.torch_dtype = _TORCH_DTYPE[dtype]
        self.dist_dtype = torch.float32 if dtype == F32 else torch.int32
        o = GrandOptions(capacity=capacity, max_batch=max_batch, P=P, c=c, k_repair=k_repair, vmax=vmax, mode=mode,
                         hash_bits=hash_bits, full_transpose=full_transpose, mips_max_norm=mips_max_norm,
                         visited_set_delete=visited_set_delete, snapshot_search=snapshot_search,
                         max_delete_edges=max_delete_edges)
        # optional allocator hooks: ctypes callbacks (void* (size_t, void*) / void (void*, void*)); kept alive here
        self._hooks = (dev_alloc, dev_free)
        if dev_alloc is not None:
            o.dev_alloc = C.cast(dev_alloc, C.c_void_p)
            o.dev_free = C.cast(dev_free, C.c_void_p)
        h = C.c_void_p()
        rc = self.lib.grand_create_ex(C.c_uint32(dim), C.c_uint32(dtype), C.c_uint32(metric), C.c_uint32(R),
                                      C.c_uint32(L), C.c_float(alpha), C.byref(o), C.byref(h))
        if rc != 0:
            raise GrandError(rc, self.lib.grand_strerror(rc).decode())
        self.h = h
        self.capacity = capacity if capacity else 1 << 20
        self.device = torch.device("cuda", torch.cuda.current_device())

    def close(self):
        if getattr(self, "h", None):
            self.lib.grand_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc):
        if rc != 0:
            raise GrandError(rc, self.lib.grand_last_error(self.h).decode() or self.lib.grand_strerror(rc).decode())

    def _ids(self, ids):
        ids = torch.as_tensor(ids)
        if ids.dtype != torch.uint32:
            ids = ids.to(torch.int64).to(torch.uint32) if ids.dtype != torch.int32 else ids.view(torch.uint32)
        return ids.contiguous()

    # ---- device-buffer calls
    def insert_batch(self, ids, vecs):
        ids = self._ids(ids).to(self.device)
        vecs = vecs.to(self.device, self.torch_dtype).contiguous()
        assert vecs.shape == (ids.numel(), self.dim)
        self._check(self.lib.grand_insert_batch(self.h, _dp(ids), _dp(vecs), C.c_uint64(ids.numel()), _stream()))

    def delete_batch(self, ids):
        ids = self._ids(ids).to(self.device)
        self._check(self.lib.grand_delete_batch(self.h, _dp(ids), C.c_uint64(ids.numel()), _stream()))

    def search(self, queries, k, L, out_ids=None, out_dists=None):
        q = queries.to(self.device, self.torch_dtype).contiguous()
        nq = q.shape[0]
        if out_ids is None:
            out_ids = torch.empty((nq, k), dtype=torch.uint32, device=self.device)
        if out_dists is None:
            out_dists = torch.empty((nq, k), dtype=self.dist_dtype, device=self.device)
        self._check(self.lib.grand_search(self.h, _dp(q), C.c_uint64(nq), C.c_uint32(k), C.c_uint32(L), _dp(out_ids),
                                          _dp(out_dists), _stream()))
        return out_ids, out_dists

    # ---- host-buffer calls (copies happen inside the library call)
    def insert_batch_host(self, ids, vecs):
        assert ids.device.type == "cpu" and vecs.device.type == "cpu" and ids.dtype == torch.uint32
        self._check(self.lib.grand_insert_batch_host(self.h, _dp(ids), _dp(vecs), C.c_uint64(ids.numel()), _stream()))

    def delete_batch_host(self, ids):
        assert ids.device.type == "cpu" and ids.dtype == torch.uint32
        self._check(self.lib.grand_delete_batch_host(self.h, _dp(ids), C.c_uint64(ids.numel()), _stream()))

    def search_host(self, queries, k, L, out_ids, out_dists):
        assert queries.device.type == "cpu" and out_ids.device.type == "cpu"
        self._check(self.lib.grand_search_host(self.h, _dp(queries), C.c_uint64(queries.shape[0]), C.c_uint32(k),
                                               C.c_uint32(L), _dp(out_ids), _dp(out_dists), _stream()))
        return out_ids, out_dists

    # ---- introspection
    def export_graph(self):
        adj = torch.empty((self.capacity, self.R), dtype=torch.uint32, device=self.device)
        deg = torch.empty(self.capacity, dtype=torch.uint32, device=self.device)
        live = torch.empty((self.capacity + 31) // 32, dtype=torch.uint32, device=self.device)
        e = C.c_uint32()
        self._check(self.lib.grand_export_graph(self.h, _dp(adj), _dp(deg), _dp(live), C.byref(e), _stream()))
        torch.cuda.current_stream().synchronize()
        return adj, deg, live, e.value

    def import_graph(self, adj, deg, live_bitmap, entry, vecs):
        adj = adj.to(self.device).contiguous(); deg = deg.to(self.device).contiguous()
        live = live_bitmap.to(self.device).contiguous()
        vecs = vecs.to(self.device, self.torch_dtype).contiguous()
        assert vecs.shape == (self.capacity, self.dim) and adj.numel() == self.capacity * self.R
        self._check(self.lib.grand_import_graph(self.h, _dp(adj), _dp(deg), _dp(live), C.c_uint32(entry), _dp(vecs),
                                                _stream()))

    def reverse_graph(self):
        off = torch.empty(self.capacity + 1, dtype=torch.uint32, device=self.device)
        E = C.c_uint64()
        self._check(self.lib.grand_reverse_graph(self.h, _dp(off), C.c_void_p(0), C.byref(E), _stream()))
        src = torch.empty(max(E.value, 1), dtype=torch.uint32, device=self.device)
        self._check(self.lib.grand_reverse_graph(self.h, _dp(off), _dp(src), C.byref(E), _stream()))
        return off, src[:E.value]

    @property
    def entry(self):
        e = C.c_uint32()
        self._check(self.lib.grand_get_entry(self.h, C.byref(e)))
        return e.value

    @entry.setter
    def entry(self, e):
        self._check(self.lib.grand_set_entry(self.h, C.c_uint32(e)))

    @property
    def live_count(self):
        n = C.c_uint64()
        self._check(self.lib.grand_live_count(self.h, C.byref(n)))
        return n.value

    @property
    def row_bytes(self):
        n = C.c_uint32()
        self._check(self.lib.grand_row_bytes(self.h, C.byref(n)))
        return n.value

    def stats(self):
        s = GrandStats()
        self._check(self.lib.grand_get_stats(self.h, C.byref(s)))
        return s.as_dict()

    def reset_stats(self):
        self._check(self.lib.grand_reset_stats(self.h))

    def set_profiling(self, on):
        self._check(self.lib.grand_set_profiling(self.h, C.c_int(int(on))))
