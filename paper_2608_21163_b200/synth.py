"""Seeded synthetic inputs shaped like the paper's streaming workloads (Table 1, Sec. 5.2).

Every value is a pure function of (seed, stream, row, column) through a counter-based hash, so
any slice of any array can be regenerated anywhere (host test, oracle run, GPU benchmark) without
carrying state.  This module holds input generation only: none of the method's arithmetic
(distances, searches, pruning) lives here, which is why both the CUDA path's callers and the CPU
oracle's callers may use it.

The real datasets (SIFT, Deep, GIST-like, text-embedding sets) are not available offline; these
generators borrow only their shapes, dtypes, metrics and value distributions.
"""
import os
import zlib
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_CHUNK = 1 << 20


def _stream_id(stream):
    return np.uint64(zlib.crc32(stream.encode()) & 0xFFFFFFFF)


def _mix(x):
    """splitmix64 finaliser on a uint64 array (wrap-around arithmetic)."""
    x = (x + np.uint64(0x9E3779B97F4A7C15))
    x = (x ^ (x >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
    x = (x ^ (x >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return x ^ (x >> np.uint64(31))


def hash_u64(seed, stream, counters):
    """64 hashed bits per counter for the (seed, stream) pair."""
    with np.errstate(over="ignore"):
        base = _mix(np.asarray([np.uint64(seed) * np.uint64(0x632BE59BD9B4E019) ^ _stream_id(stream)], np.uint64))[0]
        return _mix(_mix(np.asarray(counters, np.uint64) ^ base))


def _counters(start, n, dim):
    rows = np.arange(start, start + n, dtype=np.uint64)[:, None]
    cols = np.arange(dim, dtype=np.uint64)[None, :]
    return rows * np.uint64(dim) + cols


def _rowwise(fn, start, n, dim, dtype):
    """Fill an [n, dim] array chunk by chunk; chunks are independent, so large requests fan out
    over a few threads (numpy releases the GIL inside its loops)."""
    out = np.empty((n, dim), dtype)
    step = max(1, _CHUNK // dim)
    spans = [(lo, min(n, lo + step)) for lo in range(0, n, step)]

    def work(span):
        lo, hi = span
        out[lo:hi] = fn(start + lo, hi - lo)

    if len(spans) <= 2:
        for sp in spans:
            work(sp)
    else:
        with ThreadPoolExecutor(max_workers=min(16, len(os.sched_getaffinity(0)))) as ex:
            list(ex.map(work, spans))
    return out


def _normal(seed, stream, start, n, dim):
    """Standard normals by Box-Muller in double: one hash -> (u1, u2) -> one deviate."""
    h = hash_u64(seed, stream, _counters(start, n, dim))
    u1 = ((h >> np.uint64(32)).astype(np.float64) + 1.0) / 4294967296.0  # (0, 1]
    u2 = (h & np.uint64(0xFFFFFFFF)).astype(np.float64) / 4294967296.0   # [0, 1)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def uniform_u8(seed, stream, start, n, dim):
    """Coordinates uniform in [0, 255]."""
    return _rowwise(lambda s, m: (hash_u64(seed, stream, _counters(s, m, dim)) >> np.uint64(56)).astype(np.uint8),
                    start, n, dim, np.uint8)


def mixture_u8(seed, stream, start, n, dim, n_centres=1000, sigma=20.0):
    """SIFT-shaped bytes: Gaussian mixture, centre coordinates uniform in [0,255], clamp to [0,255]."""
    centres = uniform_u8(seed, "mixture-centres", 0, n_centres, dim).astype(np.float64)

    def gen(s, m):
        which = hash_u64(seed, stream + "/centre", np.arange(s, s + m, dtype=np.uint64)) % np.uint64(n_centres)
        x = centres[which.astype(np.int64)] + sigma * _normal(seed, stream, s, m, dim)
        return np.clip(np.rint(x), 0, 255).astype(np.uint8)

    return _rowwise(gen, start, n, dim, np.uint8)


def gaussian_unit_f32(seed, stream, start, n, dim):
    """Deep-shaped floats: isotropic Gaussian, unit-normalised."""
    def gen(s, m):
        x = _normal(seed, stream, s, m, dim)
        x /= np.linalg.norm(x, axis=1, keepdims=True)
        return x.astype(np.float32)

    return _rowwise(gen, start, n, dim, np.float32)


def halfnormal_f32(seed, stream, start, n, dim, scale=0.1):
    """GIST-shaped floats: |N(0,1)| * scale per coordinate."""
    return _rowwise(lambda s, m: (np.abs(_normal(seed, stream, s, m, dim)) * scale).astype(np.float32),
                    start, n, dim, np.float32)


def aniso_unit_f32(seed, stream, start, n, dim):
    """Embedding-shaped floats: coordinate i ~ N(0, 1/(1+i)), unit-normalised."""
    sd = 1.0 / np.sqrt(1.0 + np.arange(dim, dtype=np.float64))

    def gen(s, m):
        x = _normal(seed, stream, s, m, dim) * sd[None, :]
        x /= np.linalg.norm(x, axis=1, keepdims=True)
        return x.astype(np.float32)

    return _rowwise(gen, start, n, dim, np.float32)


def _manifold(seed, stream, start, n, dim, latent, n_centres, spread, noise):
    """Rows near a `latent`-dimensional linear image of a Gaussian mixture, plus isotropic noise:
    descriptor and embedding sets have an intrinsic dimension far below their coordinate count,
    and it is that, not the coordinate count, which decides how a proximity graph behaves.
    The linear map and the mixture centres depend on (seed, dim, latent) only, so base vectors
    and queries come from the same distribution.  Sums run in a fixed order (no BLAS)."""
    tag = f"manifold/{dim}/{latent}"
    W = _normal(seed, tag + "/map", 0, latent, dim) / np.sqrt(float(latent))
    C = _normal(seed, tag + "/centres", 0, n_centres, latent)
    which = (hash_u64(seed, stream + "/centre", np.arange(start, start + n, dtype=np.uint64)) % np.uint64(n_centres)).astype(np.int64)
    z = C[which] + spread * _normal(seed, stream + "/latent", start, n, latent)
    x = noise * _normal(seed, stream, start, n, dim)
    for k in range(latent):
        x += z[:, k:k + 1] * W[k][None, :]
    return x


def manifold_unit_f32(seed, stream, start, n, dim, latent=32, spread=1.0, noise=0.5, n_centres=4096):
    """Deep- and embedding-shaped floats: a `latent`-dimensional mixture mapped into `dim`
    coordinates, isotropic noise on top, unit-normalised."""
    def gen(s, m):
        x = _manifold(seed, stream, s, m, dim, latent, n_centres, spread, noise)
        x /= np.linalg.norm(x, axis=1, keepdims=True)
        return x.astype(np.float32)

    return _rowwise(gen, start, n, dim, np.float32)


def manifold_abs_f32(seed, stream, start, n, dim, latent=48, spread=1.0, noise=0.2, n_centres=4096, scale=0.1):
    """GIST-shaped floats: non-negative coordinates, |mixture image + noise| * scale."""
    return _rowwise(lambda s, m: (np.abs(_manifold(seed, stream, s, m, dim, latent, n_centres, spread, noise)) * scale).astype(np.float32),
                    start, n, dim, np.float32)


def choose_ids(seed, stream, population, k):
    """k ids drawn uniformly without replacement from `population` (a uint32 array): the k ids with
    the smallest hash, returned in hash order."""
    population = np.asarray(population, np.uint32)
    h = hash_u64(seed, stream, population.astype(np.uint64))
    order = np.lexsort((population, h))[:k]
    return population[order].copy()


GENERATORS = {
    "uniform_u8": uniform_u8,
    "mixture_u8": mixture_u8,
    "gaussian_unit_f32": gaussian_unit_f32,
    "halfnormal_f32": halfnormal_f32,
    "aniso_unit_f32": aniso_unit_f32,
    "manifold_unit_f32": manifold_unit_f32,
    "manifold_abs_f32": manifold_abs_f32,
}

# dtype / metric / mode codes match include/grand.h
U8, I8, F32 = 0, 1, 2
L2, IP = 0, 1
VAMANA, FIXED_DEGREE = 0, 1

# The workload shapes.  n = vectors generated, build = size of the initial index, rounds of
# (insert, delete) batch sizes, nq queries.  `scale` shrinks n/build/batches/queries together for
# parity tests and CPU timing.
CONFIGS = {
    "tiny_u8_d32": dict(gen="uniform_u8", dim=32, dtype=U8, metric=L2, mode=VAMANA, R=32, L=64, alpha=1.2,
                        n=10_000, build=8_000, first_batch=1_000, max_build_batch=1_000,
                        rounds=1, ins=2_000, dele=1_000, nq=1_000, reuse_ids=False),
    "sift_u8_d128": dict(gen="mixture_u8", dim=128, dtype=U8, metric=L2, mode=VAMANA, R=64, L=128, alpha=1.2,
                         n=1_000_000, build=900_000, first_batch=1_000, max_build_batch=10_000,
                         rounds=10, ins=10_000, dele=10_000, nq=10_000, reuse_ids=False),
    "deep_f32_d96": dict(gen="manifold_unit_f32", gen_args=dict(latent=32, spread=1.0, noise=0.5),
                         dim=96, dtype=F32, metric=L2, mode=VAMANA, R=64, L=128, alpha=1.2,
                         n=10_000_000, build=8_000_000, first_batch=1_000, max_build_batch=100_000,
                         rounds=20, ins=100_000, dele=100_000, nq=10_000, reuse_ids=False, delete_oldest=True),
    "gist_f32_d960": dict(gen="manifold_abs_f32", gen_args=dict(latent=48, spread=1.0, noise=0.2),
                          dim=960, dtype=F32, metric=L2, mode=VAMANA, R=64, L=128, alpha=1.2,
                          n=1_200_000, build=1_000_000, first_batch=1_000, max_build_batch=20_000,
                          rounds=10, ins=20_000, dele=50_000, nq=1_000, reuse_ids=True, delete_first=True),
    "embed_f32_d768_ip": dict(gen="manifold_unit_f32", gen_args=dict(latent=48, spread=1.0, noise=0.3),
                              dim=768, dtype=F32, metric=IP, mode=FIXED_DEGREE, R=64, L=128,
                              alpha=1.2, n=5_500_000, build=5_000_000, first_batch=1_000, max_build_batch=50_000,
                              rounds=10, ins=50_000, dele=50_000, nq=10_000, reuse_ids=False),
}
# Stress case: the Deep-shaped sizes on isotropic Gaussian directions, whose intrinsic dimension
# equals the coordinate count.  No descriptor set looks like this (a proximity graph barely helps:
# recall@10 stays near 0.1 at L = 128), but every search expands into rows it has never seen and
# every reverse edge forces a full prune, which makes it the heaviest load per inserted vector.
CONFIGS["deep_f32_d96_isotropic"] = dict(CONFIGS["deep_f32_d96"], gen="gaussian_unit_f32", gen_args={})


def scaled(cfg, factor):
    """Shrink a config's sizes by `factor` (shapes, dims and parameters unchanged)."""
    c = dict(cfg)
    for k in ("n", "build", "max_build_batch", "ins", "dele", "nq"):
        c[k] = max(1, int(round(cfg[k] * factor)))
    c["first_batch"] = min(cfg["first_batch"], c["build"])
    return c


def build_schedule(cfg):
    """Batch sizes that build the initial index: the first batch, then doubling up to the
    config's batch size (a batch cannot link to its own members, so it should not exceed the
    current graph size)."""
    sizes, done, b = [], 0, cfg["first_batch"]
    while done < cfg["build"]:
        b = min(b, cfg["build"] - done)
        sizes.append(b)
        done += b
        b = min(cfg["max_build_batch"], max(b, done))
    return sizes


class Workload:
    """Generates vectors, queries and the op stream for one config."""

    def __init__(self, cfg, seed=0):
        self.cfg, self.seed = cfg, seed
        self.gen = GENERATORS[cfg["gen"]]
        self.gen_args = cfg.get("gen_args", {})

    def vectors(self, start, n):
        return self.gen(self.seed, "base", start, n, self.cfg["dim"], **self.gen_args)

    def queries(self):
        return self.gen(self.seed, "query", 0, self.cfg["nq"], self.cfg["dim"], **self.gen_args)

    def capacity(self):
        c = self.cfg
        return c["build"] if c["reuse_ids"] else c["n"]


class StreamState:
    """Tracks the live id set and produces each round's insert and delete id batches."""

    def __init__(self, wl):
        self.wl = wl
        c = wl.cfg
        self.live = np.zeros(wl.capacity(), bool)
        self.next_row = 0        # next vector row to generate
        self.round = 0
        self.order = []          # insertion order, for delete-oldest streams

    def build_batches(self):
        c = self.wl.cfg
        for b in build_schedule(c):
            ids = np.arange(self.next_row, self.next_row + b, dtype=np.uint32)
            rows = (self.next_row, b)
            self.next_row += b
            self.live[ids] = True
            yield ids, rows

    def delete_ids(self):
        c = self.wl.cfg
        live_ids = np.flatnonzero(self.live).astype(np.uint32)
        k = min(c["dele"], len(live_ids))
        if c.get("delete_oldest"):
            ids = live_ids[:k].copy()          # ids are assigned in arrival order and never reused
        else:
            ids = choose_ids(self.wl.seed, f"del/{self.round}", live_ids, k)
        self.live[ids] = False
        return ids

    def insert_ids(self):
        c = self.wl.cfg
        b = c["ins"]
        if c["reuse_ids"]:
            free = np.flatnonzero(~self.live).astype(np.uint32)
            ids = free[:b].copy()              # smallest freed ids first
            b = len(ids)
        else:
            b = min(b, self.wl.capacity() - self.next_row)
            ids = np.arange(self.next_row, self.next_row + b, dtype=np.uint32)
        rows = (self.next_row, b)
        self.next_row += b
        self.live[ids] = True
        return ids, rows

    def end_round(self):
        self.round += 1


# ---------------------------------------------------------------------------------------------
# Streaming patterns of Sec. 5.2.  Each generator yields ops over a base array of `n_rows` vectors
# that the caller generates with Workload.vectors(0, n_rows); ids equal row numbers (no id reuse):
#   ("insert", ids)   ids: uint32 array      ("delete", ids)      ("search",)
# Sizes are parameters so that the same pattern runs as a shrunk parity case and as a benchmark.
def mixture_centre_of(seed, stream, start, n, n_centres=1000):
    """Mixture centre index of rows [start, start+n) of mixture_u8 (same draw as the generator)."""
    return (hash_u64(seed, stream + "/centre", np.arange(start, start + n, dtype=np.uint64)) % np.uint64(n_centres)).astype(np.int64)


def _chunks(ids, batch):
    for lo in range(0, len(ids), batch):
        yield ids[lo:lo + batch]


def pattern_sliding_window(n_rows, segments=100, active=50, batch=1000):
    """Sliding Window: the rows are cut into `segments`; `active` of them are live; each step inserts the
    next segment, deletes the oldest and searches."""
    seg = n_rows // segments
    ids = np.arange(n_rows, dtype=np.uint32)
    for s in range(active):
        for b in _chunks(ids[s * seg:(s + 1) * seg], batch):
            yield ("insert", b)
    for s in range(active, segments):
        for b in _chunks(ids[s * seg:(s + 1) * seg], batch):
            yield ("insert", b)
        for b in _chunks(ids[(s - active) * seg:(s - active + 1) * seg], batch):
            yield ("delete", b)
        yield ("search",)


def pattern_interleaved(n_rows, batch, seed=0, build_frac=0.3, n_ops=60):
    """Interleaved: after an initial build, a random sequence of 50% insert / 30% search / 20% delete
    batches (deletes draw uniformly from the live set)."""
    ids = np.arange(n_rows, dtype=np.uint32)
    nxt = int(n_rows * build_frac) // batch * batch
    for b in _chunks(ids[:nxt], batch):
        yield ("insert", b)
    live = np.zeros(n_rows, bool)
    live[:nxt] = True
    draw = hash_u64(seed, "interleaved/op", np.arange(n_ops, dtype=np.uint64)) % np.uint64(10)
    for k in range(n_ops):
        r = int(draw[k])
        if r < 5 and nxt + batch <= n_rows:
            b = ids[nxt:nxt + batch]
            nxt += batch
            live[b] = True
            yield ("insert", b)
        elif r < 8:
            yield ("search",)
        else:
            lv = np.flatnonzero(live).astype(np.uint32)
            if len(lv) > 2 * batch:
                d = choose_ids(seed, f"interleaved/del/{k}", lv, batch)
                live[d] = False
                yield ("delete", d)


def pattern_expiration(n_rows, batch, seed=0):
    """Expiration Time: every cycle inserts one batch with a lifetime of 10, 100 or unlimited cycles drawn
    in the ratio 10:2:1, deletes the batches that expire, then searches."""
    ids = np.arange(n_rows, dtype=np.uint32)
    n_cycles = n_rows // batch
    draw = hash_u64(seed, "expiration/life", np.arange(n_cycles, dtype=np.uint64)) % np.uint64(13)
    expiry = {}
    for cyc in range(n_cycles):
        b = ids[cyc * batch:(cyc + 1) * batch]
        yield ("insert", b)
        r = int(draw[cyc])
        life = 10 if r < 10 else (100 if r < 12 else None)
        if life is not None:
            expiry.setdefault(cyc + life, []).append(b)
        for d in expiry.pop(cyc, []):
            yield ("delete", d)
        if cyc % 4 == 3:
            yield ("search",)


def pattern_clustered(n_rows, batch, cluster_of, clusters=64, window=32):
    """Clustered: rows are grouped into `clusters` (here: by mixture centre); a window of `window` clusters is
    live; each step inserts the next cluster, deletes the oldest one and searches (deletes hit one region of
    the graph, which maximises the overlap of dirty sets)."""
    groups = [np.flatnonzero(cluster_of[:n_rows] == c).astype(np.uint32) for c in range(clusters)]
    for c in range(clusters):
        for b in _chunks(groups[c], batch):
            yield ("insert", b)
        if c >= window:
            for b in _chunks(groups[c - window], batch):
                yield ("delete", b)
            yield ("search",)


def pattern_insert_heavy(n_rows, batch):
    """Insert Heavy: 90% insert batches, 10% searches, no deletes."""
    ids = np.arange(n_rows, dtype=np.uint32)
    for k, b in enumerate(_chunks(ids, batch)):
        yield ("insert", b)
        if k % 9 == 8:
            yield ("search",)
