"""Reader for the hand-worked graph cases under tests/golden/ (the *_cases.txt style files).

A file holds `case <name>` blocks.  Inside a block:
  params key=value ...      dtype (u8|i8|f32), metric (l2|ip), mode (vamana|fixed), R, L, alpha, cap, dim (default 1),
                            and any of P, c, k_repair, vmax
  vectors v0 v1 ...         vectors of ids 0.. (coordinates of one vector joined by commas); starting state
  row <id>: a b c           starting adjacency rows (ids without a row line start empty)
  entry <id>                starting medoid
  insert id:v id:v ...      one insert batch        delete a b ...      one delete batch  (applied in file order)
  expect_row <id>: a b c    expected final row      expect_entry <id>   expected final medoid
Lines starting with # carry the arithmetic and are ignored.  Nothing here computes anything: the expected values
are the ones written in the files.
"""
import os

import numpy as np

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
_DT = {"u8": (0, np.uint8), "i8": (1, np.int8), "f32": (2, np.float32)}
_METRIC = {"l2": 0, "ip": 1}
_MODE = {"vamana": 0, "fixed": 1}


def _vec(tok, np_dtype):
    return np.array([float(x) for x in tok.split(",")]).astype(np_dtype)


def read_cases(filename):
    cases, cur = [], None
    for raw in open(os.path.join(GOLD, filename)):
        line = raw.strip()
        if not line or line.startswith("#"):
            continue
        key, _, rest = line.partition(" ")
        rest = rest.strip()
        if key == "case":
            cur = dict(name=rest, params={}, vectors=None, rows={}, entry=0xFFFFFFFF, ops=[], expect_rows={}, expect_entry=None)
            cases.append(cur)
        elif key == "params":
            cur["params"] = dict(kv.split("=") for kv in rest.split())
        elif key == "vectors":
            cur["vectors"] = rest.split()
        elif key in ("row", "expect_row"):
            v, _, r = rest.partition(":")
            cur["rows" if key == "row" else "expect_rows"][int(v)] = [int(x) for x in r.split()]
        elif key == "entry":
            cur["entry"] = int(rest)
        elif key == "expect_entry":
            cur["expect_entry"] = int(rest)
        elif key == "insert":
            cur["ops"].append(("insert", [(int(t.split(":")[0]), t.split(":")[1]) for t in rest.split()]))
        elif key == "delete":
            cur["ops"].append(("delete", [int(x) for x in rest.split()]))
        else:
            raise ValueError(f"{filename}: unknown line {line!r}")
    out = []
    for c in cases:
        p = c["params"]
        dtype, np_dtype = _DT[p["dtype"]]
        dim, cap, R = int(p.get("dim", 1)), int(p["cap"]), int(p["R"])
        spec = dict(name=c["name"], dim=dim, dtype=dtype, np_dtype=np_dtype, metric=_METRIC[p["metric"]], mode=_MODE[p["mode"]],
                    R=R, L=int(p["L"]), alpha=float(p["alpha"]), cap=cap,
                    opts={k: int(p[k]) for k in ("P", "c", "k_repair", "vmax") if k in p},
                    expect_rows=c["expect_rows"], expect_entry=c["expect_entry"], start=None, ops=[])
        if c["vectors"] is not None:
            vecs = np.zeros((cap, dim), np_dtype)
            for i, tok in enumerate(c["vectors"]):
                vecs[i] = _vec(tok, np_dtype)
            adj = np.full((cap, R), 0xFFFFFFFF, np.uint32)
            deg = np.zeros(cap, np.uint32)
            for v, r in c["rows"].items():
                adj[v, :len(r)] = r
                deg[v] = len(r)
            live = np.zeros(cap, bool)
            live[:len(c["vectors"])] = True
            spec["start"] = dict(vecs=vecs, adj=adj, deg=deg, live=live, entry=c["entry"])
        for kind, arg in c["ops"]:
            if kind == "insert":
                ids = np.array([i for i, _ in arg], np.uint32)
                v = np.stack([_vec(t, np_dtype) for _, t in arg]).reshape(len(arg), dim)
                spec["ops"].append(("insert", ids, v))
            else:
                spec["ops"].append(("delete", np.array(arg, np.uint32), None))
        out.append(spec)
    return out


ALL_FILES = ["fixed_degree_insert_cases.txt", "fixed_degree_delete_cases.txt", "delete_scratch_cap.txt",
             "initial_medoid_rounding.txt"]


def all_cases():
    return [(f, c) for f in ALL_FILES for c in read_cases(f)]
