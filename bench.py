#!/usr/bin/env python
"""Benchmark of the batched dynamic-update + search hot path on the SIFT-shaped stream.

One step = one pass of the whole path over one batch of synthetic input: insert 10,000 vectors,
delete 10,000 random live ids, search 10,000 queries (k=10) on an index built on 900,000
128-d uint8 vectors (R=64, L=128, alpha=1.2).  Prints ONE JSON line:

  value    update throughput, (inserted + deleted vectors) / time of the insert + delete calls, inputs
           already resident in HBM, timed with CUDA events; whole job over all ranks
  e2e      the same metric through the host-buffer C-ABI calls (host->device copy of ids + vectors and
           the device->host status/result read-back inside the timed region)
  roofline the beam-search kernel: gathered adjacency + vector bytes (in-kernel counters) per second
           against the measured HBM copy bandwidth
  cpu_baseline  the CPU oracle, as it stands, on a bounded shrink of the same stream

`--impl reference` times the oracle alone (it is the reference arm of this build).  With --gpus N
(launched by torchrun) every rank runs an independent replica of the stream: the path has no
exchange step, so there is no data-path collective.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_21163_b200 import synth  # noqa: E402

METRIC = "update_vectors_per_sec"
UNIT = "vectors/s"
WORKLOAD = "sift_u8_d128"
# DRAM bytes moved per beam-search launch divided by the algorithmic bytes of that launch, from the
# single-pass ncu capture at full size summarised in profiles/ (L2 absorbs the rest of the gathers).
NCU_TRAFFIC_RATIO = 0.375


def read_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return json.load(open(p)).get("hbm_gbs", 6650.0), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for nm, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity when not distributed).
    Replicas share nothing on the data path; this reduction of the timers is the only collective."""
    import torch
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


# ------------------------------------------------------------------ oracle arm
def oracle_run(steps, warmup, seed=0, workload=WORKLOAD):
    """The CPU oracle on a bounded shrink of the stream: build 20,000 points (untimed), then steps of
    insert 500 + delete 500 + search 500.  Returns the JSON-ready dict of the reference arm."""
    from oracle import grand_oracle as go
    cfg = dict(synth.CONFIGS[workload])
    per = 500
    cfg.update(n=20_000 + (steps + warmup) * per, build=20_000, first_batch=1_000, max_build_batch=2_000,
               ins=per, dele=per, nq=per, rounds=steps + warmup)
    wl = synth.Workload(cfg, seed)
    st = synth.StreamState(wl)
    o = go.Oracle(cfg["dim"], cfg["dtype"], cfg["metric"], cfg["R"], cfg["L"], cfg["alpha"], wl.capacity(), mode=cfg["mode"])
    t0 = time.perf_counter()
    for ids, rows in st.build_batches():
        o.insert_batch(ids, wl.vectors(*rows))
    t_build = time.perf_counter() - t0
    q = wl.queries()
    t_upd = t_search = 0.0
    for r in range(steps + warmup):
        ids, rows = st.insert_ids()
        v = wl.vectors(*rows)
        dele = None
        t0 = time.perf_counter()
        o.insert_batch(ids, v)
        t1 = time.perf_counter()
        dele = st.delete_ids()
        t2 = time.perf_counter()
        o.delete_batch(dele)
        t3 = time.perf_counter()
        o.search(q, 10, cfg["L"])
        t4 = time.perf_counter()
        st.end_round()
        if r >= warmup:
            t_upd += (t1 - t0) + (t3 - t2)
            t_search += t4 - t3
    value = 2 * per * steps / t_upd
    sample = (f"{workload} shrunk: index built on 20,000 points (untimed, {t_build:.1f} s), then {steps} steps of "
              f"insert {per} + delete {per} + search {per} (k=10, L={cfg['L']})")
    return {"value": value, "unit": UNIT, "cores": o.nthreads, "kind": "oracle", "sample": sample,
            "search_qps": per * steps / t_search, "ms_per_step": 1e3 * (t_upd + t_search) / steps}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=7)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="grand", choices=["grand", "reference"])
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the workload (profiling captures, quick checks)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--workload", default=WORKLOAD, choices=sorted(synth.CONFIGS), help="default: the bench workload; the other "
                    "configs are exploration runs (their lines carry their own workload name)")
    ap.add_argument("--pattern", default="", choices=["", "sliding_window", "interleaved", "expiration_time", "clustered", "insert_heavy"],
                    help="run one of the paper's streaming patterns (Sec. 5.2) on the SIFT-shaped data instead of the step loop")
    ap.add_argument("--hash-bits", type=int, default=0, help="log2 size of the per-query visited cache (0 = library default)")
    ap.add_argument("--visited-set-delete", action="store_true",
                    help="run the delete variant that takes in-neighbours from the visited sets (dangling edges allowed)")
    ap.add_argument("--snapshot-search", action="store_true",
                    help="keep the adjacency twice so that searches may overlap update batches; adds an 'overlap' measurement")
    ap.add_argument("--search-only", type=int, default=0, help="after the build run this many search launches and exit")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    K, W = args.steps, max(args.warmup, 0)

    if args.impl == "reference":
        if rank != 0:
            return 0
        r = oracle_run(K, W, workload=args.workload)
        line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus, "steps": K,
                "warmup": W, "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "int32", "data": "synthetic",
                "config": {"workload": args.workload, "sample": r["sample"]},
                "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
                "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "search_qps": r["search_qps"], "gpu_launches": 0}
        print(json.dumps(line))
        return 0

    import torch
    from paper_2608_21163_b200 import binding as gb
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    torch.backends.cuda.matmul.allow_tf32 = False

    if args.pattern:
        return run_pattern(args, torch, gb, dev)
    cfg = dict(synth.CONFIGS[args.workload])
    is_f32 = cfg["dtype"] == synth.F32
    dist_dtype = torch.float32 if is_f32 else torch.int32
    if args.scale != 1.0:
        cfg = synth.scaled(cfg, args.scale)
    total_steps = W + 2 * K + 1      # device-resident steps, then one untimed and K timed end-to-end steps
    if args.snapshot_search:
        total_steps += K + 1         # and the same steps once more with the searches on a second stream
    cfg["rounds"] = total_steps
    cfg["n"] = cfg["build"] + total_steps * cfg["ins"]
    cfg["reuse_ids"] = False      # fresh ids every step, whatever the config's own id policy
    seed = rank                       # replicas draw independent streams
    wl = synth.Workload(cfg, seed)
    st = synth.StreamState(wl)
    cap = wl.capacity()
    max_batch = max(cfg["first_batch"], cfg["max_build_batch"], cfg["ins"], cfg["dele"])
    g = gb.GrandIndex(cfg["dim"], cfg["dtype"], cfg["metric"], cfg["R"], cfg["L"], cfg["alpha"], capacity=cap,
                      max_batch=max_batch, mode=cfg["mode"], hash_bits=args.hash_bits,
                      visited_set_delete=int(args.visited_set_delete), snapshot_search=int(args.snapshot_search))
    row_bytes = g.row_bytes

    # ---- data: generated on the host, resident on the device before anything is timed
    t0 = time.perf_counter()
    base_host = wl.vectors(0, cfg["n"])
    base = torch.from_numpy(base_host).to(dev)
    queries_host = wl.queries()
    queries = torch.from_numpy(queries_host).to(dev)
    t_gen = time.perf_counter() - t0

    def ids_dev(ids):
        return torch.from_numpy(ids).to(dev)

    # ---- build (untimed set-up of the step loop; its rate is reported as context)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for ids, rows in st.build_batches():
        g.insert_batch(ids_dev(ids), base[rows[0]:rows[0] + rows[1]])
    torch.cuda.synchronize()
    t_build = time.perf_counter() - t0

    if args.search_only:
        out_i = torch.empty((cfg["nq"], 10), dtype=torch.uint32, device=dev)
        out_d = torch.empty((cfg["nq"], 10), dtype=dist_dtype, device=dev)
        for _ in range(args.search_only):
            g.search(queries, 10, cfg["L"], out_i, out_d)
        torch.cuda.synchronize()
        print(json.dumps({"search_only": args.search_only, "build_s": t_build}))
        return 0

    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > L2 (126 MB)
    out_i = torch.empty((cfg["nq"], 10), dtype=torch.uint32, device=dev)
    out_d = torch.empty((cfg["nq"], 10), dtype=dist_dtype, device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def one_step(timed):
        ids, rows = st.insert_ids()
        d_ins = ids_dev(ids)
        vec = base[rows[0]:rows[0] + rows[1]]
        dele = st.delete_ids()
        d_del = ids_dev(dele)
        st.end_round()
        flush.zero_()
        e = [ev() for _ in range(4)]
        torch.cuda.synchronize()
        e[0].record(); g.insert_batch(d_ins, vec)
        e[1].record(); g.delete_batch(d_del)
        e[2].record(); g.search(queries, 10, cfg["L"], out_i, out_d)
        e[3].record()
        torch.cuda.synchronize()
        return (e[0].elapsed_time(e[1]), e[1].elapsed_time(e[2]), e[2].elapsed_time(e[3]), len(ids), len(dele))

    for _ in range(W):
        one_step(False)
    g.reset_stats()
    g.set_profiling(True)
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = g.stats()["kernel_launches"]
    t_ins = t_del = t_srch = 0.0
    n_upd = 0
    for _ in range(K):
        a, b, c, ni, nd = one_step(True)
        t_ins += a; t_del += b; t_srch += c; n_upd += ni + nd
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    stats = g.stats()
    launches = stats["kernel_launches"] - launches0
    g.set_profiling(False)

    # ---- snapshot mode: the step's search on a second stream, overlapping the step's update batches
    overlap = None
    if args.snapshot_search:
        side = torch.cuda.Stream()
        main = torch.cuda.current_stream()
        t_ov = 0.0
        for it in range(K + 1):
            ids, rows = st.insert_ids()
            d_ins = ids_dev(ids)
            vec = base[rows[0]:rows[0] + rows[1]]
            d_del = ids_dev(st.delete_ids())
            st.end_round()
            flush.zero_()
            e0, e1, es = ev(), ev(), ev()
            torch.cuda.synchronize()
            e0.record()
            side.wait_event(e0)
            with torch.cuda.stream(side):
                g.search(queries, 10, cfg["L"], out_i, out_d)     # sees the graph of the previous step
                es.record()
            g.insert_batch(d_ins, vec)
            g.delete_batch(d_del)
            main.wait_event(es)
            e1.record()
            torch.cuda.synchronize()
            if it:
                t_ov += e0.elapsed_time(e1)
        overlap = {"ms_per_step_overlapped": t_ov / K, "ms_per_step_in_sequence": (t_ins + t_del + t_srch) / K,
                   "what": "insert + delete on one stream, the step's search on another (it reads the last published graph)"}

    # ---- end to end: host buffers through the host entry points, copies inside the timed region
    pin = lambda a: torch.from_numpy(a).pin_memory()
    q_pin = pin(queries_host)
    oi_pin = torch.empty((cfg["nq"], 10), dtype=torch.uint32).pin_memory()
    od_pin = torch.empty((cfg["nq"], 10), dtype=dist_dtype).pin_memory()
    t_e2e_upd = t_e2e_all = 0.0
    n_e2e = 0
    h2d = d2h = 0
    for it in range(K + 1):          # the first pass sizes the library's staging buffers and is not timed
        ids, rows = st.insert_ids()
        vec_pin = pin(base_host[rows[0]:rows[0] + rows[1]])
        ids_pin = pin(ids)
        dele = st.delete_ids()
        del_pin = pin(dele)
        st.end_round()
        flush.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        g.insert_batch_host(ids_pin, vec_pin)
        g.delete_batch_host(del_pin)
        t1 = time.perf_counter()
        g.search_host(q_pin, 10, cfg["L"], oi_pin, od_pin)
        t2 = time.perf_counter()
        if it == 0:
            continue
        t_e2e_upd += t1 - t0
        t_e2e_all += t2 - t0
        n_e2e += len(ids) + len(dele)
        h2d = ids_pin.numel() * 4 + vec_pin.numel() * vec_pin.element_size() + del_pin.numel() * 4 + q_pin.numel() * q_pin.element_size()
        d2h = oi_pin.numel() * 4 + od_pin.numel() * 4 + 4 * 104   # results + four status blocks
    torch.cuda.synchronize()

    # ---- max over ranks
    t_upd_ms, t_srch_ms, t_e2e_s = max_over_ranks([t_ins + t_del, t_srch, t_e2e_upd], dist, dev)
    value = world * n_upd / (t_upd_ms * 1e-3)
    e2e_value = world * n_e2e / t_e2e_s
    search_qps = world * cfg["nq"] * K / (t_srch_ms * 1e-3)

    # ---- roofline of the dominant kernel (beam search): gathered bytes / launch time
    peak, peak_kind = read_peaks()
    alg_bytes = stats["expansions"] * (cfg["R"] * 4 + 4) + stats["dist_evals"] * row_bytes
    n_sl = max(stats["n_search_launches"], 1)
    ach = alg_bytes / (stats["ms_search"] * 1e-3) / 1e9 if stats["ms_search"] > 0 else 0.0
    roofline = {"bound": "hbm", "kernel": "beam_search_kernel", "achieved": ach, "peak": peak, "unit": "GB/s",
                "frac": ach / peak, "peak_kind": peak_kind,
                "traffic": (NCU_TRAFFIC_RATIO * alg_bytes / n_sl) if NCU_TRAFFIC_RATIO else None,
                "algorithmic_bytes_per_launch": alg_bytes / n_sl, "launches": n_sl,
                "avg_launch_ms": stats["ms_search"] / n_sl}

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return 0

    extra = {}
    if not args.no_sweep:
        # recall@10 against brute force over the live set, and the smallest L reaching 0.95
        live = np.flatnonzero(st.live)
        truth = brute_topk_gpu(torch, base, torch.from_numpy(live).to(dev), queries, 10, cfg["metric"], is_f32)
        sweep = []
        for L in (10, 16, 24, 32, 48, 64, 96, 128):
            reps = []
            for _ in range(3):
                flush.zero_(); torch.cuda.synchronize()
                a, b = ev(), ev()
                a.record(); g.search(queries, 10, L, out_i, out_d); b.record()
                torch.cuda.synchronize()
                reps.append(a.elapsed_time(b))
            found = out_i.view(torch.int32).to(torch.int64)
            rec = recall_gpu(torch, found, truth)
            sweep.append({"L": L, "recall_at_10": rec, "qps": cfg["nq"] / (min(reps) * 1e-3)})
        ok = [s for s in sweep if s["recall_at_10"] >= 0.95]
        extra["search_sweep"] = sweep
        extra["search_qps_at_recall95"] = ok[0] if ok else None
        extra["recall_at_10_config_L"] = sweep[-1]["recall_at_10"]

    cpu = None
    if not args.no_cpu_baseline:
        r = oracle_run(steps=30, warmup=1, workload=args.workload)
        cpu = {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")}
        cpu["search_qps"] = r["search_qps"]

    ms_per_step = (t_upd_ms + t_srch_ms) / K
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if is_f32 else "int32", "data": "synthetic",
            "config": {"workload": args.workload, "scale": args.scale, "built_on": cfg["build"], "dim": cfg["dim"], "R": cfg["R"],
                       "L": cfg["L"], "alpha": cfg["alpha"], "step": f"insert {cfg['ins']} + delete {cfg['dele']} + search {cfg['nq']} (k=10)",
                       "l2": "index (vectors + adjacency) larger than L2, and a 256 MiB flush between steps",
                       "delete": "visited-set (Alg. 6 as printed)" if args.visited_set_delete else "exact in-neighbours",
                       "parallelism": f"replicas x{world}"},
            "overlap": overlap,
            "search_qps": search_qps,
            "insert_vectors_per_sec": world * (n_upd / 2) / (t_ins * 1e-3), "delete_vectors_per_sec": world * (n_upd / 2) / (t_del * 1e-3),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": 1e3 * t_e2e_all / K},
            "gpu_launches": launches, "clocks": clocks, "roofline": roofline, "cpu_baseline": cpu,
            "phases_ms_per_step": {k[3:]: stats[k] / K for k in stats if k.startswith("ms_")},
            "counters_per_step": {k: stats[k] / K for k in ("expansions", "dist_evals", "pair_dists", "dirty_nodes", "prunes", "requests")},
            "build": {"vectors": cfg["build"], "seconds": t_build, "vectors_per_sec": cfg["build"] / t_build, "datagen_s": t_gen}}
    line.update(extra)
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()
    return 0


def run_pattern(args, torch, gb, dev):
    """One of the streaming patterns of Sec. 5.2 over SIFT-shaped rows (1M x scale), batches of 10k x scale.
    Every op is timed with CUDA events; the first `warmup` ops are excluded."""
    cfg = dict(synth.CONFIGS["sift_u8_d128"])
    n = max(2000, int(round(cfg["n"] * args.scale)))
    batch = max(100, int(round(10_000 * args.scale)))
    wl = synth.Workload(cfg, 0)
    base = torch.from_numpy(wl.vectors(0, n)).to(dev)
    queries = torch.from_numpy(synth.mixture_u8(0, "query", 0, batch, cfg["dim"])).to(dev)
    gens = {
        "sliding_window": lambda: synth.pattern_sliding_window(n, 100, 50, batch),
        "interleaved": lambda: synth.pattern_interleaved(n, batch, n_ops=100),
        "expiration_time": lambda: synth.pattern_expiration(n, batch),
        "clustered": lambda: synth.pattern_clustered(n, batch, synth.mixture_centre_of(0, "base", 0, n) % 64),
        "insert_heavy": lambda: synth.pattern_insert_heavy(n, batch),
    }
    g = gb.GrandIndex(cfg["dim"], cfg["dtype"], cfg["metric"], cfg["R"], cfg["L"], cfg["alpha"], capacity=n, max_batch=batch)
    out_i = torch.empty((batch, 10), dtype=torch.uint32, device=dev)
    out_d = torch.empty((batch, 10), dtype=torch.int32, device=dev)
    t = {"insert": 0.0, "delete": 0.0, "search": 0.0}
    cnt = {"insert": 0, "delete": 0, "search": 0}
    launches0 = None
    nop = 0
    ev = lambda: torch.cuda.Event(enable_timing=True)
    for op in gens[args.pattern]():
        ids = torch.from_numpy(op[1]).to(dev) if len(op) > 1 else None
        a, b = ev(), ev()
        torch.cuda.synchronize()
        a.record()
        if op[0] == "insert":
            g.insert_batch(ids, base[ids.view(torch.int32).long()] if not _contiguous(op[1]) else base[int(op[1][0]):int(op[1][0]) + len(op[1])])
        elif op[0] == "delete":
            g.delete_batch(ids)
        else:
            g.search(queries, 10, cfg["L"], out_i, out_d)
        b.record()
        torch.cuda.synchronize()
        nop += 1
        if nop == args.warmup:
            launches0 = g.stats()["kernel_launches"]
        if nop > args.warmup:
            t[op[0]] += a.elapsed_time(b)
            cnt[op[0]] += len(op[1]) if len(op) > 1 else batch
    upd = cnt["insert"] + cnt["delete"]
    line = {"metric": METRIC, "value": upd / ((t["insert"] + t["delete"]) * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": nop - args.warmup,
            "warmup": args.warmup, "ms_per_step": sum(t.values()) / max(nop - args.warmup, 1), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "config": {"workload": f"sift_u8_d128/{args.pattern}", "rows": n, "batch": batch, "R": cfg["R"], "L": cfg["L"],
                       "step": "one op of the pattern's stream"},
            "insert_vectors_per_sec": cnt["insert"] / (t["insert"] * 1e-3) if t["insert"] else None,
            "delete_vectors_per_sec": cnt["delete"] / (t["delete"] * 1e-3) if t["delete"] else None,
            "search_qps": cnt["search"] / (t["search"] * 1e-3) if t["search"] else None,
            "live_at_end": g.live_count, "gpu_launches": g.stats()["kernel_launches"] - (launches0 or 0)}
    print(json.dumps(line))
    return 0


def _contiguous(ids):
    return len(ids) > 0 and int(ids[-1]) - int(ids[0]) + 1 == len(ids)


def brute_topk_gpu(torch, base, live_ids, queries, k, metric=0, is_f32=False):
    """Ground truth for recall (harness only).  uint8 + squared L2: exact, ties by id.  fp32: fp32 matmul."""
    if is_f32:
        out = []
        x = base[live_ids]
        xn = (x * x).sum(1)
        for lo in range(0, queries.shape[0], 128):
            q = queries[lo:lo + 128]
            d = -(q @ x.T) if metric == 1 else (xn[None, :] - 2 * (q @ x.T))
            out.append(live_ids[torch.topk(d, k, dim=1, largest=False).indices])
        return torch.cat(out)
    x = base[live_ids].to(torch.float32)
    xn = (x * x).sum(1).to(torch.int64)
    out = []
    for lo in range(0, queries.shape[0], 256):
        q = queries[lo:lo + 256].to(torch.float32)
        dot = (q @ x.T).to(torch.int64)                      # exact: |dot| < 2^24
        d = (q * q).sum(1).to(torch.int64)[:, None] + xn[None, :] - 2 * dot
        key = d * (1 << 31) + live_ids[None, :]
        out.append(live_ids[torch.topk(key, k, dim=1, largest=False).indices])
    return torch.cat(out)


def recall_gpu(torch, found, truth):
    hit = (found[:, :, None] == truth[:, None, :]).any(2).sum().item()
    return hit / truth.numel()


if __name__ == "__main__":
    sys.exit(main())
