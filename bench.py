#!/usr/bin/env python
"""Benchmark of the batched dynamic-update + search hot path.

One step = one pass of the whole path over one batch of synthetic input: insert a batch, delete a batch, search a
batch of queries (k=10) on a built index.  The headline workload is the Deep-shaped sliding window (10M x 96 fp32,
window 8M, steps of insert 100k newest + delete 100k oldest + search 10k; R=64, L=128, alpha=1.2): the largest
configuration by vectors and edges, and the one that runs the complete Vamana path (search, RobustPrune, reverse
graph, consolidated repair).  The other full-size configurations follow under `per_config` with the same fields.
Prints ONE JSON line:

  value     update throughput, (inserted + deleted vectors) / time of the insert + delete calls, inputs already
            resident in HBM, CUDA-event timed, the library's phase events OFF; whole job over all ranks
  e2e       the same metric through the host-buffer C-ABI calls (host->device copy of ids + vectors and the
            device->host status/result read-back inside the timed region)
  roofline  the dominant kernel (beam search): gathered adjacency + vector bytes (in-kernel counters) per second of
            kernel time against the measured HBM copy bandwidth; `rooflines` has one entry per kernel of the path
            (kernel times come from separate steps with the phase events ON, counters from those same steps)
  cpu_baseline  the CPU oracle, as it stands, on a bounded shrink of the same stream, plus the tiny config at full
            size; `sampled_parity` runs the oracle's search on the graph the GPU built, at full size

`--impl reference` times the oracle alone (it is the reference arm of this build).  With --gpus N (launched by
torchrun) every rank runs an independent replica of the stream: the path has no exchange step, so there is no
data-path collective.
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
WORKLOAD = "deep_f32_d96"
PER_CONFIG = ["sift_u8_d128", "gist_f32_d960", "embed_f32_d768_ip", "deep_f32_d96_isotropic"]
SWEEP_L = (10, 16, 24, 32, 48, 64, 96, 128, 192, 256, 384, 512)
# DRAM bytes of one beam-search launch divided by the launch's algorithmic bytes, from one-pass ncu captures
# (dram__bytes_read.sum + dram__bytes_write.sum); each ratio is valid for its workload at the named scale only.
NCU_TRAFFIC = {
    ("deep_f32_d96", 1.0): (0.945, "profiles/beam_search_dram_deep_f32_d96_full.txt"),
    ("sift_u8_d128", 1.0): (0.379, "profiles/beam_search_dram_sift_u8_d128_full.txt"),
    ("gist_f32_d960", 1.0): (0.680, "profiles/beam_search_dram_gist_f32_d960_full.txt"),
    ("embed_f32_d768_ip", 1.0): (0.971, "profiles/beam_search_dram_embed_f32_d768_ip_full.txt"),
    ("deep_f32_d96_isotropic", 1.0): (0.961, "profiles/beam_search_dram_deep_f32_d96_isotropic_full.txt"),
}


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
ORACLE_BUILD = 20_000
ORACLE_BATCH = 500


def oracle_run(steps, warmup, seed=0, workload=WORKLOAD, nthreads=0):
    """The CPU oracle on a bounded shrink of the stream: build 20,000 points (untimed), then steps of
    insert 500 + delete 500 + search 500.  Returns the JSON-ready dict of the reference arm."""
    from oracle import grand_oracle as go
    full = synth.CONFIGS[workload]
    cfg = dict(full)
    per = ORACLE_BATCH
    cfg.update(n=ORACLE_BUILD + (steps + warmup) * per, build=ORACLE_BUILD, first_batch=1_000, max_build_batch=2_000,
               ins=per, dele=per, nq=per, rounds=steps + warmup, reuse_ids=False)
    wl = synth.Workload(cfg, seed)
    st = synth.StreamState(wl)
    o = go.Oracle(cfg["dim"], cfg["dtype"], cfg["metric"], cfg["R"], cfg["L"], cfg["alpha"], wl.capacity(), mode=cfg["mode"],
                  nthreads=nthreads)
    t0 = time.perf_counter()
    for ids, rows in st.build_batches():
        o.insert_batch(ids, wl.vectors(*rows))
    t_build = time.perf_counter() - t0
    q = wl.queries()
    t_upd = t_search = 0.0
    for r in range(steps + warmup):
        ids, rows = st.insert_ids()
        v = wl.vectors(*rows)
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
    sample = (f"{workload} shrunk: index built on {ORACLE_BUILD:,} points (untimed, {t_build:.1f} s) instead of {full['build']:,}, "
              f"then {steps} steps of insert {per} + delete {per} + search {per} (k=10, L={cfg['L']})")
    return {"value": value, "unit": UNIT, "cores": o.nthreads, "kind": "oracle", "sample": sample,
            "index_size_ratio": full["build"] / ORACLE_BUILD, "search_qps": per * steps / t_search,
            "ms_per_step": 1e3 * (t_upd + t_search) / steps}


def oracle_tiny_full(nthreads):
    """The tiny config (10,000 x 32 uint8) at full size through the oracle: 8 x 1,000 build, +2,000, -1,000, 1,000 queries."""
    from oracle import grand_oracle as go
    cfg = synth.CONFIGS["tiny_u8_d32"]
    wl = synth.Workload(cfg, 0)
    st = synth.StreamState(wl)
    o = go.Oracle(cfg["dim"], cfg["dtype"], cfg["metric"], cfg["R"], cfg["L"], cfg["alpha"], wl.capacity(), nthreads=nthreads)
    t0 = time.perf_counter()
    for ids, rows in st.build_batches():
        o.insert_batch(ids, wl.vectors(*rows))
    t1 = time.perf_counter()
    ids, rows = st.insert_ids()
    v = wl.vectors(*rows)
    t2 = time.perf_counter()
    o.insert_batch(ids, v)
    t3 = time.perf_counter()
    dele = st.delete_ids()
    t4 = time.perf_counter()
    o.delete_batch(dele)
    t5 = time.perf_counter()
    q = wl.queries()
    t6 = time.perf_counter()
    o.search(q, 10, cfg["L"])
    t7 = time.perf_counter()
    return {"threads": o.nthreads, "build_vectors_per_sec": cfg["build"] / (t1 - t0),
            "update_vectors_per_sec": (len(ids) + len(dele)) / ((t3 - t2) + (t5 - t4)), "search_qps": len(q) / (t7 - t6)}


def sampled_parity(torch, g, cfg, base_host, queries_host, is_f32, nsample=200):
    """The oracle's own search (with a complete visited set) on the graph the GPU built, at the bench's full size, for
    a sample of the queries: its answers against the GPU's for the same queries, and the distances it evaluates per
    search (every node once) against the GPU's count (its bounded visited cache may forget and evaluate twice)."""
    from oracle import grand_oracle as go
    t0 = time.perf_counter()
    adj, deg, live, entry = g.export_graph()
    cap = g.capacity
    o = go.Oracle(cfg["dim"], cfg["dtype"], cfg["metric"], cfg["R"], cfg["L"], cfg["alpha"], cap, mode=cfg["mode"])
    o.import_graph(adj.cpu().numpy(), deg.cpu().numpy(), live.cpu().numpy(), entry, base_host[:cap])
    del adj, deg, live
    q = queries_host[:nsample]
    s0 = g.stats()
    gi, gd = g.search(torch.from_numpy(q), 10, cfg["L"])
    torch.cuda.synchronize()
    s1 = g.stats()
    gi, gd = gi.cpu().numpy(), gd.cpu().numpy()
    oi, od = o.search(q, 10, cfg["L"], use_seen_set=True)
    so = o.stats()
    out = {"queries": len(q), "index_nodes_live": int(g.live_count), "seconds": None,
           "gpu_evals_per_search": (s1["dist_evals"] - s0["dist_evals"]) / len(q),
           "unique_evals_per_search": so["dist_evals"] / len(q),
           "gpu_expansions_per_search": (s1["expansions"] - s0["expansions"]) / len(q),
           "oracle_expansions_per_search": so["expansions"] / len(q)}
    out["reevaluated_share"] = 1.0 - out["unique_evals_per_search"] / max(out["gpu_evals_per_search"], 1.0)
    if is_f32:
        out["mean_result_overlap"] = float(np.mean([len(set(a.tolist()) & set(b.tolist())) / 10 for a, b in zip(oi, gi)]))
        rel = 0.0
        for i in range(len(q)):
            ok = gi[i] != 0xFFFFFFFF
            b = base_host[gi[i][ok]].astype(np.float64)
            qq = q[i].astype(np.float64)
            if cfg["metric"] == synth.L2:
                exact = ((b - qq) ** 2).sum(1)
                scale = np.abs(exact)
            else:
                exact = -(b @ qq)
                scale = np.linalg.norm(b, axis=1) * np.linalg.norm(qq)
            rel = max(rel, float((np.abs(gd[i][ok] - exact) / np.maximum(scale, 1e-30)).max()))
        out["max_relative_distance_error"] = rel
        out["ok"] = bool(rel <= 1e-5 and out["mean_result_overlap"] > 0.95)
    else:
        out["ids_identical"] = bool((oi == gi).all())
        out["distances_identical"] = bool((od == gd.astype(np.float64)).all())
        out["ok"] = out["ids_identical"] and out["distances_identical"]
    out["seconds"] = time.perf_counter() - t0
    return out


# ------------------------------------------------------------------ one workload on the GPU
def run_workload(args, torch, gb, dev, dist, rank, world, name, scale, K, W, Kp, headline):
    local_rank = dev.index
    cfg = dict(synth.CONFIGS[name])
    is_f32 = cfg["dtype"] == synth.F32
    dist_dtype = torch.float32 if is_f32 else torch.int32
    if scale != 1.0:
        cfg = synth.scaled(cfg, scale)
    total_steps = W + K + Kp + K + 1     # warm-up, timed, profiled, then one untimed and K timed end-to-end steps
    if args.snapshot_search:
        total_steps += K + 1             # and the same steps once more with the searches on a second stream
    cfg["rounds"] = total_steps
    cfg["n"] = cfg["build"] + total_steps * cfg["ins"]
    cfg["reuse_ids"] = False             # fresh ids every step, whatever the config's own id policy
    cfg["delete_first"] = False
    seed = rank                          # replicas draw independent streams
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
        return {"search_only": args.search_only, "build_s": t_build}

    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > L2 (126 MB)
    out_i = torch.empty((cfg["nq"], 10), dtype=torch.uint32, device=dev)
    out_d = torch.empty((cfg["nq"], 10), dtype=dist_dtype, device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def one_step():
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
        one_step()
    g.reset_stats()
    g.set_profiling(False)
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
        a, b, c, ni, nd = one_step()
        t_ins += a; t_del += b; t_srch += c; n_upd += ni + nd
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    stats_timed = g.stats()
    launches = stats_timed["kernel_launches"] - launches0

    # ---- kernel times: separate steps with the library's phase events on (the events and the synchronising search
    #      they bring would otherwise sit inside `value`)
    g.reset_stats()
    g.set_profiling(True)
    if args.cuda_profiler_range:
        torch.cuda.profiler.start()      # `ncu --profile-from-start off` then sees exactly these steps
    for _ in range(Kp):
        one_step()
    torch.cuda.synchronize()
    if args.cuda_profiler_range:
        torch.cuda.profiler.stop()
    stats = g.stats()
    g.set_profiling(False)
    live_edges = int(g.export_graph()[1].view(torch.int32).to(torch.int64).sum().item())

    # ---- snapshot mode: the step's search on a second stream, overlapping the step's update batches
    overlap = None
    if args.snapshot_search:
        side = torch.cuda.Stream()
        main_s = torch.cuda.current_stream()
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
            main_s.wait_event(es)
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
    for it in range(K + 1):          # the first pass sizes the search call's staging buffers and is not timed
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
        d2h = oi_pin.numel() * 4 + od_pin.numel() * 4 + 4 * 176   # results + four status blocks
    torch.cuda.synchronize()

    # ---- max over ranks
    t_upd_ms, t_srch_ms, t_e2e_s = max_over_ranks([t_ins + t_del, t_srch, t_e2e_upd], dist, dev)
    value = world * n_upd / (t_upd_ms * 1e-3)
    e2e_value = world * n_e2e / t_e2e_s
    search_qps = world * cfg["nq"] * K / (t_srch_ms * 1e-3)

    # ---- rooflines: algorithmic bytes (counted in the kernels) per second of kernel time (phase events of the
    #      profiled steps, on the launching stream) against the measured HBM copy bandwidth
    peak, peak_kind = read_peaks()

    # fp32 FFMA peak for the kernels that are dense blocks of pair distances rather than gathers: SMs x 128 lanes x 2 flop
    # x the maximum SM clock.  A squared-L2 term is a subtract and a fused multiply-add (3 flop in 2 issue slots), so
    # 0.75 of this figure is the most such a kernel can show.
    props = torch.cuda.get_device_properties(dev)
    fp32_peak = props.multi_processor_count * 128 * 2 * 1.965e9 / 1e12

    def roof(kernel, nbytes, ms, launches_, what, pairs=None):
        if not launches_ or ms <= 0:
            return None
        ach = nbytes / (ms * 1e-3) / 1e9
        r = {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
             "peak_kind": peak_kind, "traffic": None, "algorithmic_bytes_per_launch": nbytes / launches_,
             "launches": launches_, "avg_launch_ms": ms / launches_, "bytes_counted": what}
        if pairs:
            r["pair_distances_per_sec"] = pairs / (ms * 1e-3)
            if is_f32:
                tf = 3.0 * cfg["dim"] * pairs / (ms * 1e-3) / 1e12
                r["alu"] = {"bound": "alu", "achieved": tf, "peak": fp32_peak, "unit": "TFLOP/s", "frac": tf / fp32_peak,
                            "flops_counted": "3 x dim per pair distance (subtract, multiply, add)",
                            "peak_kind": "nominal: SMs x 128 fp32 lanes x 2 x 1.965 GHz"}
        return r

    search_bytes = stats["expansions"] * (cfg["R"] * 4 + 4) + stats["dist_evals"] * row_bytes
    rooflines = {
        "beam_search": roof("beam_search_kernel", search_bytes, stats["ms_search"], stats["n_search_launches"],
                            "expansions x (R x 4 + 4) adjacency bytes + evaluated nodes x padded row bytes"),
        "rebuild": roof("rebuild_kernel", stats["rebuild_bytes"], stats["ms_rebuild"], stats["n_rebuild_launches"],
                        "per rebuilt row: row read + write (2 x R x 4), request tuples (12 each), and one vector per candidate when a prune runs"),
        "delete_picks": roof("delete_picks_*_kernel", stats["picks_bytes"], stats["ms_picks"], stats["n_picks_launches"],
                             "one vector per (deleted node, surviving in-/out-neighbour) pair + the repair candidates' vectors per deleted node",
                             pairs=stats["picks_pair_dists"]),
        "forward_prune": roof("forward_prune_*_kernel", stats["prune_bytes"], stats["ms_prune"], stats["n_prune_launches"],
                              "one vector per candidate the prune looks at", pairs=stats["prune_pair_dists"]),
        "reverse_graph": roof("transpose_hist_pairs/scatter_pairs_kernel", stats["n_transpose_launches"] * (cap * 4 + live_edges * 4),
                              stats["ms_transpose"], stats["n_transpose_launches"],
                              "one pass over the degrees and the live adjacency entries (the scan, and the list and scatter of the batch's rows, not counted)"),
    }
    tr = NCU_TRAFFIC.get((name, float(scale)))
    if tr and rooflines["beam_search"]:
        rooflines["beam_search"]["traffic"] = tr[0] * rooflines["beam_search"]["algorithmic_bytes_per_launch"]
        rooflines["beam_search"]["traffic_source"] = f"{tr[0]} x algorithmic bytes, ratio from {tr[1]}"

    if rank != 0:
        g.close()
        return None

    extra = {}
    if not args.no_sweep:
        # recall@10 against brute force over the live set, and the smallest L reaching 0.95
        live = np.flatnonzero(st.live)
        truth = brute_topk_gpu(torch, base, torch.from_numpy(live).to(dev), queries, 10, cfg["metric"], is_f32)
        sweep = []
        for L in SWEEP_L:
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
        best = max(sweep, key=lambda s: s["recall_at_10"])
        extra["search_sweep"] = sweep
        extra["search_qps_at_recall95"] = dict(ok[0], reached=True) if ok else \
            {"reached": False, "best_recall_at_10": best["recall_at_10"], "L": best["L"], "qps": best["qps"]}
        extra["recall_at_10_config_L"] = [s for s in sweep if s["L"] == cfg["L"]][0]["recall_at_10"]
        del truth

    if not args.no_cpu_baseline:
        sp = sampled_parity(torch, g, cfg, base_host, queries_host, is_f32)
        extra["sampled_parity"] = sp
        bs = rooflines["beam_search"]
        if bs:
            bs["achieved_on_unique_rows"] = bs["achieved"] * (1.0 - max(sp["reevaluated_share"], 0.0))

    ms_per_step = (t_upd_ms + t_srch_ms) / K
    res = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
           "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "f32" if is_f32 else "int32", "data": "synthetic",
           "config": {"workload": name, "scale": scale, "built_on": cfg["build"], "dim": cfg["dim"], "R": cfg["R"],
                      "L": cfg["L"], "alpha": cfg["alpha"], "mode": "fixed-degree" if cfg["mode"] else "vamana",
                      "metric": "ip" if cfg["metric"] else "l2",
                      "generator": {"name": cfg["gen"], **cfg.get("gen_args", {})},
                      "step": f"insert {cfg['ins']} + delete {cfg['dele']} + search {cfg['nq']} (k=10)",
                      "l2": "index (vectors + adjacency) larger than L2, and a 256 MiB flush between steps",
                      "delete": "visited-set (Alg. 6 as printed)" if args.visited_set_delete else "exact in-neighbours",
                      "kernel_times": f"from {Kp} further steps with the library's phase events on; `value` is timed with them off",
                      "parallelism": f"replicas x{world}"},
           "overlap": overlap,
           "search_qps": search_qps,
           "insert_vectors_per_sec": world * (n_upd / 2) / (t_ins * 1e-3), "delete_vectors_per_sec": world * (n_upd / 2) / (t_del * 1e-3),
           "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                   "ms_per_step": 1e3 * t_e2e_all / K},
           "gpu_launches": launches, "clocks": clocks, "roofline": rooflines["beam_search"], "rooflines": rooflines,
           "phases_ms_per_step": {k[3:]: stats[k] / Kp for k in stats if k.startswith("ms_")},
           "counters_per_step": {k: stats_timed[k] / K for k in ("expansions", "dist_evals", "pair_dists", "dirty_nodes", "prunes",
                                                                 "rebuild_prunes", "requests", "rebuild_bytes", "picks_bytes", "prune_bytes")},
           "build": {"vectors": cfg["build"], "seconds": t_build, "vectors_per_sec": cfg["build"] / t_build, "datagen_s": t_gen}}
    if not headline:
        for k in ("n_gpus", "higher_is_better", "scaling", "vs_baseline", "data", "overlap"):
            res.pop(k)
    res.update(extra)
    g.close()
    del g, base, queries, flush
    torch.cuda.empty_cache()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=7)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="grand", choices=["grand", "reference"])
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the workload (profiling captures, quick checks)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="run the headline workload only")
    ap.add_argument("--profiled-steps", type=int, default=3, help="extra steps with the phase events on (kernel times)")
    ap.add_argument("--workload", default=WORKLOAD, choices=sorted(synth.CONFIGS), help="headline workload of the line")
    ap.add_argument("--pattern", default="", choices=["", "sliding_window", "interleaved", "expiration_time", "clustered", "insert_heavy"],
                    help="run one of the paper's streaming patterns (Sec. 5.2) on the SIFT-shaped data instead of the step loop")
    ap.add_argument("--hash-bits", type=int, default=0, help="log2 size of the per-query visited cache (0 = library default)")
    ap.add_argument("--visited-set-delete", action="store_true",
                    help="run the delete variant that takes in-neighbours from the visited sets (dangling edges allowed)")
    ap.add_argument("--snapshot-search", action="store_true",
                    help="keep the adjacency twice so that searches may overlap update batches; adds an 'overlap' measurement")
    ap.add_argument("--search-only", type=int, default=0, help="after the build run this many search launches and exit")
    ap.add_argument("--cuda-profiler-range", action="store_true",
                    help="bracket the profiled steps with cudaProfilerStart/Stop (for captures limited to those steps)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    K, W = max(args.steps, 1), max(args.warmup, 0)

    if args.impl == "reference":
        if rank != 0:
            return 0
        r = oracle_run(K, W, workload=args.workload)
        is_f32 = synth.CONFIGS[args.workload]["dtype"] == synth.F32
        line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus, "steps": K,
                "warmup": W, "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f64" if is_f32 else "int64", "data": "synthetic",
                "config": {"workload": args.workload, "sample": r["sample"], "index_size_ratio": r["index_size_ratio"]},
                "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample", "index_size_ratio")},
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

    line = run_workload(args, torch, gb, dev, dist, rank, world, args.workload, args.scale, K, W, max(args.profiled_steps, 1), True)
    if args.search_only:
        print(json.dumps(line))
        return 0
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return 0

    # ---- the other full-size configurations, same fields, a short run each (one GPU, rank 0 of a single-rank job)
    if world == 1 and not args.no_per_config and args.scale == 1.0:
        per = {}
        for name in PER_CONFIG:
            if name == args.workload:
                continue
            per[name] = run_workload(args, torch, gb, dev, None, 0, 1, name, 1.0, 3, 3, 2, False)
        line["per_config"] = per

    # ---- the oracle on the host cores (rank 0, one-GPU runs only): a bounded shrink of the headline stream, and the
    #      tiny config at full size with all threads and with one
    line["cpu_baseline"] = None
    if world == 1 and not args.no_cpu_baseline:
        r = oracle_run(steps=6, warmup=1, workload=args.workload)
        cpu = {k: r[k] for k in ("value", "unit", "cores", "kind", "sample", "index_size_ratio", "search_qps")}
        cpu["tiny_u8_d32_full_size"] = [oracle_tiny_full(0), oracle_tiny_full(1)]
        line["cpu_baseline"] = cpu
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
    """Ground truth for recall (harness only).  uint8 + squared L2: exact, ties by id.  fp32: fp32 matmul over
    column blocks of the live set (bounded memory), candidates merged per block."""
    nq = queries.shape[0]
    if is_f32:
        best_d = torch.full((nq, k), float("inf"), device=base.device)
        best_i = torch.zeros((nq, k), dtype=torch.int64, device=base.device)
        step = 1 << 20
        for lo in range(0, live_ids.numel(), step):
            ids = live_ids[lo:lo + step]
            x = base[ids]
            xn = (x * x).sum(1)
            for qlo in range(0, nq, 512):
                q = queries[qlo:qlo + 512]
                d = -(q @ x.T) if metric == 1 else (xn[None, :] - 2 * (q @ x.T))
                dd, ii = torch.topk(d, min(k, d.shape[1]), dim=1, largest=False)
                cat_d = torch.cat([best_d[qlo:qlo + 512], dd], 1)
                cat_i = torch.cat([best_i[qlo:qlo + 512], ids[ii]], 1)
                sel = torch.topk(cat_d, k, dim=1, largest=False).indices
                best_d[qlo:qlo + 512] = torch.gather(cat_d, 1, sel)
                best_i[qlo:qlo + 512] = torch.gather(cat_i, 1, sel)
        return best_i
    x = base[live_ids].to(torch.float32)
    xn = (x * x).sum(1).to(torch.int64)
    out = []
    for lo in range(0, nq, 256):
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
