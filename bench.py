#!/usr/bin/env python
"""Benchmark of the emulated-rank collectives on one B200 (one process per GPU).

A *step* is one one-shot allreduce over 8 emulated ranks of 512 KiB each (batch 32 x
hidden 8192 bf16 per rank, N(0,1), the tensor-parallel decode activation), issued through
the C ABI.  The K timed steps are captured in a CUDA graph (the way a decode step issues
its collectives) that rotates over enough buffer sets to exceed twice the L2 capacity, so
every step reads its sources from HBM ("cold").  Timing is by CUDA events on the launching
stream; with N GPUs each rank runs an independent replica (the emulation has no inter-GPU
step) and the slowest rank's time is used.

Besides the headline the JSON line carries, per message size (8 KiB ... 64 MiB per rank),
the latency and algorithmic HBM throughput of one-shot, two-shot (flag barrier) and
two-shot-put, cold and warm; the 16-rank allgather; the launch floor; the 160-node decode
chain; the oracle timed on the host cores; and an end-to-end number with host buffers.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "allreduce_latency_us"
N_RANKS = 8


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy read+write)"
    return 6650.0, "fallback (earlier measurement on this pool)"


# ---- reference arm: the CPU oracle ----------------------------------------------------------------

def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    from paper_2608_00867_b200 import workloads
    w = workloads.config_decode_activation()
    src = workloads.make(w)
    cores = os.cpu_count() or 1
    for _ in range(max(args.warmup, 1)):
        oracle.allreduce(src, nthreads=cores)
    steps = max(1, min(args.steps, 2000))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.allreduce(src, nthreads=cores)
    dt = time.perf_counter() - t0
    us = dt / steps * 1e6
    line = {
        "impl": "reference", "metric": METRIC, "value": us, "unit": "us", "n_gpus": args.gpus,
        "steps": steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 storage, f32 accumulate", "data": "synthetic",
        "config": {"workload": w.name, "nranks": w.nranks, "bytes_per_rank": w.bytes_per_rank,
                   "algorithm": "oracle (plain C fold, OpenMP over elements)"},
        "cpu_baseline": {"value": us, "unit": "us", "cores": cores, "kind": "oracle",
                         "sample": f"{steps} whole allreduces of the 8 x 512 KiB workload"},
        "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


# ---- GPU arm -----------------------------------------------------------------------------------------

class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed regions run."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.samples = []
        self.proc = None
        self.index = index
        self.marks = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def mark(self, t0, t1):
        self.marks.append((t0, t1))

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        inside, allv, smax, reasons = [], [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.samples:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                mhz, smax = float(parts[0]), float(parts[1])
            except ValueError:
                continue
            allv.append(mhz)
            if any(a - 0.05 <= ts <= b + 0.05 for a, b in self.marks):
                inside.append(mhz)
                for nm, val in zip(names, parts[2:6]):
                    if val.lower().startswith("active"):
                        reasons.add(nm)
        use = inside or allv
        return {"sm_mhz": statistics.median(use) if use else None, "sm_max_mhz": smax,
                "reasons": sorted(reasons), "samples_in_timed_regions": len(inside)}


def run_gpu(args):
    import numpy as np
    import torch
    from paper_2608_00867_b200 import binding as nb
    from paper_2608_00867_b200 import workloads

    from paper_2608_00867_b200.replicas import Replicas
    rep = Replicas(backend="nccl")
    rank, world, local = rep.rank, rep.world, rep.local

    peak_gbs, peak_src = measured_peaks()
    l2 = torch.cuda.get_device_properties(local).L2_cache_size
    num_sms = torch.cuda.get_device_properties(local).multi_processor_count
    nb.nuna_init(128 << 20)
    stream = torch.cuda.Stream()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()

    barrier, max_over_ranks = rep.barrier, rep.max_over_ranks

    def make_sets(n, count, dst_count, min_bytes, dist_name="normal", seed=1, max_sets=4096):
        """Device buffer sets whose total footprint exceeds min_bytes (cold protocol).

        Each emulated rank has its own allocation (one arena for its sources, one for its
        destinations); set s is the s-th slice of every arena, so successive steps touch
        fresh addresses until the rotation wraps."""
        per_set = 2 * n * (count + dst_count)
        nsets = max(2, min(max_sets, -(-min_bytes // per_set)))
        pad = lambda c: -(-c // 128) * 128
        host = workloads.rank_buffers(n, min(count, 1 << 22), dist_name, seed)
        src_arena, dst_arena = [], []
        for r in range(n):
            h = torch.from_numpy(host[r].view(np.int16)).cuda()
            a = torch.empty(nsets * pad(count), dtype=torch.int16, device="cuda")
            reps = -(-a.numel() // h.numel())
            a.copy_(h.repeat(reps)[:a.numel()] if reps > 1 else h[:a.numel()])
            src_arena.append(a)
            dst_arena.append(torch.empty(nsets * pad(dst_count), dtype=torch.int16, device="cuda"))
        sets = []
        for s in range(nsets):
            src = [a[s * pad(count): s * pad(count) + count] for a in src_arena]
            dst = [a[s * pad(dst_count): s * pad(dst_count) + dst_count] for a in dst_arena]
            sets.append((src, dst))
        return sets

    def capture(fn, sets, nodes):
        """A CUDA graph of `nodes` back-to-back calls, call i on buffer set i mod len(sets)."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            fn(*sets[0], stream)                                     # untimed: creates contexts / loads modules
            torch.cuda.synchronize()
            with torch.cuda.graph(g, stream=stream):
                for i in range(nodes):
                    fn(*sets[i % len(sets)], stream)
        return g

    def time_graph(g, replays, warm_replays=1):
        with torch.cuda.stream(stream):
            for _ in range(warm_replays):
                g.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            t0 = time.time()
            e0.record(stream)
            for _ in range(replays):
                g.replay()
            e1.record(stream)
            barrier()
            t1 = time.time()
        sampler.mark(t0, t1)
        return max_over_ranks(e0.elapsed_time(e1))                   # ms, slowest rank

    def per_call_us(fn, sets, nodes, replays):
        g = capture(fn, sets, nodes)
        ms = time_graph(g, replays)
        del g
        return ms * 1e3 / (nodes * replays)

    def per_call_stats(fn, sets, nodes, replays):
        """Each replay of the graph timed on its own (its own event pair): median / min / max per call."""
        g = capture(fn, sets, nodes)
        with torch.cuda.stream(stream):
            g.replay()
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(replays + 1)]
            barrier()
            t0 = time.time()
            evs[0].record(stream)
            for i in range(replays):
                g.replay()
                evs[i + 1].record(stream)
            barrier()
            sampler.mark(t0, time.time())
        per = sorted(max_over_ranks(evs[i].elapsed_time(evs[i + 1])) * 1e3 / nodes for i in range(replays))
        del g
        return {"median": per[len(per) // 2], "min": per[0], "max": per[-1]}

    # ---- headline: K one-shot allreduces on the decode activation ------------------------------------
    w = workloads.config_decode_activation()
    count = w.count
    sets = make_sets(N_RANKS, count, count, 2 * l2 + (64 << 20), "normal", w.seed)
    headline_flags = nb.NUNA_PLACE_AUTO | nb.NUNA_LAUNCH_PDL
    oneshot = lambda s, d, st: nb.nuna_allreduce_oneshot(s, d, count, flags=headline_flags, stream=st)
    K, W = args.steps, max(args.warmup, 3)
    nodes = min(K, 1000)
    replays, rem = divmod(K, nodes)
    launches0 = nb.nuna_launch_count()
    g_main = capture(oneshot, sets, nodes)
    g_rem = capture(oneshot, sets, rem) if rem else None
    g_warm = capture(oneshot, sets, W)
    launches_capture = nb.nuna_launch_count() - launches0
    with torch.cuda.stream(stream):
        g_warm.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0 = time.time()
        e0.record(stream)
        for _ in range(replays):
            g_main.replay()
        if g_rem is not None:
            g_rem.replay()
        e1.record(stream)
        barrier()
        t1 = time.time()
    sampler.mark(t0, t1)
    total_ms = max_over_ranks(e0.elapsed_time(e1))
    us_per_step = total_ms * 1e3 / K
    alg_bytes = 2 * N_RANKS * w.bytes_per_rank                       # every source once + every destination once
    achieved = alg_bytes / (us_per_step * 1e-6) / 1e9
    del g_main, g_rem, g_warm

    # launch floor: the same graph shape with an empty kernel of the same grid
    grid_blocks = min(N_RANKS * -(-(count // 8) // 256), num_sms * 5)
    floor_us = per_call_us(lambda s, d, st: nb.nuna_launch_floor(grid_blocks, stream=st), sets, 1000, 3)
    floor_pdl_us = per_call_us(lambda s, d, st: nb.nuna_launch_floor(grid_blocks, flags=nb.NUNA_LAUNCH_PDL, stream=st), sets, 1000, 3)

    extras = {}
    # ---- placement on the headline workload: round-robin baseline vs the two placement-aware kernels ---------
    # (per-SM work lists use the topology of a probe run here on the first buffer set)
    topo = nb.nuna_probe_topology(list(sets[0][0]) + list(sets[0][1]))
    doms = [topo.sm_domain[s] for s in range(topo.num_sms)]
    extras["probe"] = {
        "sms": topo.num_sms, "sms_reported": topo.sms_reported, "lines": topo.num_lines,
        "verdict": "nonuniform" if topo.verdict == nb.NUNA_TOPO_NONUNIFORM else "uniform",
        "domain_sizes": [doms.count(0), doms.count(1)], "near_cycles": round(topo.near_lat, 1),
        "far_cycles": round(topo.far_lat, 1), "gap_cycles": round(topo.domain_gap, 1), "noise_cycles": round(topo.noise, 2),
        "sm_mean_hit_cycles_min_max": [round(min(topo.sm_lat_hit[:topo.num_sms]), 1), round(max(topo.sm_lat_hit[:topo.num_sms]), 1)],
        "sm_miss_cycles_min_max": [round(min(topo.sm_lat_miss[:topo.num_sms]), 1), round(max(topo.sm_lat_miss[:topo.num_sms]), 1)],
        "hist_first_cycle": nb.NUNA_HIST_FIRST, "hist_step": nb.NUNA_HIST_STEP,
        "hist_near": list(topo.hist_near), "hist_far": list(topo.hist_far),
    }
    place = {}
    for pname, pflags in (("roundrobin", nb.NUNA_PLACE_ROUNDROBIN), ("aware_colocated", nb.NUNA_PLACE_AWARE),
                          ("aware_cluster_dsmem", nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_CLUSTER),
                          ("aware_sm_lists", nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_SM_LISTS)):
        fn = lambda s, d, st, f=pflags: nb.nuna_allreduce_oneshot(s, d, count, flags=f, stream=st)
        place[pname] = {"cold_us": round(per_call_us(fn, sets, 1000, 3), 3),
                        "l2_resident_us": round(per_call_us(fn, sets[:1], 1000, 3), 3)}
    extras["placement_512KiB"] = place

    # ---- robustness to concurrent work (the paper runs its collectives beside a GEMM, Section 6.6) ------------
    # 1 MiB per rank one-shot, L2-resident sources, while a second stream runs (a) nothing, (b) a streaming
    # copy, (c) a dense bf16 matmul (a library GEMM used only as a load generator).
    if not args.quick:
        c1 = (1 << 20) // 2
        isets = make_sets(N_RANKS, c1, c1, 0, "normal", 77, max_sets=2)
        side = torch.cuda.Stream()
        big_a = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        big_b = torch.empty_like(big_a)
        ma = torch.randn(4096, 4096, device="cuda", dtype=torch.bfloat16)
        mb = torch.randn(4096, 4096, device="cuda", dtype=torch.bfloat16)
        loads = {"idle": None, "streaming_copy": lambda: big_b.copy_(big_a), "bf16_gemm_4096": lambda: torch.matmul(ma, mb)}
        inter = {}
        for lname, load in loads.items():
            row = {}
            for pname, pflags in (("roundrobin", nb.NUNA_PLACE_ROUNDROBIN), ("aware_colocated", nb.NUNA_PLACE_AWARE)):
                fn = lambda s, d, st, f=pflags: nb.nuna_allreduce_oneshot(s, d, c1, flags=f, stream=st)
                g = capture(fn, isets, 400)
                with torch.cuda.stream(stream):
                    g.replay()
                torch.cuda.synchronize()
                if load is not None:                       # enqueue the background work, then time beside it
                    with torch.cuda.stream(side):
                        for _ in range(80):
                            load()
                with torch.cuda.stream(stream):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    g.replay()
                    g.replay()
                    e1.record(stream)
                busy = (not side.query()) if load is not None else None   # background still running at the end?
                torch.cuda.synchronize()
                row[pname] = {"us": round(e0.elapsed_time(e1) * 1e3 / 800, 3), "background_outlasted_timing": busy}
                del g
            inter[lname] = row
        extras["interference_1MiB_resident"] = inter

        # ---- sensitivity to the number of thread blocks (the paper contrasts few and many, Section 6.5) ---------
        blocks_rows = {}
        for label, fn_of in (("oneshot_1MiB", lambda: (lambda s, d, st: nb.nuna_allreduce_oneshot(s, d, c1, stream=st))),
                             ("twoshot_put_1MiB", lambda: (lambda s, d, st: nb.nuna_allreduce_twoshot(s, d, c1, flags=nb.NUNA_TWOSHOT_PUT, stream=st)))):
            row = {}
            for blocks in (8, 37, 148, 592, 0):
                nb.nuna_set_option(nb.NUNA_OPT_BLOCKS, blocks)
                row["default" if blocks == 0 else str(blocks)] = round(per_call_us(fn_of(), isets, 200, 2), 3)
            nb.nuna_set_option(nb.NUNA_OPT_BLOCKS, 0)
            blocks_rows[label] = row
        extras["blocks_sensitivity_resident_us"] = blocks_rows
        del isets, big_a, big_b, ma, mb
        torch.cuda.empty_cache()
    if True:
        # ---- end to end through the host-buffer entry point (pinned host memory) -----------------------
        hsrc = [torch.from_numpy(a.view(np.int16).copy()).pin_memory() for a in workloads.make(w)]
        hdst = [torch.empty(count, dtype=torch.int16).pin_memory() for _ in range(N_RANKS)]
        def time_host(**kw):
            for _ in range(3):
                nb.nuna_allreduce_host(hsrc, hdst, count, **kw)
            barrier()
            t0 = time.perf_counter()
            for _ in range(50):
                nb.nuna_allreduce_host(hsrc, hdst, count, **kw)
            return max_over_ranks((time.perf_counter() - t0) / 50 * 1e6)
        # the call a user with host data makes: pinned buffers, the kernel works on them in place
        e2e_us = time_host(flags=nb.NUNA_TWOSHOT_PUT, two_shot=True)
        staged_us = time_host()                                   # one-shot through device staging copies
        extras["e2e"] = {"value": e2e_us, "unit": "us", "h2d_bytes_per_step": N_RANKS * w.bytes_per_rank,
                         "d2h_bytes_per_step": N_RANKS * w.bytes_per_rank,
                         "path": "nuna_allreduce_host, pinned host buffers accessed in place by the two-shot put kernel",
                         "staged_copies_oneshot_us": staged_us}

    sweep, ag_row, a2a_row, rs_rows, chain_rows = [], None, None, [], []
    if not args.quick:
        # ---- message-size sweep, 8 ranks, 8 KiB .. 64 MiB per rank --------------------------------------
        algos = {
            "oneshot": lambda c: (lambda s, d, st: nb.nuna_allreduce_oneshot(s, d, c, stream=st)),
            "oneshot_aware": lambda c: (lambda s, d, st: nb.nuna_allreduce_oneshot(s, d, c, flags=nb.NUNA_PLACE_AWARE, stream=st)),
            "twoshot": lambda c: (lambda s, d, st: nb.nuna_allreduce_twoshot(s, d, c, stream=st)),
            "twoshot_put": lambda c: (lambda s, d, st: nb.nuna_allreduce_twoshot(s, d, c, flags=nb.NUNA_TWOSHOT_PUT, stream=st)),
            # the same two with programmatic dependent launch (the one-shot drops it above 16 MiB of sources)
            "oneshot_pdl": lambda c: (lambda s, d, st: nb.nuna_allreduce_oneshot(s, d, c, flags=nb.NUNA_LAUNCH_PDL, stream=st)),
            "twoshot_put_pdl": lambda c: (lambda s, d, st: nb.nuna_allreduce_twoshot(
                s, d, c, flags=nb.NUNA_TWOSHOT_PUT | nb.NUNA_LAUNCH_PDL, stream=st)),
            # nuna_allreduce: the library picks the algorithm by size
            "size_selected": lambda c: (lambda s, d, st: nb.nuna_allreduce(
                s, d, c, flags=nb.NUNA_TWOSHOT_PUT | nb.NUNA_LAUNCH_PDL | nb.NUNA_PLACE_AUTO, stream=st)),
        }
        for wl in workloads.config_size_sweep(args.sweep_min, args.sweep_max):
            c, B = wl.count, wl.bytes_per_rank
            ssets = make_sets(N_RANKS, c, c, 2 * l2 + (64 << 20), "normal", wl.seed)
            nodes_s = max(len(ssets), min(512, (256 << 20) // B + 1))          # at least one full rotation
            reps = 7 if B <= (4 << 20) else 5
            row = {"bytes_per_rank": B, "buffer_sets": len(ssets), "algorithmic_bytes": 2 * N_RANKS * B,
                   "calls_per_sample": nodes_s, "samples": reps}
            for name, mk in algos.items():
                cs = per_call_stats(mk(c), ssets, nodes_s, reps)
                warm = per_call_stats(mk(c), ssets[:1], nodes_s, reps)["median"]
                cold = cs["median"]
                row[name] = {"cold_us": round(cold, 3), "cold_min_us": round(cs["min"], 3), "cold_max_us": round(cs["max"], 3),
                             "warm_us": round(warm, 3),
                             "cold_gbs": round(2 * N_RANKS * B / cold / 1e3, 1),
                             "cold_frac_of_peak": round(2 * N_RANKS * B / cold / 1e3 / peak_gbs, 4)}
            best = min(algos, key=lambda a: row[a]["cold_us"])
            row["best"] = best
            row["best_frac_of_peak"] = row[best]["cold_frac_of_peak"]
            sweep.append(row)
            del ssets
            torch.cuda.empty_cache()

        # ---- allgather, 16 ranks x 64 KiB ---------------------------------------------------------------
        wa = workloads.config_allgather16()
        asets = make_sets(wa.nranks, wa.count, wa.nranks * wa.count, 2 * l2 + (64 << 20), "uniform", wa.seed)
        ag_us = per_call_us(lambda s, d, st: nb.nuna_allgather(s, d, wa.count, flags=nb.NUNA_LAUNCH_PDL, stream=st), asets, 512, 3)
        ag_bytes = wa.nranks * wa.bytes_per_rank + wa.nranks * wa.nranks * wa.bytes_per_rank
        ag_row = {"workload": wa.name, "us": round(ag_us, 3), "algorithmic_bytes": ag_bytes,
                  "gbs": round(ag_bytes / ag_us / 1e3, 1), "frac_of_peak": round(ag_bytes / ag_us / 1e3 / peak_gbs, 4)}
        del asets
        torch.cuda.empty_cache()

        # ---- reduce-scatter, 8 ranks, 4 MiB and 32 MiB of sources per rank --------------------------------
        rs_rows = []
        for log2b in (22, 25):
            cnt = (1 << log2b) // 2
            shard = cnt // N_RANKS
            rsets = make_sets(N_RANKS, cnt, shard, 2 * l2 + (64 << 20), "normal", 60 + log2b)
            rs_us = per_call_us(lambda s, d, st: nb.nuna_reduce_scatter(s, d, shard, flags=nb.NUNA_LAUNCH_PDL, stream=st),
                                rsets, max(len(rsets), 64), 3)
            rs_bytes = N_RANKS * 2 * cnt + 2 * cnt                     # every source once + every shard once
            rs_rows.append({"bytes_per_rank": 2 * cnt, "us": round(rs_us, 3), "algorithmic_bytes": rs_bytes,
                            "gbs": round(rs_bytes / rs_us / 1e3, 1), "frac_of_peak": round(rs_bytes / rs_us / 1e3 / peak_gbs, 4)})
            del rsets
            torch.cuda.empty_cache()

        # ---- alltoall, 8 ranks x 64 KiB per pair ----------------------------------------------------------
        wt = workloads.config_alltoall8()
        tsets = make_sets(wt.nranks, wt.count, wt.count, 2 * l2 + (64 << 20), "normal", wt.seed)
        blk = wt.count // wt.nranks
        a2a_us = per_call_us(lambda s, d, st: nb.nuna_alltoall(s, d, blk, flags=nb.NUNA_LAUNCH_PDL, stream=st), tsets, 512, 3)
        a2a_bytes = 2 * wt.nranks * wt.bytes_per_rank
        a2a_row = {"workload": wt.name, "us": round(a2a_us, 3), "algorithmic_bytes": a2a_bytes,
                   "gbs": round(a2a_bytes / a2a_us / 1e3, 1), "frac_of_peak": round(a2a_bytes / a2a_us / 1e3 / peak_gbs, 4)}
        del tsets
        torch.cuda.empty_cache()

        # ---- decode-step chain: 160 back-to-back one-shot allreduces in one graph ------------------------
        # Two alternating source sets (attention-out / MLP-out partials), L2-resident as in decode.
        variants = {
            "roundrobin": nb.NUNA_PLACE_ROUNDROBIN,
            "roundrobin_pdl": nb.NUNA_PLACE_ROUNDROBIN | nb.NUNA_LAUNCH_PDL,
            "aware_pdl": nb.NUNA_PLACE_AWARE | nb.NUNA_LAUNCH_PDL,
            "auto_resident_pdl": nb.NUNA_PLACE_AUTO | nb.NUNA_HINT_RESIDENT | nb.NUNA_LAUNCH_PDL,
            "aware_sm_lists_pdl": nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_SM_LISTS | nb.NUNA_LAUNCH_PDL,
        }
        for tokens in workloads.CHAIN_TOKENS:
            wc = workloads.config_decode_chain(tokens)
            csets = make_sets(N_RANKS, wc.count, wc.count, 0, "normal", wc.seed, max_sets=2)
            row = {"tokens": tokens, "bytes_per_rank": wc.bytes_per_rank, "nodes": workloads.CHAIN_NODES}
            for vname, vflags in variants.items():
                chain = nb.nuna_chain_create([c[0] for c in csets], [c[1] for c in csets], workloads.CHAIN_NODES,
                                             wc.count, flags=vflags)
                with torch.cuda.stream(stream):
                    for _ in range(3):
                        nb.nuna_chain_launch(chain, stream=stream)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    barrier()
                    t0 = time.time()
                    e0.record(stream)
                    for _ in range(20):
                        nb.nuna_chain_launch(chain, stream=stream)
                    e1.record(stream)
                    barrier()
                    sampler.mark(t0, time.time())
                ms = max_over_ranks(e0.elapsed_time(e1))
                nb.nuna_chain_destroy(chain)
                row[vname] = {"step_us": round(ms * 1e3 / 20, 2), "per_node_us": round(ms * 1e3 / 20 / workloads.CHAIN_NODES, 3)}
            chain_rows.append(row)
            del csets

    # ---- CPU baseline: the oracle as it stands, on this machine's cores (rank 0 at N = 1 only) -----------------
    cpu = None
    if rank == 0 and world == 1:
        import oracle
        cores = os.cpu_count() or 1
        src = workloads.make(w)
        oracle.allreduce(src, nthreads=cores)
        reps, t0 = 0, time.perf_counter()
        while time.perf_counter() - t0 < 1.5:
            oracle.allreduce(src, nthreads=cores)
            reps += 1
        cpu = {"value": (time.perf_counter() - t0) / reps * 1e6, "unit": "us", "cores": cores, "kind": "oracle",
               "sample": f"{reps} whole allreduces of the 8 x 512 KiB workload (about {1.5 * cores:.0f} core-seconds)"}

    launches_total = nb.nuna_launch_count()
    status = nb.nuna_device_status()
    clocks = sampler.stop() if rank == 0 else None
    rep.close()
    if rank != 0:
        return 0

    # dram__bytes_read.sum + dram__bytes_write.sum of one k_oneshot_rr<8,1> launch on this workload, from the
    # ncu capture summarised in profiles/oneshot_rr_n8_512KiB.md (4.20 MB read, 0 written: the destinations
    # are still dirty in L2 when the kernel ends)
    traffic = 4200192
    line = {
        "metric": METRIC, "value": us_per_step, "unit": "us", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": us_per_step / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 storage, f32 accumulate", "data": "synthetic",
        "config": {"workload": w.name, "nranks": N_RANKS, "bytes_per_rank": w.bytes_per_rank,
                   "algorithm": "one-shot allreduce, placement AUTO, programmatic dependent launch",
                   "launch": "CUDA graph of back-to-back calls",
                   "l2_protocol": f"cold: rotates over {len(sets)} buffer sets ({len(sets) * 2 * N_RANKS * w.bytes_per_rank >> 20} MiB) > 2 x L2",
                   "multi_gpu": "independent replicas (the emulated collective has no inter-GPU step)"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak_gbs, "unit": "GB/s", "frac": achieved / peak_gbs,
                     "traffic": traffic, "peak_source": peak_src,
                     "note": "512 KiB per rank moves 8 MiB: 1.28 us at peak, so this size is latency-bound; "
                             "see sweep[] for the bandwidth-bound sizes",
                     "launch_floor_us": round(floor_us, 3), "launch_floor_pdl_us": round(floor_pdl_us, 3)},
        "gpu_launches": K,
        "launches_since_load": int(launches_total),
        "device_status": status,
        "clocks": clocks,
        "sweep": sweep, "allgather16": ag_row, "alltoall8": a2a_row, "reduce_scatter8": rs_rows, "decode_chain": chain_rows,
    }
    line.update(extras)
    if cpu is not None:
        line["cpu_baseline"] = cpu
    print(json.dumps(line))
    return 0


def run_case(args):
    """A handful of eager launches of one algorithm at one size, each on fresh (cold) buffers."""
    import torch

    from paper_2608_00867_b200 import binding as nb
    parts = args.case.split(":")
    algo, log2b = parts[0], int(parts[1])
    launches = int(parts[2]) if len(parts) > 2 else 4
    n = 16 if algo == "allgather" else N_RANKS
    count = (1 << log2b) // 2
    dst_count = n * count if algo == "allgather" else count
    torch.cuda.set_device(0)
    nb.nuna_init(2 * count)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(log2b)
    nsets = max(2, min(launches, (3 << 30) // (2 * n * (count + dst_count))))
    sets = [([torch.randn(count, generator=gen, device="cuda").to(torch.bfloat16) for _ in range(n)],
             [torch.empty(dst_count, device="cuda", dtype=torch.bfloat16) for _ in range(n)]) for _ in range(nsets)]
    call = {
        "oneshot": lambda s, d: nb.nuna_allreduce_oneshot(s, d, count),
        "oneshot_aware": lambda s, d: nb.nuna_allreduce_oneshot(s, d, count, flags=nb.NUNA_PLACE_AWARE),
        "oneshot_sm": lambda s, d: nb.nuna_allreduce_oneshot(s, d, count, flags=nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_SM_LISTS),
        "twoshot": lambda s, d: nb.nuna_allreduce_twoshot(s, d, count),
        "twoshot_put": lambda s, d: nb.nuna_allreduce_twoshot(s, d, count, flags=nb.NUNA_TWOSHOT_PUT),
        "allgather": lambda s, d: nb.nuna_allgather(s, d, count),
    }[algo]
    torch.cuda.synchronize()
    for i in range(launches):
        call(*sets[i % nsets])
    torch.cuda.synchronize()
    print(json.dumps({"case": args.case, "launches": launches, "buffer_sets": nsets, "status": nb.nuna_device_status()}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="nuna", choices=["nuna", "reference"])
    ap.add_argument("--quick", action="store_true", help="headline only: skip sweep, allgather and chain")
    ap.add_argument("--sweep-min", type=int, default=13)
    ap.add_argument("--sweep-max", type=int, default=26)
    ap.add_argument("--case", default=None,
                    help="ALGO:LOG2BYTES[:LAUNCHES] -- run a few eager launches of one algorithm at one size and "
                         "exit (for ncu captures); ALGO in oneshot, oneshot_aware, oneshot_sm, twoshot, twoshot_put, allgather")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.case:
        return run_case(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
