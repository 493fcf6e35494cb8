#!/usr/bin/env python
"""Benchmark of the incremental-propagation hot path.

A step is one pass of the whole path over one batch of B synthetic updates: normalise the batch,
update the graph store, build the per-layer frontiers, scatter the delta messages, re-apply the
layer update to the affected rows.  Default workload: the dense graph (2 449 029 vertices,
123 718 280 edges, 100 features), 2-layer GraphSAGE-mean 100-256-47, B = 1000.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--batch B]
    python bench.py --impl reference ...     # the CPU oracle on the same workload (host cores)

Prints one JSON line (rank 0).  With N > 1 (under torchrun) every rank runs an independent replica
of the workload on its own GPU with its own update stream; there is no data-path collective.
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

from paper_2601_12347_b200 import inputs as I  # noqa: E402

# DRAM traffic of the dominant kernels, measured with ncu at FULL size on the dense graph (one-pass
# captures of dram__bytes_read.sum + dram__bytes_write.sum; profiles/dram_traffic_dense_full_size_ncu.txt):
#   last-hop push scatter of dense-2l (k_scatter_push_packed<12>, rows of 48 floats), three launches of
#   18.6 M - 20.6 M messages: 79.4 - 79.9 bytes per message;
#   rebuilding gather of dense-3l's last hop (k_regather + k_spmm_hubs, rows of 48 floats, 122 M in-edges):
#   6.47 GB per pass = 53 bytes per in-edge.
# A launch's traffic is the per-unit figure times the units it processed: same graph, same kernel, same
# row width, so traffic grows in proportion to the messages (resp. in-edges).
NCU_DRAM_BYTES_PER_MESSAGE = {("dense", 48): 79.6}
NCU_DRAM_BYTES_PER_IN_EDGE = {("dense", 48): 53.0}
METRIC = "updates_per_sec"
UNIT = "updates/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples clocks and throttle reasons while the timed region runs: nvidia-smi every 100 ms, and, because the
    default region is a few tens of milliseconds long, the same counters read through NVML every 2 ms (reads only)."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []
        self.nvml = []          # (sm MHz, max sm MHz, throttle-reason bits)
        self.running = False

    def _poll_nvml(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            idx = int(visible.split(",")[self.gpu]) if visible and visible.split(",")[self.gpu].isdigit() else self.gpu
            h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            mx = pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM)
            while self.running:
                self.nvml.append((pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM), mx,
                                  pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)))
                time.sleep(0.002)
        except Exception:
            pass

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None
        self.running = True
        self.t2 = threading.Thread(target=self._poll_nvml, daemon=True)
        self.t2.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        self.running = False
        if self.proc is None and not self.nvml:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        if self.proc is None:
            self.lines = []
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                pass
        sm, mx, reasons = [], [], set()
        # NVML reason bits: 0x8 hw slowdown, 0x40 hw thermal slowdown, 0x20 sw thermal slowdown, 0x4 sw power cap
        for clk, cmax, bits in self.nvml:
            sm.append(float(clk)); mx.append(float(cmax))
            for name, bit in (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
                              ("sw_power_cap", 0x4)):
                if bits & bit:
                    reasons.add(name)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def pct(xs, p):
    xs = sorted(xs)
    if not xs:
        return None
    k = max(0, min(len(xs) - 1, int(np.ceil(p / 100.0 * len(xs))) - 1))
    return xs[k]


def scatter_bytes(stats, l, ld):
    """Algorithmic bytes of hop l's scatter in the form that ran (fp32, row width ld floats).
    push: each sender row read once, its out-list read once, one read + one write of an aggregate
    row per message.  pull: in-lists of the affected sinks, one delta row per message, one read +
    one write of each affected aggregate row."""
    e = stats["active_edges"][l] - (stats["n_added"] + stats["n_deleted"])
    if stats["scatter_pull"][l]:
        # in-list entry + position-map entry per in-edge of an affected sink; every sender's delta
        # row once (it is re-read from L2 after that); read + write of each affected aggregate row
        return stats["in_edges"][l] * 8 + stats["senders"][l - 1] * 4 * ld + stats["affected"][l] * 8 * ld
    return stats["senders"][l - 1] * (4 * ld + 8) + 4 * e + e * 8 * ld


def max_over_ranks(values_ms, world, device="cuda"):
    """Every rank's timings replaced by the maximum over ranks (the job is as slow as its slowest
    replica).  No-op for one rank."""
    if world <= 1:
        return list(values_ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values_ms), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_rate(world, batch, steps, ms):
    """Updates per second of the whole job: every replica processed batch * steps updates."""
    return world * batch * steps / (ms / 1e3)


def make_workload(name, seed):
    w = I.workloads()[name]
    w.seed = seed
    src, dst = I.make_graph(w)
    X = I.features(w.n, w.model.dims[0], w.seed)
    W = I.make_weights(w.model, w.seed)
    # workloads whose edges carry stored weights: one weight per initial edge, one per operation of a batch
    w.edge_w = I.edge_weights(src.size, w.seed) if w.extra.get("edge_weights") else None
    return w, src, dst, X, W


def draw_batch(stream, w, b):
    """(ups, rows, op_weights or None) of the next batch of the workload's stream"""
    if w.edge_w is not None:
        return stream.next_batch_weighted(b)
    ups, rows = stream.next_batch(b)
    return ups, rows, None


def run_reference(args, rank, world):
    """The CPU oracle (incremental route) on the same workload; one step = one batch."""
    if rank != 0:
        return
    from oracle import oracle as O
    O.build()
    w, src, dst, X, W = make_workload(args.workload, args.seed)
    orc = O.Oracle(w.n, src, dst, X, w.model, W, edge_weights=w.edge_w)
    stream = I.make_stream(w, src, dst)
    lat = []
    # a step is one batch; if full batches would take the run beyond a few minutes, every step after
    # the first applies a bounded sample of its batch instead (the first n_sample updates)
    n_sample, budget_s = args.batch, 150.0
    for s in range(args.warmup + args.steps):
        ups, rows, ow = draw_batch(stream, w, args.batch)
        if n_sample < args.batch:
            ups = ups[:n_sample]
            ow = ow[:n_sample] if ow is not None else None
        t0 = time.perf_counter()
        assert orc.apply_incremental(ups, rows, pull=True, op_weights=ow) == 0
        dt = time.perf_counter() - t0
        if s == 0 and dt * (args.warmup + args.steps) > budget_s:
            n_sample = max(1, int(args.batch * budget_s / (dt * (args.warmup + args.steps))))
        if s >= max(args.warmup, 1 if n_sample < args.batch else 0):
            lat.append(dt)
    total = sum(lat)
    value = n_sample * len(lat) / total
    cores = O.num_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(lat),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": f"{args.workload}, batch {args.batch}", "batch": args.batch,
                   "vertices": w.n, "edges": w.e, "dims": w.model.dims},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{len(lat)} steps of {n_sample} updates (of batches of {args.batch}), incremental route, "
                                   "messages gathered per affected sink on all cores"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "latency_ms": {"p50": 1e3 * pct(lat, 50), "p99": 1e3 * pct(lat, 99)},
    }
    print(json.dumps(line), flush=True)


def cpu_baseline(args, w, src, dst, X, W, budget_s=16.0):
    """The oracle as it stands, timed on the host cores on a bounded sample of the workload: the
    incremental route with its messages gathered per affected sink on all cores (the faster of its two
    delivery orders), and, on a shorter sample, with its messages pushed by one thread."""
    from oracle import oracle as O
    O.build()
    t0 = time.perf_counter()
    orc = O.Oracle(w.n, src, dst, X, w.model, W, edge_weights=w.edge_w)
    setup = time.perf_counter() - t0
    stream = I.make_stream(w, src, dst)
    out = {}
    for pull, budget in ((True, budget_s), (False, budget_s / 2)):
        spent, nb = 0.0, 0
        while spent < budget and nb < 50:
            ups, rows, ow = draw_batch(stream, w, args.batch)
            t0 = time.perf_counter()
            assert orc.apply_incremental(ups, rows, pull=pull, op_weights=ow) == 0
            spent += time.perf_counter() - t0
            nb += 1
        out[pull] = (args.batch * nb / spent, nb, spent)
    orc.close()
    return {"value": out[True][0], "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
            "sample": f"incremental route, messages gathered per affected sink on all cores: first {out[True][1]} batches of "
                      f"{args.batch} updates of the same stream ({out[True][2]:.1f} s); oracle set-up incl. its own "
                      f"bootstrap {setup:.0f} s, untimed",
            "single_thread_scatter": {"value": out[False][0], "unit": UNIT,
                                      "sample": f"the next {out[False][1]} batches with the messages pushed along the "
                                                f"senders' out-lists by one thread ({out[False][2]:.1f} s)"}}


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    from paper_2601_12347_b200 import build as B
    from paper_2601_12347_b200 import ripple
    B.build_library()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    seed = args.seed + rank
    w, src, dst, X, W = make_workload(args.workload, seed)
    L = len(w.model.layers)
    rp = ripple.Ripple(w.n, src, dst, X, w.model, W, timing=True, max_batch=max(args.batch, 16),
                       scatter_mode=args.scatter, edge_weights=w.edge_w)
    bootstrap_ms = rp.stats()["ms_bootstrap"]
    stream = I.make_stream(w, src, dst, seed)
    K, Wm = args.steps, args.warmup
    batches = [draw_batch(stream, w, args.batch) for _ in range(Wm + 2 * K)]

    def to_dev(ups, rows, ow):
        u = torch.from_numpy(np.stack([ups["op"], ups["u"], ups["v"]], axis=1).astype(np.int32)).cuda()
        return u, torch.from_numpy(rows).cuda(), (torch.from_numpy(ow).cuda() if ow is not None else None)

    def to_pinned(ups, rows, ow):
        u = torch.from_numpy(np.stack([ups["op"], ups["u"], ups["v"]], axis=1).astype(np.int32)).pin_memory()
        return u, torch.from_numpy(rows).pin_memory(), (torch.from_numpy(ow).pin_memory() if ow is not None else None)

    dev_batches = [to_dev(*b) for b in batches[: Wm + K]]
    pin_batches = [to_pinned(*b) for b in batches[Wm + K:]]
    st = rp.stream

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(Wm):
        rp.apply_batch(*dev_batches[i])

    # ---- device-resident timing -------------------------------------------------------------
    sampler = ClockSampler(local_rank)
    launches = 0
    sc_ms, sc_bytes, stage = 0.0, 0, {"graph": 0.0, "frontier": 0.0, "scatter": 0.0, "update": 0.0}
    sizes = {"affected": np.zeros(L + 1), "active_edges": np.zeros(L + 1)}
    ld_last = (w.model.dims[L - 1] + 3) // 4 * 4
    pulls = rebuilt = 0
    rg_ms, rg_edges = 0.0, 0
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    ev0.record(st)
    for i in range(Wm, Wm + K):
        rp.apply_batch(*dev_batches[i])
        s = rp.stats()
        launches += s["gpu_launches"]
        stage["graph"] += s["ms_graph"]
        for l in range(1, L + 1):
            stage["frontier"] += s["ms_frontier"][l]
            stage["scatter"] += s["ms_scatter"][l]
            stage["update"] += s["ms_update"][l]
        pulls += s["scatter_pull"][L] == 1
        rebuilt += s["scatter_pull"][L] == 2
        rg_ms += s["ms_regather"][L]
        rg_edges += s["in_edges"][L] if s["scatter_pull"][L] == 2 else 0
        sc_ms += s["ms_scatter_kernel"][L]
        ld_last = s["message_width"][L]
        sc_bytes += scatter_bytes(s, L, ld_last)
        sizes["affected"] += np.array(s["affected"][: L + 1])
        sizes["active_edges"] += np.array(s["active_edges"][: L + 1])
        if args.verbose_steps:
            print(f"step {i - Wm}: hop {L} messages {s['active_edges'][L]} scatter kernel {s['ms_scatter_kernel'][L]:.4f} ms",
                  file=sys.stderr, flush=True)
    ev1.record(st)
    barrier()
    clocks = sampler.stop()
    dev_ms = ev0.elapsed_time(ev1)

    # ---- end to end: pinned host inputs, H2D inside, result ids read back ----------------------
    lat = []
    h2d = d2h = 0
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ids_host = torch.empty(w.n, dtype=torch.int32).pin_memory()   # the read-out lands in pinned memory, like the inputs
    e0.record(st)
    for u, r, ow in pin_batches:
        t0 = time.perf_counter()
        rp.apply_batch(u, r, ow)
        dev_ids = rp.affected(L)          # trigger-style read-out: who changed at the last layer
        ids = ids_host[: dev_ids.numel()]
        ids.copy_(dev_ids, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        lat.append(time.perf_counter() - t0)
        h2d += u.numel() * 4 + r.numel() * 4 + (ow.numel() * 4 if ow is not None else 0)
        d2h += ids.numel() * 4
    e1.record(st)
    barrier()
    e2e_ms = e0.elapsed_time(e1)

    dev_ms, e2e_ms = max_over_ranks([dev_ms, e2e_ms], world)
    if world > 1:   # the replicas are done with each other; rank 0 alone reports
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        rp.close()
        return

    hbm_peak, peak_kind = load_peaks()
    # The dominant kernel is the last hop's push scatter.  Every message is delivered as vector
    # reductions (red.global.add.v4.f32) that the L2 slices retire; whether issued lane by lane or as
    # one bulk reduction of the copy engine per message, they take the same time, so the bound of the
    # kernel is the reduction path of L2, not HBM.  achieved = payload (messages x row bytes) per second;
    # peak = the same reductions, and nothing else, issued into consecutive rows of an L2-resident
    # window, the fastest pattern of that path, timed live by the library's probe.
    msgs = float(sizes["active_edges"][L]) / K
    graph_kind = args.workload.split("-")[0]
    per_msg = NCU_DRAM_BYTES_PER_MESSAGE.get((graph_kind, ld_last)) if pulls == 0 and rebuilt == 0 else None
    traffic = per_msg * msgs if per_msg else None
    payload = msgs * ld_last * 4
    achieved = payload / 1e9 / (sc_ms / K / 1e3) if sc_ms > 0 else None
    algorithmic = (sc_bytes / 1e9) / (sc_ms / 1e3) if sc_ms > 0 else None
    compulsory = (sizes["affected"][L - 1] / K * 4 * ld_last + 4 * msgs + sizes["affected"][L] / K * 8 * ld_last)
    roofline = {"bound": "l2-reduction", "achieved": achieved, "peak": None, "unit": "GB/s", "frac": None,
                "traffic": traffic,
                "frac_hbm": (traffic / 1e9 / (sc_ms / K / 1e3) / hbm_peak) if (traffic and sc_ms > 0) else None,
                "hbm_peak": hbm_peak, "hbm_peak_source": f"of {peak_kind}",
                "kernel": f"{'k_scatter_gather' if pulls * 2 > K else 'k_scatter_push'} (hop {L}, row width {ld_last} floats)",
                "pull_steps": int(pulls),
                "ms_per_launch": sc_ms / K,
                "messages_per_launch": msgs,
                "algorithmic_push_form": {"bytes_per_launch": sc_bytes / K, "GBps": algorithmic,
                                          "note": "the push formula: sender rows and out-lists once, one read + one write "
                                                  "of the sink's row per message; the rows mostly sit in L2, so this is "
                                                  "not a DRAM rate"},
                "compulsory_bytes_per_launch": compulsory,
                "note": "achieved = messages x row bytes / kernel time; peak = probe of the L2 reduction path "
                        "(consecutive rows, 64 MB window); traffic = DRAM bytes per launch from a one-pass ncu capture "
                        "at full size, per message, times this run's messages; frac_hbm = traffic / time / measured "
                        "HBM copy rate.  The target of 60 % of HBM peak does not apply to a kernel whose rows are "
                        "served and reduced in L2"}
    line = {
        "metric": METRIC, "value": whole_job_rate(world, args.batch, K, dev_ms), "unit": UNIT,
        "n_gpus": world, "steps": K, "warmup": Wm, "ms_per_step": dev_ms / K,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": f"{args.workload}, batch {args.batch}", "batch": args.batch,
                   "vertices": w.n, "edges": w.e, "dims": w.model.dims,
                   "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                   "l2": "working set (aggregate and embedding rows, GBs) far larger than L2; no flush needed"},
        "clocks": clocks,
        "e2e": {"value": whole_job_rate(world, args.batch, K, e2e_ms), "unit": UNIT,
                "h2d_bytes_per_step": h2d // K, "d2h_bytes_per_step": d2h // K},
        "gpu_launches": int(launches),
        "latency_ms": {"p50": 1e3 * pct(lat, 50), "p99": 1e3 * pct(lat, 99), "mean": 1e3 * float(np.mean(lat)),
                       "note": "host wall clock around the C-ABI call with pinned host inputs"},
        "roofline": roofline,
        "stage_ms_per_step": {k: v / K for k, v in stage.items()},
        "per_layer": {"affected": (sizes["affected"] / K).tolist(),
                      "active_edges": (sizes["active_edges"] / K).tolist()},
        "bootstrap_ms": bootstrap_ms,
    }
    rp.close()
    del rp
    torch.cuda.empty_cache()
    if rebuilt * 2 > K and rg_ms > 0:
        # The last hop rebuilt its aggregates in most steps: the dominant kernels are the gather over the in-lists of
        # the affected sinks, bounded by the rate at which L2 serves whole-row gathers.  achieved = in-edges x row
        # bytes per second; peak = the library's gather probe (same lane layout, no index traffic) on a 64 MB window.
        edges = rg_edges / rebuilt
        ms = rg_ms / rebuilt
        got = edges * ld_last * 4 / 1e9 / (ms / 1e3)
        pk = edges * ld_last * 4 / 1e9 / (ripple.probe_gather_rate(max(1, (64 << 20) // (ld_last * 4)), ld_last, int(edges)) / 1e3)
        per_edge = NCU_DRAM_BYTES_PER_IN_EDGE.get((graph_kind, ld_last))
        traffic = per_edge * edges if per_edge else None
        line["roofline"] = {
            "bound": "l2-gather", "achieved": got, "peak": pk, "unit": "GB/s", "frac": got / pk, "traffic": traffic,
            "frac_hbm": (traffic / 1e9 / (ms / 1e3) / hbm_peak) if traffic else None,
            "hbm_peak": hbm_peak, "hbm_peak_source": f"of {peak_kind}",
            "kernel": f"k_regather + k_spmm_hubs (hop {L}, row width {ld_last} floats)",
            "ms_per_launch": ms, "in_edges_per_launch": edges, "rebuilt_steps": int(rebuilt),
            "note": "the last hop rebuilds the affected aggregates from their in-lists; achieved = in-edges x row bytes / "
                    "time of the two gather kernels; peak = probe of L2 row gathers on a 64 MB window"}
    elif pulls == 0 and sc_ms > 0 and msgs >= 1:
        # The push scatter is made of 16-byte vector reductions that mostly land in L2.  The same
        # number of reductions of the same row width into pseudo-random rows, timed alone, gives the
        # ceiling of that path on this GPU: with a window that fits L2, and with a window of the
        # size of the aggregate matrix (every row its own DRAM line).
        rows64 = max(1, (64 << 20) // (ld_last * 4))
        rate = lambda ms: payload / 1e9 / (ms / 1e3)
        ms_seq = ripple.probe_reduction_rate(rows64, ld_last, int(msgs), 1)
        roofline["peak"] = rate(ms_seq)
        roofline["frac"] = achieved / roofline["peak"]
        roofline["reduction_path"] = {
            "probe_consecutive_rows_64MB_GBps": rate(ms_seq),
            "probe_uniform_rows_64MB_GBps": rate(ripple.probe_reduction_rate(rows64, ld_last, int(msgs), 0)),
            "probe_uniform_rows_aggregate_sized_GBps": rate(ripple.probe_reduction_rate(w.n, ld_last, int(msgs), 0)),
            "note": "the probes issue the same count of red.global.add.v4.f32 rows, and nothing else, into a zeroed "
                    "window: consecutive rows are the best case of the path, uniformly random rows of a window as "
                    "large as the aggregate matrix its worst"}
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(args, w, src, dst, X, W)
    print(json.dumps(line), flush=True)


def run_table(args):
    """One JSON line per (workload, batch size): latency percentiles over 100 consecutive batches
    through the C ABI from pinned host buffers, stage times, frontier sizes, the last hop's scatter
    rate, and the oracle on a bounded sample of the same stream."""
    import torch
    from paper_2601_12347_b200 import build as B
    from paper_2601_12347_b200 import ripple
    B.build_library()
    torch.cuda.set_device(0)
    peak, peak_kind = load_peaks()
    for name in args.table.split(","):
        w, src, dst, X, W = make_workload(name, args.seed)
        L = len(w.model.layers)
        rp = ripple.Ripple(w.n, src, dst, X, w.model, W, timing=True, max_batch=w.extra.get("max_batch", 16384),
                           scatter_mode=args.scatter, edge_weights=w.edge_w,
                           regather_threshold=args.regather_threshold)
        boot = rp.stats()["ms_bootstrap"]
        rp.recompute_full()   # warm: the recompute-everything alternative on the same state
        full_ms = rp.stats()["ms_bootstrap"]
        stream = I.make_stream(w, src, dst, args.seed)
        orc = ostream = None
        if not args.no_cpu_baseline and args.oracle_seconds > 0:
            from oracle import oracle as O
            O.build()
            orc = O.Oracle(w.n, src, dst, X, w.model, W, edge_weights=w.edge_w)
            ostream = I.make_stream(w, src, dst, args.seed)
        for bsz in (args.batch_sizes or w.batch_sizes):
            nb = args.table_batches
            nt = min(20, nb)   # extra batches with per-stage event timing (small batches then run ungraphed)
            batches = [draw_batch(stream, w, bsz) for _ in range(5 + nb + nt)]
            pinned = []
            for ups, rows, ow in batches:
                u = torch.from_numpy(np.stack([ups["op"], ups["u"], ups["v"]], axis=1).astype(np.int32)).pin_memory()
                pinned.append((u, torch.from_numpy(rows).pin_memory(),
                               torch.from_numpy(ow).pin_memory() if ow is not None else None))
            lat, sc_ms, sc_bytes = [], 0.0, 0
            stage = {"graph": 0.0, "frontier": 0.0, "scatter": 0.0, "update": 0.0}
            aff, act = np.zeros(L + 1), np.zeros(L + 1)
            hop = {k: np.zeros(L + 1) for k in ("scatter", "update", "regather", "rebuilt", "gathered", "in_edges", "rows_rebuilt")}
            rp.set_timing(False)
            for i, (u, r, ow) in enumerate(pinned):
                if i == 5 + nb:
                    rp.set_timing(True)
                t0 = time.perf_counter()
                rp.apply_batch(u, r, ow)
                dt = time.perf_counter() - t0
                if i < 5:
                    continue
                if i < 5 + nb:
                    lat.append(dt)
                    continue
                s = rp.stats()
                stage["graph"] += s["ms_graph"]
                for l in range(1, L + 1):
                    stage["frontier"] += s["ms_frontier"][l]
                    stage["scatter"] += s["ms_scatter"][l]
                    stage["update"] += s["ms_update"][l]
                sc_ms += s["ms_scatter_kernel"][L]
                hop["scatter"] += np.array(s["ms_scatter"][: L + 1])
                hop["update"] += np.array(s["ms_update"][: L + 1])
                hop["regather"] += np.array(s["ms_regather"][: L + 1])
                hop["rebuilt"] += np.array(s["scatter_pull"][: L + 1]) == 2
                hop["gathered"] += np.array(s["scatter_pull"][: L + 1]) == 1
                hop["in_edges"] += np.array(s["in_edges"][: L + 1]) * (np.array(s["scatter_pull"][: L + 1]) == 2)
                hop["rows_rebuilt"] += np.array(s["rows_rebuilt"][: L + 1])
                sc_bytes += scatter_bytes(s, L, s["message_width"][L])
                aff += np.array(s["affected"][: L + 1])
                act += np.array(s["active_edges"][: L + 1])
            line = {"workload": name, "batch": bsz, "batches": nb,
                    "updates_per_sec": bsz * nb / sum(lat),
                    "latency_ms": {"mean": 1e3 * float(np.mean(lat)), "p50": 1e3 * pct(lat, 50), "p99": 1e3 * pct(lat, 99)},
                    "stage_ms": {k: v / nt for k, v in stage.items()},
                    "affected": (aff / nt).round(1).tolist(), "active_edges": (act / nt).round(1).tolist(),
                    "last_hop_scatter": {"ms": sc_ms / nt, "algorithmic_GBps": (sc_bytes / 1e9) / (sc_ms / 1e3) if sc_ms else None,
                                         "frac_of_" + peak_kind: ((sc_bytes / 1e9) / (sc_ms / 1e3) / peak) if sc_ms else None},
                    "hop_ms": {k: (v[1:] / nt).round(3).tolist() for k, v in hop.items() if k not in ("in_edges", "rows_rebuilt")},
                    "rows_rebuilt_on_budget": (hop["rows_rebuilt"][1:] / nt).round(1).tolist(),
                    "bootstrap_ms": boot, "full_recompute_ms": full_ms}
            if hop["rebuilt"][L] > 0:
                # the dominant kernels of a rebuilding hop: the gather over the in-lists of the affected sinks
                # (k_regather for short lists, k_spmm_hubs for the chunks of long ones).  It is bounded by the
                # rate at which L2 serves row gathers: achieved = in-edges x row bytes per second, peak = the
                # library's gather probe (same lane layout, no index traffic at all) on an L2-resident window
                # of 64 MB; the same probe on a window of the source matrix's size (uniformly random rows, so
                # mostly DRAM) is reported beside it.
                ldw = s["message_width"][L]
                ms = hop["regather"][L] / hop["rebuilt"][L]
                edges = hop["in_edges"][L] / hop["rebuilt"][L]
                got = edges * ldw * 4 / 1e9 / (ms / 1e3)
                pk = edges * ldw * 4 / 1e9 / (ripple.probe_gather_rate(max(1, (64 << 20) // (ldw * 4)), ldw, int(edges)) / 1e3)
                pk_big = edges * ldw * 4 / 1e9 / (ripple.probe_gather_rate(w.n, ldw, int(edges)) / 1e3)
                per_edge = NCU_DRAM_BYTES_PER_IN_EDGE.get((name.split("-")[0], ldw))
                line["last_hop_gather"] = {
                    "bound": "l2-gather", "kernel": f"k_regather + k_spmm_hubs (hop {L}, row width {ldw} floats)",
                    "ms": ms, "in_edges": edges, "achieved_GBps": got, "peak_GBps": pk, "frac": got / pk,
                    "probe_uniform_rows_matrix_sized_GBps": pk_big,
                    "traffic": per_edge * edges if per_edge else None,
                    "frac_hbm": (per_edge * edges / 1e9 / (ms / 1e3) / peak) if per_edge else None}
            if orc is not None:
                spent, done = 0.0, 0
                while spent < args.oracle_seconds and done < nb:
                    ups, rows, ow = draw_batch(ostream, w, bsz)
                    t0 = time.perf_counter()
                    assert orc.apply_incremental(ups, rows, pull=True, op_weights=ow) == 0
                    spent += time.perf_counter() - t0
                    done += 1
                line["oracle"] = {"updates_per_sec": bsz * done / spent, "batches": done, "cores": O.num_threads()}
            print(json.dumps(line), flush=True)
        rp.close()
        del rp
        if orc is not None:
            orc.close()
        torch.cuda.empty_cache()


def run_partitioned(args):
    """The partitioned execution (Sec. 4 of the paper) with P workers ON ONE GPU: every phase runs worker
    after worker, so the wall time per batch is the sum over the workers; beside it the line gives, per
    batch, the sum over the phases of the slowest worker's time for that phase: what P GPUs would take if
    the exchange cost nothing beyond what one GPU's memory system charges for it.  Neither is a
    measurement on NVLink hardware.  Also: combined halo rows sent per hop, and the single-context time on
    the same stream."""
    import torch
    from paper_2601_12347_b200 import build as B
    from paper_2601_12347_b200 import partitioned as PT
    from paper_2601_12347_b200 import ripple
    B.build_library()
    torch.cuda.set_device(0)
    Pn = args.partitioned
    for name in args.table.split(","):
        w, src, dst, X, W = make_workload(name, args.seed)
        L = len(w.model.layers)
        owner = np.random.default_rng(args.seed).integers(0, Pn, size=w.n).astype(np.int32)
        cl = PT.Cluster(Pn, owner, src, dst, X, w.model, W, max_batch=w.extra.get("max_batch", 16384),
                        edge_weights=w.edge_w)
        rp = ripple.Ripple(w.n, src, dst, X, w.model, W, max_batch=w.extra.get("max_batch", 16384),
                           scatter_mode=ripple.SCATTER_PUSH, rebuild_budget=-1.0, edge_weights=w.edge_w)
        stream = I.make_stream(w, src, dst, args.seed)
        for bsz in (args.batch_sizes or w.batch_sizes):
            nb = args.table_batches
            wall, model, single = [], [], []
            sent = np.zeros(L + 1)
            for i in range(5 + nb):
                ups, rows, ow = draw_batch(stream, w, bsz)
                t0 = time.perf_counter()
                rp.apply_batch(ups, rows, ow)
                t_single = time.perf_counter() - t0
                t0 = time.perf_counter()
                cl.router.route(ups)
                shares = [cl.router.batch(r) for r in range(Pn)]
                t_route = time.perf_counter() - t0
                crit = t_route

                def phase(fn):
                    worst = 0.0
                    for r, wk in enumerate(cl.workers):
                        t1 = time.perf_counter()
                        fn(r, wk)
                        worst = max(worst, time.perf_counter() - t1)
                    return worst

                def begin(r, wk):
                    lu, nc, row_of, first, ho, hr, op_of = shares[r]
                    if ho.size:
                        wk.set_halos(first, ho, hr)
                    wk.begin(lu, PT.payload_rows(rows, row_of, wk.dims[0]), nc, ow[op_of] if ow is not None else None)

                crit += phase(begin)
                for l in range(1, L + 1):
                    crit += phase(lambda r, wk: wk.hop_send(l))
                    crit += phase(lambda r, wk: wk.hop_compute(l))
                crit += phase(lambda r, wk: wk.end())
                t_wall = time.perf_counter() - t0
                if i >= 5:
                    wall.append(t_wall); model.append(crit); single.append(t_single)
                    sent += np.array(cl.rows_sent())
            print(json.dumps({
                "workload": name, "batch": bsz, "batches": nb, "workers": Pn, "placement": "uniformly random owners",
                "one_gpu_sequential_ms": {"p50": 1e3 * pct(wall, 50), "p99": 1e3 * pct(wall, 99)},
                "slowest_worker_per_phase_ms": {"p50": 1e3 * pct(model, 50), "p99": 1e3 * pct(model, 99)},
                "single_context_push_ms": {"p50": 1e3 * pct(single, 50), "p99": 1e3 * pct(single, 99)},
                "halo_rows_sent_per_hop": (sent[1:] / nb).round(1).tolist(),
                "note": "all workers on one GPU; not a measurement on NVLink hardware"}), flush=True)
        cl.close()
        rp.close()
        torch.cuda.empty_cache()


def run_partitioned_dist(args, rank, world, local_rank):
    """One worker of the partitioned execution (Sec. 4 of the paper) per process: the whole graph is split over
    the ranks (uniformly random vertex-partition map, the worst cut), every rank routes the same batches with
    its own replica of the router, peers are reached through CUDA IPC mappings, a barrier separates the phases
    of a hop.  Strong scaling: the job is one stream of batches.  Times are wall clock between barriers, the
    maximum over ranks.  With fewer GPUs than ranks (how this mode was exercised: two processes on one GPU) the
    ranks share devices and the process group runs on gloo."""
    import torch
    import torch.distributed as dist
    from paper_2601_12347_b200 import build as B
    from paper_2601_12347_b200 import partitioned as PT
    B.build_library()
    ndev = torch.cuda.device_count()
    torch.cuda.set_device(local_rank % ndev)
    shared = world > ndev
    if shared:
        dist.init_process_group("gloo")
    else:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    w, src, dst, X, W = make_workload(args.workload, args.seed)
    owner = np.random.default_rng(args.seed).integers(0, world, size=w.n).astype(np.int32)
    dw = PT.DistributedWorker(owner, src, dst, X, w.model, W, max_batch=max(args.batch, 16) * 2, edge_weights=w.edge_w)
    stream = I.make_stream(w, src, dst, args.seed)
    K, Wm = args.steps, args.warmup
    batches = [draw_batch(stream, w, args.batch) for _ in range(Wm + K)]
    for b in batches[:Wm]:
        dw.apply_batch(*b)
    L = len(w.model.layers)
    sent = np.zeros(L + 1)
    dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for b in batches[Wm:]:
        dw.apply_batch(*b)
        sent += np.array(dw.worker.rows_sent())
    torch.cuda.synchronize()
    dist.barrier()
    ms = (time.perf_counter() - t0) * 1e3
    (ms,) = max_over_ranks([ms], world, device="cpu" if shared else "cuda")
    tot = torch.tensor(sent, dtype=torch.float64, device="cpu" if shared else "cuda")
    dist.all_reduce(tot)
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": args.batch * K / (ms / 1e3), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": Wm, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{args.workload}, batch {args.batch}", "batch": args.batch,
                       "parallelism": f"partitioned over {world} workers, uniformly random owners",
                       "devices": min(world, ndev)},
            "halo_rows_sent_per_step": [round(float(x) / K, 1) for x in tot[1:].tolist()],
            "note": "wall clock between barriers, max over ranks" + ("; ranks share GPUs: not a scaling measurement" if shared else "")}),
            flush=True)
    dist.barrier()
    dw.close()
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--table", default="", help="comma-separated workloads: print one line per batch size")
    ap.add_argument("--table-batches", type=int, default=100)
    ap.add_argument("--batch-sizes", type=lambda s: [int(x) for x in s.split(",")], default=None,
                    help="--table: these batch sizes instead of the workload's own")
    ap.add_argument("--oracle-seconds", type=float, default=10.0)
    ap.add_argument("--regather-threshold", type=float, default=0.0,
                    help="share of all edges from which a hop rebuilds its aggregates (0: library default, <0: never)")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="dense-2l")
    ap.add_argument("--batch", type=int, default=1000)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--scatter", type=int, default=0, help="0 auto, 1 push, 2 gather per sink")
    ap.add_argument("--partitioned", type=int, default=0,
                    help="with --table: run the workloads as this many workers of the partitioned execution, all on one GPU")
    ap.add_argument("--partitioned-dist", action="store_true",
                    help="under torchrun: one worker of the partitioned execution per rank (strong scaling) instead of replicas")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--verbose-steps", action="store_true", help="per timed step: messages and scatter time (stderr)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.partitioned_dist and args.impl == "ours":
        run_partitioned_dist(args, rank, world, local_rank)
    elif args.table and args.partitioned > 0:
        if rank == 0:
            run_partitioned(args)
    elif args.table:
        if rank == 0:
            run_table(args)
    elif args.impl == "reference":
        run_reference(args, rank, world)
    else:
        if world > 1 and rank != 0:
            args.no_cpu_baseline = True
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
