#!/usr/bin/env python
"""Benchmark of the MultiWrite dispatch hot path (plan -> pack -> deliver) on B200.

One step = one whole pass over one batch: mw_plan_prefetch, then mw_pack and mw_deliver in the MultiWrite
layout, all through the C ABI, inputs resident in device memory.  The workload is the
DeepSeek-V3-shaped prefill dispatch (64 ranks, 256 experts, top-8, 4096 tokens, 7168 bf16 per row).
The step cycles over several buffer sets so that every step's inputs and outputs come from HBM,
not L2.  Prints one JSON line: the headline keys first, then the blocks for the other shapes and paths; the
last keys are tiny, unicast, large_ep, pipelined, bytes_saved_pct, decode and a compact metric_summary.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-extras]

With N > 1 every rank runs the same workload on its own GPU with its own seed: independent replicas, no
collective on the data path; the time is the maximum over ranks.  Started without a launcher (no WORLD_SIZE in
the environment) the script starts the N ranks itself through torch.distributed.run.
`--impl reference` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "dispatch pack+deliver HBM GB/s & % of peak; decode-shape p50 µs; bytes saved %"
WORKLOAD = "dsv3_prefill"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy read+write)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def algorithmic_bytes(tot: dict, B: int) -> dict:
    Tn, SD = tot["T_nonempty"], tot["total_dest"]
    return {"pack": 2 * Tn * B, "deliver": (Tn + SD) * B, "step": (3 * Tn + SD) * B}


def recorded_traffic(workload: str = WORKLOAD):
    """DRAM bytes per deliver launch from the committed ncu summary of that workload, or None when the kernel source
    has changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", f"deliver_{workload}_ncu.md")
    try:
        text = open(path).read()
        m_t = re.search(r"traffic_bytes_per_launch\s*=\s*(\d+)", text)
        m_h = re.search(r"kernel_source_sha256\s*=\s*([0-9a-f]{64})", text)
        if not m_t or not m_h or m_h.group(1) != kernel_source_hash():
            return None
        return int(m_t.group(1))
    except Exception:
        return None


def kernel_source_hash() -> str:
    h = hashlib.sha256()
    for name in ("mw_copy.cu",):
        with open(os.path.join(ROOT, "paper_2605_22428_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def roofline_block(kernel: str, alg_bytes: int, times_ms: list, traffic, peak: float, peak_src: str) -> dict:
    """The roofline object of one kernel from its per-launch CUDA-event durations: `achieved` counts the algorithmic
    bytes, `dram_gbs` the DRAM bytes ncu recorded for one launch (reads served by L2 are not in it)."""
    mean_ms = statistics.mean(times_ms)
    achieved = alg_bytes / (mean_ms * 1e-3) / 1e9
    out = {"bound": "hbm", "kernel": kernel, "launches_timed": len(times_ms), "achieved": round(achieved, 1), "peak": peak,
           "unit": "GB/s", "frac": round(achieved / peak, 4), "peak_source": peak_src,
           "mean_us": round(mean_ms * 1e3, 2), "p50_us": round(statistics.median(times_ms) * 1e3, 2),
           "algorithmic_bytes_per_launch": alg_bytes, "traffic": traffic}
    if traffic:
        out["dram_gbs"] = round(traffic / (mean_ms * 1e-3) / 1e9, 1)
        out["dram_frac"] = round(out["dram_gbs"] / peak, 4)
        out["dram_frac_of_nominal_8TBs"] = round(out["dram_gbs"] / NOMINAL_HBM_GBS, 4)
    return out


def time_deliver_launches(ctx, mw, torch, ids, e2r, T, sets, Tn, SD, launches: int = 200, warmup: int = 20) -> list:
    """CUDA-event duration (ms) of `launches` deliver launches, each right after the plan and pack launches of its
    step (so the send rows are where the step leaves them), cycling over the buffer sets."""
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(launches)]
    for i in range(warmup + launches):
        x, send, recv = sets[i % len(sets)]
        ctx.mw_plan_prefetch(ids, e2r, T, x)
        ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send, Tn)
        if i >= warmup:
            evs[i - warmup][0].record()
        ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send, recv, 0, SD)
        if i >= warmup:
            evs[i - warmup][1].record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in evs]


# ---- clocks ------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock, power and clock-event reasons through NVML while the GPU is under load."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
               0x80: "hw_power_brake", 0x2: "applications_clocks_setting", 0x100: "display_clock_setting",
               0x10: "sync_boost"}

    def __init__(self, device_index: int):
        self.samples = []
        self.error = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # pragma: no cover
            self.error = f"{type(e).__name__}: {e}"

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                watts = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                self.samples.append((time.perf_counter(), mhz, reasons, watts))
            except Exception as e:  # pragma: no cover
                self.error = f"{type(e).__name__}: {e}"
                return
            time.sleep(0.002)

    def start(self):
        if self.error is None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=2)

    def summary(self, t0: float, t1: float) -> dict:
        if self.error is not None and not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "error": self.error}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        window = "timed region"
        if len(inside) < 2:
            inside, window = list(self.samples), "warm-up + timed region + the roofline kernel's own loop + end-to-end runs (the timed region alone is too short to sample)"
        bits = 0
        for s in inside:
            bits |= s[2]
        reasons = sorted(name for bit, name in self.REASONS.items() if bits & bit)
        return {"sm_mhz": statistics.median(s[1] for s in inside) if inside else None, "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "power_w_max": max((s[3] for s in inside), default=None),
                "samples": len(inside), "window": window}


# ---- the oracle as a CPU baseline ---------------------------------------------------------------------
def oracle_pass(inp, R: int, B: int):
    """One pass of the hot path on the CPU oracle; returns (seconds, totals)."""
    from oracle import mwo
    t0 = time.perf_counter()
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, B)
    send = mwo.pack_mw(p, inp.x)
    mwo.deliver_mw(p, send)
    return time.perf_counter() - t0, p.totals


def sample_inputs(inp, T: int):
    from paper_2605_22428_b200 import workloads as wl
    if T >= inp.T:
        return inp
    return wl.DispatchInputs(inp.shape, inp.seed, np.ascontiguousarray(inp.topk_ids[:T]), inp.expert_to_rank,
                             np.ascontiguousarray(inp.x[:T]))


def oracle_stages(inp, R: int, B: int, threads: int = 1, keep: bool = False):
    """One pass of the oracle, stage by stage: (plan s, pack s, deliver s, totals).  With threads > 1 the send rows are
    cut into contiguous slices and the oracle's own pack / deliver functions run on one slice per thread (the C calls
    release the interpreter lock; slices write disjoint rows); the plan is a sequential walk and stays on one core."""
    import ctypes as C
    from oracle import mwo
    t0 = time.perf_counter()
    p = mwo.plan(inp.topk_ids, inp.expert_to_rank, R, B)
    t1 = time.perf_counter()
    Tn, SD = p.totals["T_nonempty"], p.totals["total_dest"]
    if threads <= 1:
        send = mwo.pack_mw(p, inp.x)
        t2 = time.perf_counter()
        recv = mwo.deliver_mw(p, send)
        t3 = time.perf_counter()
        return (t1 - t0, t2 - t1, t3 - t2, p.totals) + ((send, recv) if keep else ())
    from concurrent.futures import ThreadPoolExecutor
    lib = mwo.lib()
    xb = np.ascontiguousarray(inp.x).view(np.uint8).reshape(inp.T, B)
    send = np.empty((max(Tn, 1), B), np.uint8)
    recv = np.empty(max(SD, 1) * B, np.uint8)
    cuts = [Tn * k // threads for k in range(threads + 1)]
    vp = C.c_void_p

    def pack(k):
        j0, n = cuts[k], cuts[k + 1] - cuts[k]
        lib.mwo_pack_mw(vp(xb.ctypes.data), C.c_int64(B), vp(p.mw_row_token.ctypes.data + 4 * j0), C.c_int64(n),
                        vp(send.ctypes.data + j0 * B))

    def deliver(k):
        j0, n = cuts[k], cuts[k + 1] - cuts[k]
        lib.mwo_deliver_mw(vp(send.ctypes.data + j0 * B), C.c_int64(B), C.c_int64(n), C.c_int32(R), C.c_int32(p.K),
                           vp(p.mw_row_token.ctypes.data + 4 * j0), vp(p.token_group.ctypes.data), vp(p.group_mask.ctypes.data),
                           vp(p.dest_pos.ctypes.data), vp(p.rank_offsets.ctypes.data), vp(recv.ctypes.data), C.c_int64(0))

    with ThreadPoolExecutor(threads) as pool:
        list(pool.map(pack, range(threads)))
        t2 = time.perf_counter()
        list(pool.map(deliver, range(threads)))
        t3 = time.perf_counter()
    return (t1 - t0, t2 - t1, t3 - t2, p.totals) + ((send[:Tn], recv[:SD * B]) if keep else ())


def cpu_baseline(inp, R: int, B: int, budget_s: float = 10.0) -> dict:
    """The oracle on the host cores: single thread (the headline figure of this block) and all cores, per stage."""
    first = oracle_stages(inp, R, B)                # also warms the page cache
    secs = sum(first[:3])
    reps = max(1, min(8, int(budget_s / max(secs, 1e-3))))
    runs = [oracle_stages(inp, R, B) for _ in range(reps)]
    best = min(runs, key=lambda r: sum(r[:3]))
    tot = best[3]
    step_bytes = algorithmic_bytes(tot, B)["step"]
    cores = os.cpu_count() or 1
    par_runs = [oracle_stages(inp, R, B, threads=cores) for _ in range(max(1, min(4, reps)))]
    par = min(par_runs, key=lambda r: sum(r[:3]))
    ms = lambda v: round(v * 1e3, 2)
    return {"value": step_bytes / sum(best[:3]) / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
            "sample": f"full {WORKLOAD} batch ({inp.T} tokens), best of {reps} passes after one warm-up pass, "
                      f"plan+pack+deliver in plain single-threaded C",
            "ms_per_step": ms(sum(best[:3])), "plan_ms": ms(best[0]), "pack_ms": ms(best[1]), "deliver_ms": ms(best[2]),
            "median_ms": ms(statistics.median(sum(r[:3]) for r in runs)),
            "all_cores": {"value": step_bytes / sum(par[:3]) / 1e9, "unit": "GB/s", "cores": cores,
                          "ms_per_step": ms(sum(par[:3])), "plan_ms": ms(par[0]), "pack_ms": ms(par[1]), "deliver_ms": ms(par[2]),
                          "how": "send rows cut into one slice per core, the oracle's pack and deliver run per slice on a "
                                 "thread each; the plan stays sequential"}}


def run_reference(args):
    """`--impl reference`: the CPU oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2605_22428_b200 import workloads as wl
    inp = wl.make_dispatch(WORKLOAD)
    s = inp.shape
    B = s.row_bytes
    first, _ = oracle_pass(inp, s.R, B)
    total_steps = args.steps + args.warmup
    T = s.T
    while T > 256 and first * (T / s.T) * total_steps > 150.0:   # bound the whole run to a few minutes
        T //= 2
    smp = sample_inputs(inp, T)
    for _ in range(args.warmup):
        oracle_pass(smp, s.R, B)
    t0 = time.perf_counter()
    tot = None
    for _ in range(args.steps):
        _, tot = oracle_pass(smp, s.R, B)
    dt = time.perf_counter() - t0
    ms = dt / args.steps * 1e3
    value = algorithmic_bytes(tot, B)["step"] / (dt / args.steps) / 1e9
    sample = f"first {T} of {s.T} tokens of {WORKLOAD} per step, plan+pack+deliver in plain single-threaded C"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": WORKLOAD, "R": s.R, "E": s.E, "K": s.K, "T": T, "row_bytes": B, "layout": "multiwrite"},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ---- the CUDA path -------------------------------------------------------------------------------------
def percentile(v, q):
    v = sorted(v)
    return v[min(len(v) - 1, int(round(q * (len(v) - 1))))]


def decode_latency(mw, wl, torch, launches: int = 1000) -> dict:
    """Decode shape (64 tokens, 256 ranks): p50 / p99 over `launches` calls of plan, dispatch and the chain."""
    inp = wl.make_dispatch("decode")
    s = inp.shape
    B = s.row_bytes
    ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    x = torch.from_numpy(inp.x.view(np.int16)).cuda()
    out = {}
    with mw.Context(s.R, s.E, s.K, s.T, B) as ctx:
        ctx.mw_plan(ids, e2r, s.T)
        tot = ctx.mw_get_totals()
        send = torch.empty(tot["T_nonempty"] * B, dtype=torch.uint8, device="cuda")
        recv = torch.empty(tot["total_dest"] * B, dtype=torch.uint8, device="cuda")
        Tn, SD = tot["T_nonempty"], tot["total_dest"]

        def plan():
            ctx.mw_plan(ids, e2r, s.T)

        def dispatch():
            ctx.mw_dispatch(x, mw.MW_LAYOUT_MULTIWRITE, send, Tn, recv, 0, SD)

        def chain():
            plan()
            dispatch()

        def one_call():
            ctx.mw_plan_dispatch(ids, e2r, s.T, x, mw.MW_LAYOUT_MULTIWRITE, send, Tn, recv, 0, SD)

        for name, fn in (("plan", plan), ("pack_deliver", dispatch), ("chain", chain), ("one_call", one_call)):
            for _ in range(min(50, launches)):
                fn()
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(launches)]
            torch.cuda.synchronize()
            for a, b in evs:
                a.record()
                fn()
                b.record()
            torch.cuda.synchronize()
            us = [a.elapsed_time(b) * 1e3 for a, b in evs]
            out[name] = {"p50_us": round(percentile(us, 0.5), 2), "p99_us": round(percentile(us, 0.99), 2)}
        # the single-launch call keeps no host-side state, so it can be replayed from a CUDA graph: no host launch cost
        torch.cuda.synchronize()
        graph, chained, n_chain = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph(), 20
        with torch.cuda.graph(graph):
            one_call()
        with torch.cuda.graph(chained):
            for _ in range(n_chain):
                one_call()
        for _ in range(20):
            graph.replay()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(launches)]
        torch.cuda.synchronize()
        for a, b in evs:
            a.record()
            graph.replay()
            b.record()
        torch.cuda.synchronize()
        us = [a.elapsed_time(b) * 1e3 for a, b in evs]
        out["one_call_graph"] = {"p50_us": round(percentile(us, 0.5), 2), "p99_us": round(percentile(us, 0.99), 2)}
        evs = evs[:min(50, launches)]
        for a, b in evs:
            a.record()
            chained.replay()
            b.record()
        torch.cuda.synchronize()
        us = [a.elapsed_time(b) * 1e3 / n_chain for a, b in evs]
        out["one_call_graph_chained"] = {"p50_us": round(percentile(us, 0.5), 2), "calls_per_graph": n_chain}
        assert ctx.mw_get_totals()["status"] == 0
    out["launches"] = launches
    out["note"] = ("L2-resident (0.9 MB in, 7.3 MB out): latency, not an HBM fraction; chain = mw_plan + mw_dispatch, one_call = "
                   "mw_plan_dispatch (1 launch); host launch cost included except in the graph replays (chained: 20 calls per graph)")
    return out


def allgather_sweep(mw, wl, torch) -> list:
    """AllGather pack + deliver over shard sizes 4 KB .. 64 MB at R = 64 (MultiWrite layout).  The full
    R x R result does not fit in memory for large shards: a window of destination ranks is materialised
    (the largest power of two whose receive area stays under 8 GB); GB/s counts the bytes actually moved."""
    R = wl.ALLGATHER_R
    out = []
    with mw.Context(R, 8, 2, 16, 32) as ctx:
        for S in wl.ALLGATHER_SHARD_BYTES:
            window = R
            while window > 1 and window * R * S > (8 << 30):
                window //= 2
            shards = torch.empty(R * S, dtype=torch.uint8, device="cuda").random_(0, 256)
            send = torch.empty(R * S, dtype=torch.uint8, device="cuda")
            recv = torch.empty(window * R * S, dtype=torch.uint8, device="cuda")
            reps = 20 if S <= (1 << 20) else 5

            def run():
                ctx.mw_allgather_pack(shards, S, mw.MW_LAYOUT_MULTIWRITE, send, recv, 0, 0, window)

            for _ in range(3):
                run()
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
            torch.cuda.synchronize()
            for a, b in evs:
                a.record()
                run()
                b.record()
            torch.cuda.synchronize()
            us = statistics.median(a.elapsed_time(b) for a, b in evs) * 1e3
            moved = R * S + R * S + window * R * S            # one pass: shards read, send buffer + window copies written
            out.append({"shard_bytes": S, "window_ranks": window, "p50_us": round(us, 1),
                        "gbs": round(moved / us / 1e3, 1), "l2_resident": bool(moved < (100 << 20))})
            del shards, send, recv
            torch.cuda.empty_cache()
    return out


def relay_measure(mw, wl, torch, n: int = 50) -> dict:
    """Two-level dispatch (Section 3.2) on the dsv3_prefill routing: 8 servers of 8 ranks, source = rank 0."""
    inp = wl.make_dispatch(WORKLOAD)
    s = inp.shape
    B, T, P, src = s.row_bytes, s.T, 8, 0
    ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    x = torch.from_numpy(inp.x.view(np.int16)).cuda()
    with mw.Relay(s.R, s.E, s.K, T, B, src, P) as relay:
        relay.mw_relay_plan(ids, e2r, T)
        tot = relay.mw_relay_get_totals()
        rows_send = relay.hop.mw_get_totals()["T_nonempty"]
        H, SD = tot["hop_rows"], tot["delivered_rows"]
        sets = [(torch.empty(rows_send * B, dtype=torch.uint8, device="cuda"), torch.empty(H * B, dtype=torch.uint8, device="cuda"),
                 torch.empty(SD * B, dtype=torch.uint8, device="cuda")) for _ in range(2)]

        def step(i):
            send, hop, recv = sets[i % 2]
            relay.mw_relay_plan(ids, e2r, T)
            relay.mw_relay_dispatch(x, send, rows_send, hop, H, recv, 0, SD)

        for i in range(5):
            step(i)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(n):
            step(i)
        b.record()
        torch.cuda.synchronize()
        us = a.elapsed_time(b) * 1e3 / n
        a.record()
        for i in range(n):
            relay.mw_relay_plan(ids, e2r, T)
        b.record()
        torch.cuda.synchronize()
        plan_us = a.elapsed_time(b) * 1e3 / n
        assert relay.mw_relay_get_totals()["status"] == 0
    fwd = tot["forward_bytes"] // B                                     # copies the relays forward
    held = tot["inter_multiwrite_bytes"] // B                           # copies held by relays (read back unless there is nothing to forward)
    alg = (2 * rows_send + H + held + fwd) * B                          # x read, send + hop copies written, copies read back, forwards written
    dram = (2 * rows_send + H + fwd) * B                                # the read-backs come out of L2
    return {"servers": s.R // P, "ranks_per_server": P, "src_rank": src, "hop_rows": H, "staged_rows": tot["staged_rows"],
            "delivered_rows": SD,
            "inter_server_unicast_mb": round(tot["inter_unicast_bytes"] / 1e6, 1),
            "inter_server_multiwrite_mb": round(tot["inter_multiwrite_bytes"] / 1e6, 1),
            "inter_server_bytes_saved_pct": round(100 * (1 - tot["inter_multiwrite_bytes"] / tot["inter_unicast_bytes"]), 2),
            "direct_mb": round(tot["direct_bytes"] / 1e6, 1), "relay_forward_mb": round(tot["forward_bytes"] / 1e6, 1),
            "step_us": round(us, 1), "plan_us": round(plan_us, 1), "gbs": round(alg / us / 1e3, 1),
            "dram_side_gbs": round(dram / us / 1e3, 1), "frac_of_measured_peak": round(alg / us / 1e3 / measured_peak()[0], 4),
            "note": "step = both plans (concurrent) + descriptors + one launch for both levels; gbs counts x read, send and hop "
                    "copies written, relay copies read back (upper bound) and forwards written; dram_side_gbs leaves the read-backs out"}


def paper_setup_measure(mw, wl, torch) -> list:
    """The paper's own dispatch setup (Section 6.1 / Table 1: 2 servers x 8 devices, 64 experts, top-8, balanced load,
    batches 64 / 128 / 1k / 2k), run through the two-level relayed dispatch: bytes that cross between the servers with one
    copy per destination rank against one copy per remote server.  The paper reports transfer TIMES on its hardware
    (ratios 2.58 / 3.16 / 3.84 / 3.91); the byte ratio here is the part of that which the method itself determines."""
    out = []
    R, P, E, K, src = 16, 8, 64, 8, 0
    for T in (64, 128, 1024, 2048):
        inp = wl.make_random_dispatch(1000 + T, T=T, K=K, E=E, R=R, H=7168, contiguous_map=True)
        B = inp.shape.row_bytes
        ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
        x = torch.from_numpy(inp.x.view(np.int16)).cuda()
        with mw.Relay(R, E, K, T, B, src, P) as relay:
            relay.mw_relay_plan(ids, e2r, T)
            tot = relay.mw_relay_get_totals()
            rows_send = relay.hop.mw_get_totals()["T_nonempty"]
            H, SD = tot["hop_rows"], tot["delivered_rows"]
            send = torch.empty(rows_send * B, dtype=torch.uint8, device="cuda")
            hop = torch.empty(H * B, dtype=torch.uint8, device="cuda")
            recv = torch.empty(SD * B, dtype=torch.uint8, device="cuda")

            def step():
                relay.mw_relay_plan(ids, e2r, T)
                relay.mw_relay_dispatch(x, send, rows_send, hop, H, recv, 0, SD)

            for _ in range(5):
                step()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(50):
                step()
            b.record()
            torch.cuda.synchronize()
            assert relay.mw_relay_get_totals()["status"] == 0
        out.append({"T": T, "inter_server_unicast_mb": round(tot["inter_unicast_bytes"] / 1e6, 2),
                    "inter_server_multiwrite_mb": round(tot["inter_multiwrite_bytes"] / 1e6, 2),
                    "byte_ratio": round(tot["inter_unicast_bytes"] / max(tot["inter_multiwrite_bytes"], 1), 3),
                    "step_us": round(a.elapsed_time(b) * 1e3 / 50, 1)})
    return out


def fused_dispatch_measure(mw, wl, torch) -> dict:
    """mw_dispatch on the headline workload: pack and deliver in one pass (x read once, send buffer and receive
    regions written), reported against its own byte count; the two-call path stays the headline."""
    inp = wl.make_dispatch(WORKLOAD)
    s = inp.shape
    B, T = s.row_bytes, s.T
    ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    xh = torch.from_numpy(inp.x.view(np.int16))
    with mw.Context(s.R, s.E, s.K, T, B) as ctx:
        ctx.mw_plan(ids, e2r, T)
        tot = ctx.mw_get_totals()
        Tn, SD = tot["T_nonempty"], tot["total_dest"]
        sets = [(xh.cuda(), torch.empty(Tn * B, dtype=torch.uint8, device="cuda"),
                 torch.empty(SD * B, dtype=torch.uint8, device="cuda")) for _ in range(3)]

        def dispatch(i):
            x, send, recv = sets[i % 3]
            ctx.mw_dispatch(x, mw.MW_LAYOUT_MULTIWRITE, send, Tn, recv, 0, SD)

        def step(i):
            ctx.mw_plan(ids, e2r, T)
            dispatch(i)

        def step_prefetch(i):
            ctx.mw_plan_prefetch(ids, e2r, T, sets[i % 3][0])      # x comes out of L2; the receive slots are streamed
            dispatch(i)

        out = {}
        for name, fn, n in (("dispatch_us", dispatch, 200), ("step_us", step, 400), ("step_prefetch_us", step_prefetch, 400)):
            for i in range(6):
                fn(i)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(n):
                fn(i)
            b.record()
            torch.cuda.synchronize()
            out[name] = round(a.elapsed_time(b) * 1e3 / n, 1)
        assert ctx.mw_get_totals()["status"] == 0
    own = (2 * Tn + SD) * B
    out.update({"own_bytes_per_step": own, "dispatch_gbs": round(own / out["dispatch_us"] / 1e3, 1),
                "step_gbs": round(own / out["step_us"] / 1e3, 1), "tokens_per_s": round(T / out["step_us"] * 1e6, 1),
                "note": "one launch reads x once and writes send buffer + receive regions: (2T' + sum D) x B bytes; "
                        "step = mw_plan + mw_dispatch"})
    return out


def large_ep_measure(mw, wl, torch) -> dict:
    """The other large-batch shape (R = 128, T = 8192, Zipf-skewed experts): the same three calls as the headline step."""
    inp = wl.make_dispatch("large_ep")
    s = inp.shape
    B, T = s.row_bytes, s.T
    ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    xh = torch.from_numpy(inp.x.view(np.int16))
    with mw.Context(s.R, s.E, s.K, T, B) as ctx:
        ctx.mw_plan(ids, e2r, T)
        tot = ctx.mw_get_totals()
        Tn, SD = tot["T_nonempty"], tot["total_dest"]
        sets = [(xh.cuda(), torch.empty(Tn * B, dtype=torch.uint8, device="cuda"),
                 torch.empty(SD * B, dtype=torch.uint8, device="cuda")) for _ in range(2)]      # 2 x 1.17 GB > L2

        def step(i):
            x, send, recv = sets[i % 2]
            ctx.mw_plan_prefetch(ids, e2r, T, x)
            ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send, Tn)
            ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send, recv, 0, SD)

        def step_plain(i):
            x, send, recv = sets[i % 2]
            ctx.mw_plan(ids, e2r, T)
            ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send, Tn)
            ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send, recv, 0, SD)

        def copies(i):
            x, send, recv = sets[i % 2]
            ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send, Tn)
            ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send, recv, 0, SD)

        out = {}
        for name, fn, n in (("step_us", step, 200), ("step_without_prefetch_us", step_plain, 200), ("pack_plus_deliver_us", copies, 200)):
            for i in range(6):
                fn(i)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(n):
                fn(i)
            b.record()
            torch.cuda.synchronize()
            out[name] = round(a.elapsed_time(b) * 1e3 / n, 1)
        peak, peak_src = measured_peak()
        deliver_roofline = roofline_block("k_copy_rows<1, SCATTER, after pack> (deliver, MultiWrite layout, large_ep)", (Tn + SD) * B,
                                          time_deliver_launches(ctx, mw, torch, ids, e2r, T, sets, Tn, SD),
                                          recorded_traffic("large_ep"), peak, peak_src)
        assert ctx.mw_get_totals()["status"] == 0
    nbytes = (3 * Tn + SD) * B
    out["roofline"] = deliver_roofline
    out.update({"rows_packed": Tn, "rows_delivered": SD, "groups": tot["G"], "algorithmic_bytes_per_step": nbytes,
                "step_frac_of_measured_peak": round(nbytes / out["step_us"] / 1e3 / measured_peak()[0], 4),
                "step_gbs": round(nbytes / out["step_us"] / 1e3, 1),
                "pack_plus_deliver_gbs": round(nbytes / out["pack_plus_deliver_us"] / 1e3, 1),
                "pack_plus_deliver_fraction_of_nominal_8TBs": round(nbytes / out["pack_plus_deliver_us"] / 1e3 / 8000.0, 4),
                "tokens_per_s": round(T / out["step_us"] * 1e6, 1)})
    return out


def mid_batch_measure(mw, wl, torch) -> list:
    """Batches between the decode shape and the prefill shape (the paper's batch 128 to 2k, Section 6.3), routing of the
    headline workload: mw_plan_dispatch (one launch up to 1024 tokens) replayed from a CUDA graph, against the three
    calls of the headline step launched one by one."""
    out = []
    for T in (128, 512, 1024, 2048, 4096):
        inp = wl.make_dispatch(WORKLOAD, T=T)
        s = inp.shape
        B = s.row_bytes
        ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
        xh = torch.from_numpy(inp.x.view(np.int16))
        with mw.Context(s.R, s.E, s.K, T, B) as ctx:
            ctx.mw_plan(ids, e2r, T)
            tot = ctx.mw_get_totals()
            Tn, SD = tot["T_nonempty"], tot["total_dest"]
            own = (2 * Tn + SD) * B
            nset = max(3, int((300 << 20) // own) + 1)
            sets = [(xh.cuda(), torch.empty(Tn * B, dtype=torch.uint8, device="cuda"),
                     torch.empty(SD * B, dtype=torch.uint8, device="cuda")) for _ in range(nset)]

            def one(i):
                x, send, recv = sets[i % nset]
                ctx.mw_plan_dispatch(ids, e2r, T, x, mw.MW_LAYOUT_MULTIWRITE, send, Tn, recv, 0, SD)

            def three(i):
                x, send, recv = sets[i % nset]
                ctx.mw_plan_prefetch(ids, e2r, T, x)
                ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send, Tn)
                ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send, recv, 0, SD)

            row = {"T": T, "own_bytes": own}
            for i in range(2 * nset):
                three(i)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(200):
                three(i)
            b.record()
            torch.cuda.synchronize()
            row["three_calls_us"] = round(a.elapsed_time(b) * 1e3 / 200, 1)
            # the same three calls replayed from a CUDA graph (the tiled plan keeps its running counts on the device)
            graph3 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph3):
                for i in range(2 * nset):
                    three(i)
            for _ in range(3):
                graph3.replay()
            torch.cuda.synchronize()
            a.record()
            for _ in range(20):
                graph3.replay()
            b.record()
            torch.cuda.synchronize()
            row["three_calls_graph_us"] = round(a.elapsed_time(b) * 1e3 / (40 * nset), 1)
            if T <= 1024:           # the single launch keeps no host-side state and can be replayed
                one(0)
                torch.cuda.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph):
                    for i in range(4 * nset):
                        one(i)
                for _ in range(3):
                    graph.replay()
                torch.cuda.synchronize()
                a.record()
                for _ in range(10):
                    graph.replay()
                b.record()
                torch.cuda.synchronize()
                row["one_call_graph_us"] = round(a.elapsed_time(b) * 1e3 / (40 * nset), 1)
                row["one_call_gbs"] = round(own / row["one_call_graph_us"] / 1e3, 1)
            assert ctx.mw_get_totals()["status"] == 0
            out.append(row)
    return out


def pipelined_measure(mw, wl, torch, name: str, steps: int = 400) -> dict:
    """The headline step with the plan of batch i+1 made while batch i is packed and delivered, through ONE context
    (mw_plan_swap / mw_plan_next): time per step (p50 over `steps` steps, CUDA events between the steps) and the latency
    of one batch from the moment its plan may start to the end of its deliver."""
    inp = wl.make_dispatch(name)
    s = inp.shape
    B, T = s.row_bytes, s.T
    ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    xh = torch.from_numpy(inp.x.view(np.int16))
    nsets = 3 if name == WORKLOAD else 2
    with mw.Context(s.R, s.E, s.K, T, B) as ctx:
        ctx.mw_plan(ids, e2r, T)
        tot = ctx.mw_get_totals()
        Tn, SD = tot["T_nonempty"], tot["total_dest"]
        sets = [(xh.cuda(), torch.empty(Tn * B, dtype=torch.uint8, device="cuda"),
                 torch.empty(SD * B, dtype=torch.uint8, device="cuda")) for _ in range(nsets)]
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 2)]

        def step(i, mark=None):
            x, send, recv = sets[i % nsets]
            ctx.mw_plan_swap()                                   # the plan of this batch, issued one step ago
            if mark is not None:
                mark.record()                                    # from here the next batch's plan may run
            ctx.mw_plan_next(ids, e2r, T)                        # no prefetch: DRAM is busy with this batch's copies
            ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send, Tn)
            ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send, recv, 0, SD)

        ctx.mw_plan_next(ids, e2r, T)
        for i in range(20):
            step(i)
        torch.cuda.synchronize()
        for i in range(steps + 1):
            step(i, marks[i])
        marks[steps + 1].record()
        torch.cuda.synchronize()
        ctx.mw_plan_swap()
        assert ctx.mw_get_totals()["status"] == 0
    per_step = [marks[i].elapsed_time(marks[i + 1]) * 1e3 for i in range(steps)]
    # batch i+1: its plan may start at mark i, its deliver ends where step i+2 begins (mark i+2)
    latency = [marks[i].elapsed_time(marks[i + 2]) * 1e3 for i in range(steps)]
    nbytes = (3 * Tn + SD) * B
    us = statistics.median(per_step)
    return {"steps": steps, "step_p50_us": round(us, 2), "step_mean_us": round(marks[0].elapsed_time(marks[steps]) * 1e3 / steps, 2),
            "step_p99_us": round(percentile(per_step, 0.99), 2), "batch_latency_p50_us": round(statistics.median(latency), 2),
            "step_gbs": round(nbytes / us / 1e3, 1), "frac_of_measured_peak": round(nbytes / us / 1e3 / measured_peak()[0], 4),
            "tokens_per_s": round(T / us * 1e6, 1),
            "note": "one context, one caller stream: mw_plan_swap + mw_plan_next + mw_pack + mw_deliver per step; latency = plan may start -> deliver done"}


def unicast_measure(mw, wl, torch, name: str, n: int = 100) -> dict:
    """The unicast layout (one copy per destination in the send buffer: Sections 2.2, 6.3) against the MultiWrite layout on
    the same batch: pack, deliver and whole step of each, same context, same plan."""
    inp = wl.make_dispatch(name)
    s = inp.shape
    B, T = s.row_bytes, s.T
    ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    xh = torch.from_numpy(inp.x.view(np.int16))
    out = {}
    with mw.Context(s.R, s.E, s.K, T, B) as ctx:
        ctx.mw_plan(ids, e2r, T)
        tot = ctx.mw_get_totals()
        Tn, SD = tot["T_nonempty"], tot["total_dest"]
        xs = [xh.cuda() for _ in range(2)]
        recvs = [torch.empty(SD * B, dtype=torch.uint8, device="cuda") for _ in range(2)]
        for layout, lname, rows in ((mw.MW_LAYOUT_UNICAST, "unicast", SD), (mw.MW_LAYOUT_MULTIWRITE, "multiwrite", Tn)):
            sends = [torch.empty(rows * B, dtype=torch.uint8, device="cuda") for _ in range(2)]
            evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n)]
            for i in range(10 + n):
                x, send, recv = xs[i % 2], sends[i % 2], recvs[i % 2]
                e = evs[i - 10] if i >= 10 else None
                if e:
                    e[0].record()
                ctx.mw_plan_prefetch(ids, e2r, T, x)
                if e:
                    e[1].record()
                ctx.mw_pack(x, layout, send, rows)
                if e:
                    e[2].record()
                ctx.mw_deliver(layout, send, recv, 0, SD)
                if e:
                    e[3].record()
            torch.cuda.synchronize()
            med = lambda a, b: statistics.median(e[a].elapsed_time(e[b]) for e in evs) * 1e3
            pack_b = (Tn + rows) * B                              # hidden rows read once, send rows written
            deliver_b = (rows + SD) * B
            out[lname] = {"pack_us": round(med(1, 2), 1), "deliver_us": round(med(2, 3), 1), "step_us": round(med(0, 3), 1),
                          "send_rows": rows, "pack_gbs": round(pack_b / med(1, 2) / 1e3, 1),
                          "deliver_gbs": round(deliver_b / med(2, 3) / 1e3, 1),
                          "bytes_moved_per_step": pack_b + deliver_b}
            del sends
        assert ctx.mw_get_totals()["status"] == 0
    u, m = out["unicast"], out["multiwrite"]
    out["time_saved_pct"] = round(100 * (1 - m["step_us"] / u["step_us"]), 2)
    out["transmitted_bytes_saved_pct"] = round(100.0 * (1 - tot["mw_bytes"] / tot["unicast_bytes"]), 3)
    out["note"] = "p50 of CUDA events around each call, %d steps; one GPU emulates every link: time follows bytes moved in HBM" % n
    return out


def tiny_measure(mw, wl, torch, launches: int = 500) -> dict:
    """The smallest configuration (8 ranks, 256 tokens of 2 KB): latency in microseconds (its working set lives in L2)."""
    inp = wl.make_dispatch("tiny")
    s = inp.shape
    B = s.row_bytes
    ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    x = torch.from_numpy(inp.x.view(np.int16)).cuda()
    out = {}
    with mw.Context(s.R, s.E, s.K, s.T, B) as ctx:
        ctx.mw_plan(ids, e2r, s.T)
        tot = ctx.mw_get_totals()
        Tn, SD = tot["T_nonempty"], tot["total_dest"]
        send = torch.empty(Tn * B, dtype=torch.uint8, device="cuda")
        recv = torch.empty(SD * B, dtype=torch.uint8, device="cuda")

        def three():
            ctx.mw_plan(ids, e2r, s.T)
            ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send, Tn)
            ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send, recv, 0, SD)

        def one_call():
            ctx.mw_plan_dispatch(ids, e2r, s.T, x, mw.MW_LAYOUT_MULTIWRITE, send, Tn, recv, 0, SD)

        for name, fn in (("three_calls", three), ("one_call", one_call)):
            for _ in range(30):
                fn()
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(launches)]
            torch.cuda.synchronize()
            for a, b in evs:
                a.record()
                fn()
                b.record()
            torch.cuda.synchronize()
            us = [a.elapsed_time(b) * 1e3 for a, b in evs]
            out[name] = {"p50_us": round(percentile(us, 0.5), 2), "p99_us": round(percentile(us, 0.99), 2)}
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            one_call()
        for _ in range(10):
            graph.replay()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(launches)]
        torch.cuda.synchronize()
        for a, b in evs:
            a.record()
            graph.replay()
            b.record()
        torch.cuda.synchronize()
        us = [a.elapsed_time(b) * 1e3 for a, b in evs]
        out["one_call_graph"] = {"p50_us": round(percentile(us, 0.5), 2), "p99_us": round(percentile(us, 0.99), 2)}
        assert ctx.mw_get_totals()["status"] == 0
    out["rows_delivered"], out["groups"] = SD, tot["G"]
    out["note"] = "L2-resident (0.5 MB in, 1.8 MB out): microseconds, not an HBM fraction; host launch cost included except one_call_graph"
    return out


def order_measure(mw, wl, torch) -> dict:
    """Group-major receive order (Sections 4.3.1, 4.3.2) and expert index (Section 2.3.2) on the headline workload."""
    inp = wl.make_dispatch(WORKLOAD, payload=False)
    s = inp.shape
    B, T = s.row_bytes, s.T
    ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    with mw.Context(s.R, s.E, s.K, T, B) as ctx:
        ctx.mw_plan(ids, e2r, T)
        tot = ctx.mw_get_totals()
        Tn, SD = tot["T_nonempty"], tot["total_dest"]
        ctx.mw_group_major()
        sends = [torch.empty(Tn * B, dtype=torch.uint8, device="cuda").random_(0, 256) for _ in range(2)]
        recvs = [torch.empty(SD * B, dtype=torch.uint8, device="cuda") for _ in range(2)]
        off = torch.empty(s.E + 1, dtype=torch.int32, device="cuda")
        tok = torch.empty(T * s.K, dtype=torch.int32, device="cuda")
        slot = torch.empty(T * s.K, dtype=torch.int32, device="cuda")
        cases = (("group_major_arrays_us", lambda i: ctx.mw_group_major(), 200),
                 ("deliver_group_major_us", lambda i: ctx.mw_deliver_group_major(sends[i % 2], recvs[i % 2], 0, SD), 100),
                 ("expert_index_us", lambda i: ctx.mw_expert_index(ids, e2r, off, tok, slot), 200))
        out = {}
        for name, fn, n in cases:
            for i in range(5):
                fn(i)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(n):
                fn(i)
            b.record()
            torch.cuda.synchronize()
            out[name] = round(a.elapsed_time(b) * 1e3 / n, 1)
        assert ctx.mw_get_totals()["status"] == 0
    out["deliver_group_major_gbs"] = round((Tn + SD) * B / out["deliver_group_major_us"] / 1e3, 1)
    out["groups"] = tot["G"]
    out["note"] = "1 + 2 short kernels over the plan (latency-bound); the deliver is the same row-copy kernel with other slots"
    return out


def combine_measure(mw, wl, torch) -> dict:
    """Combine (Section 2.3.2) on the dsv3_prefill routing: every destination returns one bf16 row per token."""
    inp = wl.make_dispatch(WORKLOAD, payload=False)
    s = inp.shape
    B, T = s.row_bytes, s.T
    ids, e2r = torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda()
    with mw.Context(s.R, s.E, s.K, T, B) as ctx:
        ctx.mw_plan(ids, e2r, T)
        SD = ctx.mw_get_totals()["total_dest"]
        Kd = min(s.K, s.R)
        zs = [torch.randn(SD * B // 2, dtype=torch.bfloat16, device="cuda") for _ in range(2)]     # 2 x 340 MB > L2
        ys = [torch.empty(T * B, dtype=torch.uint8, device="cuda") for _ in range(2)]
        w = torch.rand(T * Kd, dtype=torch.float32, device="cuda")
        for i in range(4):
            ctx.mw_combine(zs[i % 2], 0, w, ys[i % 2])
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 40
        a.record()
        for i in range(n):
            ctx.mw_combine(zs[i % 2], 0, w, ys[i % 2])
        b.record()
        torch.cuda.synchronize()
        us = a.elapsed_time(b) * 1e3 / n
    moved = (SD + T) * B + T * Kd * 4
    return {"rows_read": SD, "rows_written": T, "us": round(us, 1), "gbs": round(moved / us / 1e3, 1),
            "note": "bf16 rows, fp32 accumulation; bytes = rows read + rows written + weights"}


def paired_allgather_measure(mw, torch) -> list:
    """Paired-relay AllGather (Sections 3.1, 5.2): 8 ranks, two TP=4 domains, 16 MB per rank (the paper's size)."""
    R, S = 8, 16 << 20
    n = R // 2
    out = []
    with mw.Context(R, 8, 2, 16, 32) as ctx:
        shards = torch.empty(R * S, dtype=torch.uint8, device="cuda").random_(0, 256)
        recv = torch.empty(R * n * S, dtype=torch.uint8, device="cuda")
        relay = torch.empty(R * (n - 1) * S, dtype=torch.uint8, device="cuda")
        cases = (("direct only", mw.MW_LAYOUT_MULTIWRITE, S),
                 ("unicast relay", mw.MW_LAYOUT_UNICAST, mw.mw_pair_balanced_direct_bytes(S, n, mw.MW_LAYOUT_UNICAST)),
                 ("multiwrite relay", mw.MW_LAYOUT_MULTIWRITE, mw.mw_pair_balanced_direct_bytes(S, n, mw.MW_LAYOUT_MULTIWRITE)))
        for name, layout, direct in cases:
            tot = None
            for _ in range(3):
                _, tot = ctx.mw_paired_allgather(shards, S, direct, layout, relay, recv)
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(10)]
            torch.cuda.synchronize()
            for a, b in evs:
                a.record()
                ctx.mw_paired_allgather(shards, S, direct, layout, relay, recv)
                b.record()
            torch.cuda.synchronize()
            us = statistics.median(a.elapsed_time(b) for a, b in evs) * 1e3
            copies = 1 if layout == mw.MW_LAYOUT_MULTIWRITE else n - 1
            moved = R * ((1 + n) * direct + (S - direct) * (1 + copies + 1) + (n - 1) * 2 * (S - direct)) if direct < S \
                else R * (1 + n) * S
            out.append({"scheme": name, "direct_bytes": direct, "p50_us": round(us, 1), "gbs": round(moved / us / 1e3, 1),
                        "max_link_mb": round(tot["max_link_bytes"] / 1e6, 2),
                        "model_time_vs_direct_only": round(tot["max_link_bytes"] / S, 4)})
    return out


def bytes_saved(wl) -> dict:
    """Transmitted-byte savings of the MultiWrite layout, exact integers from the plan (device side)."""
    import torch
    from paper_2605_22428_b200 import binding as mw
    out = {}
    for shape in wl.DISPATCH_SHAPES:
        inp = wl.make_dispatch(shape.name, payload=False)
        with mw.Context(shape.R, shape.E, shape.K, shape.T, shape.row_bytes) as ctx:
            ctx.mw_plan(torch.from_numpy(inp.topk_ids).cuda(), torch.from_numpy(inp.expert_to_rank).cuda(), shape.T)
            tot = ctx.mw_get_totals()
        out[shape.name] = round(100.0 * (1 - tot["mw_bytes"] / tot["unicast_bytes"]), 3)
    R = wl.ALLGATHER_R
    out["allgather_r64"] = round(100.0 * (1 - 1 / (R - 1)), 3)
    return out


def aggregate_over_ranks(dist, total_ms: float, e2e_ms: float, step_bytes: float, device):
    """Replicas only: times are the maximum over ranks, work is the sum over ranks (no data-path collective)."""
    if dist is None:
        return total_ms, e2e_ms, step_bytes
    import torch
    v = torch.tensor([total_ms, e2e_ms], dtype=torch.float64, device=device)
    dist.all_reduce(v, op=dist.ReduceOp.MAX)
    units = torch.tensor([step_bytes], dtype=torch.float64, device=device)
    dist.all_reduce(units, op=dist.ReduceOp.SUM)
    return float(v[0]), float(v[1]), float(units[0])


def run_cuda(args):
    import torch
    from paper_2605_22428_b200 import binding as mw
    from paper_2605_22428_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation of the path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    workload = WORKLOAD
    if args.profile_workload:
        if not args.kernels_only:
            raise SystemExit("--profile-workload goes with --kernels-only (the benchmark line is always quoted on " + WORKLOAD + ")")
        workload = args.profile_workload
    inp = wl.make_dispatch(workload, seed=1 + 1000 * rank if rank else None)
    s = inp.shape
    B, T = s.row_bytes, s.T
    ids = torch.from_numpy(inp.topk_ids).cuda()
    e2r = torch.from_numpy(inp.expert_to_rank).cuda()
    ctx = mw.Context(s.R, s.E, s.K, T, B, device=local, flags=args.flags)
    ctx.mw_plan(ids, e2r, T)
    tot = ctx.mw_get_totals()
    assert tot["status"] == 0, tot
    Tn, SD = tot["T_nonempty"], tot["total_dest"]
    alg = algorithmic_bytes(tot, B)
    # buffer sets cycled step by step: 3 x (x 59 MB + send 59 MB + recv 450 MB) = 1.7 GB >> 126 MB of L2
    nsets = 3
    x_host = torch.from_numpy(inp.x.view(np.int16))
    sets = [(x_host.cuda(), torch.empty(Tn * B, dtype=torch.uint8, device="cuda"),
             torch.empty(SD * B, dtype=torch.uint8, device="cuda")) for _ in range(nsets)]

    def step(i, evs=None):
        x, send, recv = sets[i % nsets]
        if evs:
            evs[0].record()
        if args.no_prefetch:
            ctx.mw_plan(ids, e2r, T)
        else:
            ctx.mw_plan_prefetch(ids, e2r, T, x)      # the same plan; idle SMs bring x into L2 meanwhile
        if evs:
            evs[1].record()
        ctx.mw_pack(x, mw.MW_LAYOUT_MULTIWRITE, send, Tn)
        if evs:
            evs[2].record()
        ctx.mw_deliver(mw.MW_LAYOUT_MULTIWRITE, send, recv, 0, SD)
        if evs:
            evs[3].record()

    sampler = ClockSampler(local)
    sampler.start()
    for i in range(max(args.warmup, 3)):
        step(i)
    # Stage events sit between kernels and so switch off the overlap of one kernel's start-up with the
    # previous kernel's tail; they are recorded on every 8th step only (always on the first), and the
    # per-kernel durations below are means over those sampled steps of the timed region.
    sampled = [i for i in range(args.steps) if i % 8 == 0]
    evs = {i: [torch.cuda.Event(enable_timing=True) for _ in range(4)] for i in sampled}
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
        torch.cuda.synchronize()
    launches0 = ctx.mw_kernel_launches()
    t0 = time.perf_counter()
    e_begin.record()
    for i in range(args.steps):
        step(i, evs.get(i))
    e_end.record()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    if dist:
        dist.barrier()
        torch.cuda.synchronize()
    launches = ctx.mw_kernel_launches() - launches0
    total_ms = e_begin.elapsed_time(e_end)
    assert ctx.mw_get_totals()["status"] == 0
    plan_ms = [e[0].elapsed_time(e[1]) for e in evs.values()]
    pack_ms = [e[1].elapsed_time(e[2]) for e in evs.values()]
    deliver_ms = [e[2].elapsed_time(e[3]) for e in evs.values()]
    # the roofline kernel's duration does not depend on --steps: 20 warm-up + 200 timed launches of their own, each after
    # the plan and pack launches of its step
    roof_ms = time_deliver_launches(ctx, mw, torch, ids, e2r, T, sets, Tn, SD, launches=50 if args.kernels_only else 200)

    if args.kernels_only:
        sampler.stop()
        print(json.dumps({"kernels_only": True, "ms_per_step": total_ms / args.steps, "steps": args.steps,
                          "deliver_launch_mean_us": statistics.mean(roof_ms) * 1e3,
                          "combine": combine_measure(mw, wl, torch),
                          "stages_us": {"plan": statistics.mean(plan_ms) * 1e3, "pack": statistics.mean(pack_ms) * 1e3,
                                        "deliver": statistics.mean(deliver_ms) * 1e3}}))
        ctx.close()
        return 0

    # ---- end to end from host buffers (pinned), copies inside the timed region ----
    ctx_h = mw.Context(s.R, s.E, s.K, T, B, device=local, flags=mw.MW_FLAG_HOST_STAGING)
    ids_h, e2r_h = torch.from_numpy(inp.topk_ids).pin_memory(), torch.from_numpy(inp.expert_to_rank).pin_memory()
    x_h = x_host.pin_memory()
    recv_h = torch.empty(SD * B, dtype=torch.uint8).pin_memory()
    ro_h = torch.empty(s.R + 1, dtype=torch.int32).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        ctx_h.mw_dispatch_host(ids_h, e2r_h, x_h, T, mw.MW_LAYOUT_MULTIWRITE, recv_h, SD, ro_h)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    th0 = time.perf_counter()
    for _ in range(e2e_steps):
        ctx_h.mw_dispatch_host(ids_h, e2r_h, x_h, T, mw.MW_LAYOUT_MULTIWRITE, recv_h, SD, ro_h)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - th0) * 1e3 / e2e_steps
    sampler.stop()
    launches += 0  # end-to-end launches are outside the timed region and not counted
    ctx_h.close()

    total_ms, e2e_ms, step_bytes_all = aggregate_over_ranks(dist, total_ms, e2e_ms, float(alg["step"]),
                                                            torch.device("cuda", local))

    ms_per_step = total_ms / args.steps
    value = step_bytes_all / (ms_per_step * 1e-3) / 1e9
    peak, peak_src = measured_peak()
    d_ms, p_ms = statistics.mean(deliver_ms), statistics.mean(pack_ms)
    roof = roofline_block("k_copy_rows<1, SCATTER, after pack> (deliver, MultiWrite layout)", alg["deliver"], roof_ms,
                          recorded_traffic(WORKLOAD), peak, peak_src)
    roof["timed_region_mean_us"] = round(d_ms * 1e3, 2)
    roof["timed_region_samples"] = len(evs)
    stages = {"plan": round(statistics.mean(plan_ms) * 1e3, 2), "pack": round(p_ms * 1e3, 2), "deliver": round(d_ms * 1e3, 2),
              "pack_gbs": round(alg["pack"] / p_ms / 1e6, 1),
              "pack_plus_deliver_gbs": round((alg["pack"] + alg["deliver"]) / (p_ms + d_ms) / 1e6, 1),
              "sampled_steps": len(evs), "note": "CUDA events on every 8th step of the timed region"}
    if roof["traffic"]:
        # the same two launches counted in DRAM bytes: pack reads and writes every row once, deliver as ncu recorded it
        dram = (alg["pack"] + roof["traffic"]) / (p_ms + d_ms) / 1e6
        stages["pack_plus_deliver_dram_gbs"] = round(dram, 1)
        stages["pack_plus_deliver_dram_frac_of_nominal_8TBs"] = round(dram / NOMINAL_HBM_GBS, 4)
        # the whole step in DRAM bytes (plan traffic is under 1 MB): what `value` is in the other byte counting
        stages["step_dram_gbs"] = round((alg["pack"] + roof["traffic"]) / (ms_per_step * 1e-3) / 1e9, 1)
    line = {
        "metric": METRIC, "value": round(value, 2), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "R": s.R, "E": s.E, "K": s.K, "T": T, "row_bytes": B, "layout": "multiwrite",
                   "parallelism": "replicas only" if world > 1 else "1 gpu",
                   "step": ("mw_plan" if args.no_prefetch else "mw_plan_prefetch") + " + mw_pack + mw_deliver (three kernel launches)",
                   "l2": f"cycles over {nsets} buffer sets of {(2 * Tn + SD) * B / 1e6:.0f} MB each (larger than the 126 MB L2)",
                   "rows_packed": Tn, "rows_delivered": SD, "groups": tot["G"],
                   "algorithmic_bytes_per_step": alg["step"]},
        "tokens_per_s": round(T * world / (ms_per_step * 1e-3), 1),
        "fraction_of_measured_peak": round(value / world / peak, 4),
        "fraction_of_nominal_8TBs": round(value / world / NOMINAL_HBM_GBS, 4),
        "stages_us": stages,
        "roofline": roof,
        "e2e": {"value": round(step_bytes_all / (e2e_ms * 1e-3) / 1e9, 3), "unit": "GB/s", "ms_per_step": round(e2e_ms, 3),
                "h2d_bytes_per_step": int(ids_h.numel() * 4 + e2r_h.numel() * 4 + T * B),
                "d2h_bytes_per_step": int(SD * B + (s.R + 1) * 4 + 64), "steps": e2e_steps,
                "api": "mw_dispatch_host (pinned host buffers; plan + pack + deliver + copies)"},
        "gpu_launches": int(launches),
        "clocks": sampler.summary(t0, t1),
        "bytes_saved_pct_this_workload": round(100.0 * (1 - tot["mw_bytes"] / tot["unicast_bytes"]), 3),
    }
    ctx.close()
    if rank == 0 and world == 1:
        del sets
        torch.cuda.empty_cache()
        line["cpu_baseline"] = cpu_baseline(inp, s.R, B)
        line["paper_context"] = "paper reports up to 33% lower operator latency on Ascend 910B (other hardware; not a target)"
        if not args.no_extras:
            line["allgather_r64"] = allgather_sweep(mw, wl, torch)
            line["relay_two_level"] = relay_measure(mw, wl, torch)
            line["paper_setup_2x8"] = paper_setup_measure(mw, wl, torch)
            line["paired_allgather_8x16MB"] = paired_allgather_measure(mw, torch)
            line["combine_dsv3_prefill"] = combine_measure(mw, wl, torch)
            line["dispatch_fused"] = fused_dispatch_measure(mw, wl, torch)
            line["receiver_order"] = order_measure(mw, wl, torch)
            line["mid_batches"] = mid_batch_measure(mw, wl, torch)
            # the keys the metric names come last
            line["tiny"] = tiny_measure(mw, wl, torch)
            line["unicast"] = {name: unicast_measure(mw, wl, torch, name) for name in (WORKLOAD, "large_ep")}
            line["large_ep"] = large_ep_measure(mw, wl, torch)
            line["pipelined"] = {name: pipelined_measure(mw, wl, torch, name) for name in (WORKLOAD, "large_ep")}
            line["bytes_saved_pct"] = bytes_saved(wl)
            line["decode"] = decode_latency(mw, wl, torch)
            # the three parts of the metric once more, compactly, as the very end of the line
            dec, pipe, uni, lep = line["decode"], line["pipelined"], line["unicast"], line["large_ep"]
            line["metric_summary"] = {
                "pack_plus_deliver_gbs": {WORKLOAD: stages["pack_plus_deliver_gbs"], "large_ep": lep["pack_plus_deliver_gbs"]},
                "pack_plus_deliver_pct_of_measured_peak": {WORKLOAD: round(100 * stages["pack_plus_deliver_gbs"] / peak, 1),
                                                           "large_ep": round(100 * lep["pack_plus_deliver_gbs"] / peak, 1)},
                "pack_plus_deliver_pct_of_nominal_8TBs": {WORKLOAD: round(100 * stages["pack_plus_deliver_gbs"] / NOMINAL_HBM_GBS, 1),
                                                          "large_ep": round(100 * lep["pack_plus_deliver_gbs"] / NOMINAL_HBM_GBS, 1)},
                "pack_plus_deliver_dram_pct_of_nominal_8TBs": round(100 * stages.get("pack_plus_deliver_dram_frac_of_nominal_8TBs", 0), 1) or None,
                "deliver_roofline_frac": {WORKLOAD: roof["frac"], "large_ep": lep["roofline"]["frac"]},
                "deliver_dram_frac": {WORKLOAD: roof.get("dram_frac"), "large_ep": lep["roofline"].get("dram_frac")},
                "step_us": {WORKLOAD: round(ms_per_step * 1e3, 2), "large_ep": lep["step_us"]},
                "pipelined_step_p50_us": {k: v["step_p50_us"] for k, v in pipe.items()},
                "unicast_vs_multiwrite_step_us": {k: [v["unicast"]["step_us"], v["multiwrite"]["step_us"]] for k, v in uni.items()},
                "tokens_per_s": line["tokens_per_s"],
                "decode_us": {"one_call_p50": dec["one_call"]["p50_us"], "one_call_p99": dec["one_call"]["p99_us"],
                              "graph_p50": dec["one_call_graph"]["p50_us"], "graph_p99": dec["one_call_graph"]["p99_us"],
                              "graph_chained_per_call": dec["one_call_graph_chained"]["p50_us"],
                              "plan_p50": dec["plan"]["p50_us"], "three_launch_chain_p50": dec["chain"]["p50_us"]},
                "tiny_one_call_p50_us": line["tiny"]["one_call"]["p50_us"],
                "bytes_saved_pct": line["bytes_saved_pct"]}
    if rank == 0:
        print(json.dumps(line))
    if dist:
        dist.destroy_process_group()
    return 0


def selftest_aggregate(args):
    """Launcher and aggregation check without a GPU (gloo on the CPU): every rank contributes made-up figures, rank 0
    prints what the real run would print from them."""
    import torch
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    total, e2e, units = aggregate_over_ranks(dist if world > 1 else None, 10.0 + rank, 100.0 - rank, 1000.0 * (rank + 1),
                                             torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"selftest": "aggregate", "n_gpus": world, "total_ms": total, "e2e_ms": e2e, "units": units}))
    if world > 1:
        dist.destroy_process_group()
    return 0


def launch_ranks(n: int) -> int:
    """Starts n ranks of this script on this node through torch.distributed.run (one per GPU; 127.0.0.1 rendezvous) and
    returns its exit code.  Used when the script is started plainly with --gpus n > 1."""
    import socket
    import subprocess
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the decode-latency and bytes-saved extras")
    ap.add_argument("--flags", type=lambda v: int(v, 0), default=0, help="MW_FLAG_* bits for the timed context")
    ap.add_argument("--kernels-only", action="store_true",
                    help="only the device-timed steps (for profiler runs): no end-to-end leg, extras or CPU baseline")
    ap.add_argument("--no-prefetch", action="store_true",
                    help="plan with mw_plan instead of mw_plan_prefetch (hidden rows not brought into L2 while planning)")
    ap.add_argument("--profile-workload", default="", help="with --kernels-only: run that dispatch shape instead (profiler captures)")
    ap.add_argument("--relay-only", type=int, default=0, metavar="STEPS",
                    help="only the two-level relayed dispatch measurement with this many timed steps (for profiler runs)")
    ap.add_argument("--selftest-aggregate", action="store_true",
                    help="no GPU work: check the rank launcher and the max/sum aggregation over ranks on the CPU (gloo)")
    ap.add_argument("--decode-only", type=int, default=0, metavar="LAUNCHES",
                    help="only the decode-shape latency measurement with this many launches per figure (for profiler runs)")
    args = ap.parse_args()
    if args.decode_only > 0 and args.impl == "cuda":
        import torch
        from paper_2605_22428_b200 import binding as mw
        from paper_2605_22428_b200 import workloads as wl
        torch.cuda.set_device(0)
        print(json.dumps({"decode_only": True, "decode": decode_latency(mw, wl, torch, args.decode_only)}))
        return 0
    if args.relay_only and args.impl == "cuda":
        import torch
        from paper_2605_22428_b200 import binding as mw
        from paper_2605_22428_b200 import workloads as wl
        torch.cuda.set_device(0)
        print(json.dumps({"relay_only": True, "relay_two_level": relay_measure(mw, wl, torch, n=args.relay_only)}))
        return 0
    if args.steps < 1:
        raise SystemExit("--steps must be >= 1")
    if args.impl == "reference":
        return run_reference(args)                  # rank 0 alone works; started plainly it is the only process
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return launch_ranks(args.gpus)              # one replica per GPU
    if args.selftest_aggregate:
        return selftest_aggregate(args)
    return run_cuda(args)


if __name__ == "__main__":
    sys.exit(main())
