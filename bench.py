#!/usr/bin/env python
"""Benchmark of the whole hot path: build the load-look-ahead maps, route arrivals, advance decode
iterations, on the seeded synthetic configurations.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 0..4]

Configurations 0-3 are one-shot: one "step" = pre_anticipate + pre_route_batch (the whole batch) +
pre_step.  Configuration 4 is the stream: one "step" = one scheduler tick (pre_step, then
pre_route_batch of that tick's arrivals), after one pre_anticipate on the initial table.
The default run times configuration 3 (4,096 instances, H = 2,048, 2,097,152 in-flight requests,
65,536 arrivals), checks what it timed against the CPU oracle, and adds one short entry per
configuration under "configs".

Prints ONE JSON line on rank 0.  `--impl reference` times the CPU oracle instead (a deliberately
plain sequential program) on a bounded sample of the same workload.  `--gpus N` without a
launcher starts N worker processes itself (independent replicas, one per GPU).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "routes/sec over the whole step (anticipate + route batch + decode step)"
METRIC_STREAM = "routes/sec over the whole stream (decode step + routing of the tick's arrivals, per tick)"

# DRAM bytes (read + write) per launch from the ncu captures summarised under profiles/ (configuration 3; other
# configurations report null).  profiles/ncu_full_route_scan_kernel_config3_256_arrivals.txt: the scanning routing kernel
# reads the maps once per launch, whatever the batch length (67.32 MB), and wrote 688,640 B for 256 arrivals
# (folded cells, appended requests): the written part is scaled to the batch.  The single-launch build reads the
# table and moves the tiles' lists; most of the 64 MiB of maps is still in L2 when the launch ends, which is why
# its figure is below the algorithmic bytes.  pre_step: its two kernels added.
# profiles/ncu_full_tick_scaler_refine_config3.txt: refinement and the fused tick (two kernels added).
ROUTE_DRAM_READ = {3: 67322880}
# profiles/ncu_dram_route_summary_kernels_config3_full_batch.txt: both kernels of the summary router on the full
# batch (the traffic does not grow in proportion to the batch, so the figure is used for the full batch only)
ROUTE_SUMMARY_DRAM_TRAFFIC = {(3, 65536): 67724288 + 116224 + 55949824 + 5290240}
# warp instructions per arrival of pre_route_summaries (smsp__inst_executed.sum of the 2,048-arrival capture in
# profiles/ncu_full_step_kernels_config3_2048_arrivals.txt: 9,365,991 / 2,048)
ROUTE_SUMMARY_WARP_INSTRUCTIONS_PER_ARRIVAL = {3: 9365991 / 2048}
ROUTE_DRAM_WRITE_PER_ARRIVAL = {3: 679168 / 256}
ANTICIPATE_DRAM_TRAFFIC = {3: 33808640 + 21654272}
STEP_DRAM_TRAFFIC = {3: 33668864 + 67196416 + 8912640}
SCALER_DRAM_TRAFFIC = {3: 67127552 + 291584}   # profiles/ncu_full_scaler_rows_config3.txt
REFINE_DRAM_TRAFFIC = {3: 44151040 + 25344}
TICK_DRAM_TRAFFIC = {3: 44137216 + 46080 + 67199744 + 9207552}


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) == 6:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm = [float(r[0]) for r in self.rows if r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for k, n in enumerate(names) if any(r[2 + k].lower().startswith("active") for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(self.rows)}


def algorithmic_bytes(wl, n_table_after):
    """Bytes each call must move by its definition (not what an implementation happens to move)."""
    n, a, i, h = wl.n_requests, wl.n_arrivals, wl.n_instances, wl.horizon
    build = 16 * n + 8 * i * h + 8 * i                       # read the table, write the maps
    route = a * (8 * i * h + 16 * h + 16 * i)                # literal scan per arrival + fold + scalars
    step = 16 * i * h + 16 * n_table_after                   # shift the maps, one pass over the table
    return build, route, step


def config_dict(wl, index, streaming_ticks=None):
    if wl.streaming:
        what = (f"config {index} ({wl.name}): {wl.n_instances} instances, H={wl.horizon}, {wl.n_requests} initial "
                f"in-flight requests, {len(wl.ticks)} ticks, {wl.n_arrivals} arrivals in all")
    else:
        what = (f"config {index} ({wl.name}): {wl.n_instances} instances, H={wl.horizon}, "
                f"{wl.n_requests} in-flight requests, {wl.n_arrivals} arrivals in one batch")
    return {"workload": what, "capacity_tokens": wl.capacity_tokens, "t_mem": wl.t_mem, "beta": wl.beta,
            "l2": "flushed between steps by writing a 512 MiB buffer" if not wl.streaming else
                  "not flushed between ticks: a tick's calls follow each other as in service (the maps, 8 MiB, stay in L2)",
            "timing": "CUDA events around each C-ABI call on the launching stream; state reset and L2 flush "
                      "between steps are not timed"}


# ----------------------------------------------------------------------------- CPU oracle legs

def oracle_sample(wl, n_route):
    """Times the oracle, as it stands, on a bounded sample of a one-shot configuration (literal routing of the
    first n_route arrivals).  Returns seconds per part."""
    import oracle
    ref = oracle.State.from_workload(wl)
    t0 = time.perf_counter()
    ref.anticipate()
    t1 = time.perf_counter()
    ap, ad = wl.ticks[0]
    ref.route_batch(ap[:n_route], ad[:n_route])
    t2 = time.perf_counter()
    ref.step()
    t3 = time.perf_counter()
    return t1 - t0, t2 - t1, t3 - t2


def oracle_stream_sample(wl, n_ticks):
    """The same for the streaming configuration: the first n_ticks ticks (running-maxima mode of the oracle,
    which is admitted by equality with its literal mode; the literal mode needs minutes per tick here)."""
    import oracle
    ref = oracle.State.from_workload(wl)
    t0 = time.perf_counter()
    ref.anticipate()
    t1 = time.perf_counter()
    routed = 0
    for ap, ad in wl.ticks[:n_ticks]:
        ref.step()
        ref.route_batch(ap, ad, fast=True)
        routed += len(ap)
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1, routed


def oracle_full_step(wl):
    """One whole step of a one-shot configuration in the oracle (routing in its running-maxima mode for
    configuration 3, where the literal mode needs hours; literal below).  Returns the state, the decisions and
    the seconds per part: this is both the expected value of the parity check and a measured CPU baseline."""
    import oracle
    ref = oracle.State.from_workload(wl)
    fast = wl.n_instances * wl.horizon * wl.n_arrivals > 8e9
    t0 = time.perf_counter()
    ref.anticipate()
    t1 = time.perf_counter()
    ap, ad = wl.ticks[0]
    choice, score = ref.route_batch(ap, ad, fast=fast)
    t2 = time.perf_counter()
    ref.step()
    t3 = time.perf_counter()
    return ref, choice, score, (t1 - t0, t2 - t1, t3 - t2), fast


def run_reference(args, wl, rank):
    """The reference arm: the CPU oracle on the host cores; rank 0 only."""
    if rank != 0:
        return
    if wl.streaming:
        n_ticks = max(1, min(len(wl.ticks), args.ref_ticks))
        per_step, routed = [], 0
        for _ in range(args.steps):
            tb, tt, routed = oracle_stream_sample(wl, n_ticks)
            per_step.append(tt)
        t = float(np.mean(per_step))
        value = routed / t
        sample = (f"per step: the first {n_ticks} of {len(wl.ticks)} ticks ({routed} arrivals), decode step + routing "
                  f"in the oracle's running-maxima mode")
        metric = METRIC_STREAM
    else:
        n_route = min(wl.n_arrivals, args.ref_arrivals)
        for _ in range(min(args.warmup, 1)):
            oracle_sample(wl, min(n_route, 8))
        per_step, values = [], []
        for _ in range(args.steps):
            tb, tr, ts = oracle_sample(wl, n_route)
            per_step.append(tb + tr + ts)
            # routing cost is linear in the number of arrivals; the build and the decode step ran in full
            values.append(wl.n_arrivals / (tb + tr * (wl.n_arrivals / n_route) + ts))
        t = float(np.mean(per_step))
        value = float(np.mean(values))
        sample = (f"per step: anticipate over all {wl.n_requests} requests, literal routing of the first {n_route} of "
                  f"{wl.n_arrivals} arrivals, one decode step; ms_per_step is the time of that sample, value is "
                  f"arrivals / (whole-step time with the routing part scaled to the full batch)")
        metric = METRIC
    print(json.dumps({
        "impl": "reference", "metric": metric, "value": value, "unit": "routes/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int64+f64", "data": "synthetic",
        "config": config_dict(wl, args.config),
        "cpu_baseline": {"value": value, "unit": "routes/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "routes/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ----------------------------------------------------------------------------- several GPUs without a launcher

def spawn_workers(args):
    """`--gpus N` given to a plain `python bench.py`: start N copies of this script, one per GPU, with the
    environment a launcher would set.  Replicas only: the processes talk to each other for the timing protocol
    (barrier, maximum over ranks) and nothing else."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(args.gpus):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(args.gpus),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    rc = 0
    for p in procs:
        rc = max(rc, abs(p.wait()))
    return rc


# ----------------------------------------------------------------------------- GPU legs

def ev():
    import torch
    return torch.cuda.Event(enable_timing=True)


def roof_hbm(nbytes, ms, launches, traffic, kernel, **more):
    peak, peak_kind = measured_peak_gbs()
    gbs = nbytes / (ms * 1e-3) / 1e9
    return dict({"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                 "peak_kind": f"of {peak_kind}", "traffic": traffic, "algorithmic_bytes_per_launch": nbytes,
                 "ms_per_launch": ms, "launches_per_step": launches, "kernel": kernel}, **more)


def compare_with_oracle(st, ref, choice, score, want_choice, want_score):
    """Element by element: decisions and int64 state bit-exact, scores within 1e-12 relative."""
    got_c = choice.cpu().numpy()
    got_s = score.cpu().numpy()
    ok = bool((got_c == want_choice).all())
    routed = want_choice >= 0
    rel = np.abs(got_s[routed] - want_score[routed]) / np.maximum(np.abs(want_score[routed]), 1.0)
    ok = ok and (rel.size == 0 or float(rel.max()) <= 1e-12)
    ok = ok and bool((st.curves.cpu().numpy() == ref.curves).all())
    ok = ok and bool((st.current_d.cpu().numpy() == ref.current_d).all())
    ok = ok and bool((st.queued_p.cpu().numpy() == ref.queued_p).all())
    n = int(st.n_requests.item())
    ok = ok and n == int(ref.n[0]) and bool((st.generated[:n].cpu().numpy() == ref.generated[:n]).all())
    return ok


def bench_oneshot(args, wl, index, device, group, world, steps, warmup, headline):
    """Configurations 0-3.  Returns the measurements of the step and, for the headline run, of the separate calls."""
    import torch
    from paper_2504_03702_b200 import binding as B
    from paper_2504_03702_b200 import dist as D
    from paper_2504_03702_b200.state import DeviceState

    n0, a = wl.n_requests, wl.n_arrivals
    arr_p_host, arr_d_host = wl.ticks[0]
    st = DeviceState.from_workload(wl, device=device)
    if args.router == "scan":
        st.select_router(B.ROUTE_SCAN)
    pristine_generated = st.generated[:n0].clone()
    arr_p = torch.as_tensor(arr_p_host).to(device)
    arr_d = torch.as_tensor(arr_d_host).to(device)
    choice = torch.empty(a, dtype=torch.int32, device=device)
    score = torch.empty(a, dtype=torch.float64, device=device)
    n0_dev = torch.tensor([n0], dtype=torch.int64, device=device)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)

    def reset():
        st.generated[:n0].copy_(pristine_generated)
        st.n_requests.copy_(n0_dev)
        st.queued_p.zero_()
        flush.zero_()

    def calls():
        B.check(B.pre_anticipate(st.ctx, st.prompt, st.generated, st.predicted, st.instance, n0, st.curves,
                                 st.current_d), "pre_anticipate")
        yield
        B.check(B.pre_route_batch(st.ctx, arr_p, arr_d, a, st.curves, st.queued_p, st.current_d, st.prompt,
                                  st.generated, st.predicted, st.instance, st.n_requests, choice, score),
                "pre_route_batch")
        yield
        B.check(B.pre_step(st.ctx, st.prompt, st.generated, st.predicted, st.instance, st.n_requests, st.curves,
                           st.queued_p, st.current_d), "pre_step")
        yield

    def one_step():
        reset()
        e = [ev() for _ in range(4)]
        e[0].record()
        for k, _ in enumerate(calls()):
            e[k + 1].record()
        return e

    for _ in range(max(warmup, 0)):
        one_step()
    torch.cuda.synchronize()
    B.check(st.status(), "warm-up")

    sampler = ClockSampler(device.index or 0)
    D.barrier(group)
    torch.cuda.synchronize()
    sampler.start()
    wall0 = time.perf_counter()
    events = [one_step() for _ in range(steps)]
    torch.cuda.synchronize()
    D.barrier(group)
    wall1 = time.perf_counter()
    clocks = sampler.stop()
    B.check(st.status(), "timed steps")

    res = {"st": st, "choice": choice, "score": score, "clocks": clocks, "wall_s": wall1 - wall0}
    res["t_build"] = float(np.mean([e[0].elapsed_time(e[1]) for e in events]))
    res["t_route"] = float(np.mean([e[1].elapsed_time(e[2]) for e in events]))
    res["t_dstep"] = float(np.mean([e[2].elapsed_time(e[3]) for e in events]))
    res["t_step"] = D.max_over_ranks(res["t_build"] + res["t_route"] + res["t_dstep"], group, device)
    res["map_max"] = int(st.curves.max().item())
    res["route_kernel"] = "summary" if B.pre_route_select(st.ctx, B.ROUTE_SUMMARY) == B.PRE_OK and args.router != "scan" else "scan"
    B.check(B.pre_route_select(st.ctx, B.ROUTE_SCAN if args.router == "scan" else B.ROUTE_AUTO), "pre_route_select")
    # what the timed steps left behind, for the parity check (taken before anything else touches the state)
    res["snapshot"] = (choice.clone(), score.clone())
    res["reset"], res["flush"], res["arr"] = reset, flush, (arr_p, arr_d)
    if not headline:
        return res

    # end-to-end leg: host buffers in, host results out, copies inside the timed region
    host_table = [torch.as_tensor(np.ascontiguousarray(x)).pin_memory()
                  for x in (wl.prompt, wl.generated, wl.predicted, wl.instance)]
    host_arr = [torch.as_tensor(np.ascontiguousarray(x)).pin_memory() for x in (arr_p_host, arr_d_host)]
    host_choice = torch.empty(a, dtype=torch.int32).pin_memory()
    host_score = torch.empty(a, dtype=torch.float64).pin_memory()
    res["h2d"] = sum(t.numel() * t.element_size() for t in host_table + host_arr)
    res["d2h"] = host_choice.numel() * 4 + host_score.numel() * 8
    res["state_after_timed"] = None
    res["host_io"] = (host_table, host_arr, host_choice, host_score)
    return res


def e2e_leg(res, wl, steps, group, device):
    import torch
    from paper_2504_03702_b200 import binding as B
    from paper_2504_03702_b200 import dist as D
    st, choice, score = res["st"], res["choice"], res["score"]
    arr_p, arr_d = res["arr"]
    host_table, host_arr, host_choice, host_score = res["host_io"]
    n0, a = wl.n_requests, wl.n_arrivals
    ms = []
    for k in range(1 + steps):
        res["reset"]()
        e0, e1 = ev(), ev()
        e0.record()
        for dst, src in zip((st.prompt, st.generated, st.predicted, st.instance), host_table):
            dst[:n0].copy_(src, non_blocking=True)
        arr_p.copy_(host_arr[0], non_blocking=True)
        arr_d.copy_(host_arr[1], non_blocking=True)
        B.check(B.pre_anticipate(st.ctx, st.prompt, st.generated, st.predicted, st.instance, n0, st.curves,
                                 st.current_d), "pre_anticipate")
        B.check(B.pre_route_batch(st.ctx, arr_p, arr_d, a, st.curves, st.queued_p, st.current_d, st.prompt,
                                  st.generated, st.predicted, st.instance, st.n_requests, choice, score),
                "pre_route_batch")
        B.check(B.pre_step(st.ctx, st.prompt, st.generated, st.predicted, st.instance, st.n_requests, st.curves,
                           st.queued_p, st.current_d), "pre_step")
        host_choice.copy_(choice, non_blocking=True)
        host_score.copy_(score, non_blocking=True)
        e1.record()
        torch.cuda.synchronize()
        if k:  # the first one warms the pinned-copy path
            ms.append(e0.elapsed_time(e1))
    B.check(st.status(), "end-to-end steps")
    return D.max_over_ranks(float(np.mean(ms)), group, device), int((host_choice >= 0).sum())


def extras_leg(res, wl, index, device):
    """Separate calls, not part of the step: admission router, scaler signals, refinement, full-width maps."""
    import torch
    from paper_2504_03702_b200 import binding as B
    from paper_2504_03702_b200 import workloads as W
    from paper_2504_03702_b200.state import DeviceState
    st, choice, score, flush = res["st"], res["choice"], res["score"], res["flush"]
    arr_p, arr_d = res["arr"]
    n0, a = wl.n_requests, wl.n_arrivals
    out = {}

    def rebuild_and_route():
        res["reset"]()
        B.check(B.pre_anticipate(st.ctx, st.prompt, st.generated, st.predicted, st.instance, n0, st.curves,
                                 st.current_d), "pre_anticipate")

    # the same batch through the router with its admission queue (Sec. 4.3.3), the paper's overload levels
    rebuild_and_route()
    st.make_queue(4096)
    e0, e1 = ev(), ev()
    e0.record()
    _, adm_choice, _ = st.route_admit(arr_p, arr_d, overload_level=0.95, overload_share=0.10)
    e1.record()
    torch.cuda.synchronize()
    t_admit = e0.elapsed_time(e1)
    out["route_admit"] = {"routed": int((adm_choice >= 0).sum()), "waiting": int((adm_choice == -2).sum()),
                          "turned_away": int((adm_choice == -3).sum()), "ms": t_admit,
                          "decided_per_s": a / (t_admit * 1e-3),
                          "kernel": "pre_route_summaries<admit>" if res["route_kernel"] == "summary" else "pre_route_persistent<admit>",
                          "overload_level": 0.95, "overload_share": 0.10, "queue_capacity": 4096,
                          "note": "separate call, not part of the step; same batch, same maps"}
    B.check(st.status(), "admission call")
    # leave the state as the step leaves it (the calls below continue from there)
    rebuild_and_route()
    B.check(B.pre_route_batch(st.ctx, arr_p, arr_d, a, st.curves, st.queued_p, st.current_d, st.prompt,
                              st.generated, st.predicted, st.instance, st.n_requests, choice, score),
            "pre_route_batch")
    st.step()

    # the scanning kernel on the first arrivals of the same batch (it routes what the summary kernel declines)
    if res["route_kernel"] == "summary":
        n_scan = min(a, 8192)
        st.select_router(B.ROUTE_SCAN)
        rebuild_and_route()
        flush.zero_()
        e0, e1 = ev(), ev()
        e0.record()
        B.check(B.pre_route_batch(st.ctx, arr_p, arr_d, n_scan, st.curves, st.queued_p, st.current_d, st.prompt,
                                  st.generated, st.predicted, st.instance, st.n_requests, choice, score),
                "pre_route_batch (scanning kernel)")
        e1.record()
        torch.cuda.synchronize()
        B.check(st.status(), "scanning kernel")
        out["route_scan_sample"] = (e0.elapsed_time(e1), n_scan, int(st.curves.max().item()))
        st.select_router(B.ROUTE_AUTO)
        rebuild_and_route()
        B.check(B.pre_route_batch(st.ctx, arr_p, arr_d, a, st.curves, st.queued_p, st.current_d, st.prompt,
                                  st.generated, st.predicted, st.instance, st.n_requests, choice, score),
                "pre_route_batch")
        st.step()

    # scaler signals over the maps (Sec. 4.3.2)
    sc_ev = []
    for _ in range(5):
        flush.zero_()
        e0, e1 = ev(), ev()
        e0.record()
        st.scaler_signals()
        e1.record()
        sc_ev.append((e0, e1))
    torch.cuda.synchronize()
    t_scaler = float(np.median([x.elapsed_time(y) for x, y in sc_ev[1:]]))
    out["roofline_scaler_signals"] = roof_hbm(8 * wl.n_instances * wl.horizon + 12 * wl.n_instances, t_scaler, 1,
                                              SCALER_DRAM_TRAFFIC.get(index), "pre_scaler_rows",
                                              note="separate call, not part of the step")

    # misprediction refinement (Sec. 4.3.1): one pass over the table per tick against real lengths; also the
    # tick with the three passes in one call
    table_actual, tick_actual = W.make_actual(wl, W.BASE_SEED + index)
    actual = torch.zeros(wl.max_requests, dtype=torch.int32, device=device)
    actual[:n0] = torch.from_numpy(table_actual).to(device)
    actual[n0:n0 + a] = torch.from_numpy(tick_actual[0][:a]).to(device)
    rf_ev, st_ev, rf_counts = [], [], None
    for _ in range(5):
        flush.zero_()
        e0, e1, e2 = ev(), ev(), ev()
        e0.record()
        st.step()
        e1.record()
        rf_counts = st.refine(actual)
        e2.record()
        rf_ev.append((e1, e2))
        st_ev.append((e0, e1))
    torch.cuda.synchronize()
    t_refine = float(np.median([x.elapsed_time(y) for x, y in rf_ev[1:]]))
    t_step_here = float(np.median([x.elapsed_time(y) for x, y in st_ev[1:]]))
    rf_counts = [int(v) for v in rf_counts.cpu().tolist()]
    B.check(st.status(), "refinement ticks")
    out["roofline_refine"] = roof_hbm(20 * (n0 + a), t_refine, 1, REFINE_DRAM_TRAFFIC.get(index), "pre_refine_requests",
                                      events_last_tick={"early_finish": rf_counts[0], "extended": rf_counts[1]},
                                      note="separate call, not part of the step; timed right after pre_step of the same "
                                           "tick (table and maps partly in L2); bytes = five int32 columns of the table, "
                                           "the read-modify-write of the touched map cells is not counted")
    if hasattr(st, "tick"):
        tk_ev = []
        for _ in range(5):
            flush.zero_()
            e0, e1 = ev(), ev()
            e0.record()
            st.tick(actual)
            e1.record()
            tk_ev.append((e0, e1))
        torch.cuda.synchronize()
        t_tick = float(np.median([x.elapsed_time(y) for x, y in tk_ev[1:]]))
        out["tick_fused"] = {"tick_fused_ms": t_tick, "pre_step_alone_ms": t_step_here, "traffic": TICK_DRAM_TRAFFIC.get(index),
                             "separate_calls_ms": {"pre_step": t_step_here, "pre_refine": t_refine, "pre_scaler_signals": t_scaler},
                             "ratio_to_pre_step": t_tick / t_step_here,
                             "note": "pre_tick: decode step, refinement against real lengths and scaler signals in one pass "
                                     "over the table and one over the maps"}

    # full-width maps kept as a ring (Sec. 4.3.1), routed on the paper's window of 100 iterations
    ring_window = min(100, wl.horizon)
    ring_st = DeviceState(wl.n_instances, ring_window, wl.capacity_tokens, n0 + 2 * a, wl.t_mem, wl.beta,
                          device=device)
    ring_st.load_requests(wl.prompt, wl.generated, wl.predicted, wl.instance)
    ring_st.make_ring(wl.horizon)
    ring_ms = None
    for k in range(2):
        flush.zero_()
        e = [ev() for _ in range(5)]
        e[0].record()
        ring_st.ring_step()
        e[1].record()
        ring_st.ring_window()
        e[2].record()
        ring_choice, _ = ring_st.route_batch(arr_p, arr_d)
        e[3].record()
        ring_st.ring_fold(arr_p, arr_d, ring_choice)
        e[4].record()
        torch.cuda.synchronize()
        ring_ms = [e[i].elapsed_time(e[i + 1]) for i in range(4)]
    B.check(ring_st.status(), "ring tick")
    out["full_width_maps"] = {
        "width": wl.horizon, "window": ring_window, "routed": int((ring_choice >= 0).sum()),
        "tick_ms": {"pre_ring_step": ring_ms[0], "pre_ring_window": ring_ms[1], "pre_route_batch": ring_ms[2],
                    "pre_ring_fold": ring_ms[3]},
        "routes_per_s": a / (sum(ring_ms) * 1e-3),
        "note": "separate state, not part of the step: maps of the configuration's full width kept as a ring over "
                "absolute iterations, peaks taken over the next 100 iterations (the paper's l); one scheduler tick = "
                "decode step + window copy + routing of the batch + real update of the ring"}
    ring_st.close()
    return out


def bench_stream(args, wl, index, device, group, n_check_ticks):
    """Configuration 4: pre_anticipate once, then per tick pre_step + pre_route_batch of the tick's arrivals.
    Every call is timed with events; the first n_check_ticks ticks are compared with the oracle."""
    import torch
    from paper_2504_03702_b200 import binding as B
    from paper_2504_03702_b200 import dist as D
    from paper_2504_03702_b200.state import DeviceState
    st = DeviceState.from_workload(wl, device=device)
    if args.router == "scan":
        st.select_router(B.ROUTE_SCAN)
    arrs = [(torch.as_tensor(ap).to(device), torch.as_tensor(ad).to(device)) for ap, ad in wl.ticks]
    e_b0, e_b1 = ev(), ev()
    torch.cuda.synchronize()
    D.barrier(group)
    e_b0.record()
    st.anticipate()
    e_b1.record()
    evs, outs = [], []
    e_start = ev()
    e_start.record()
    for t, (ap, ad) in enumerate(arrs):
        e0, e1, e2 = ev(), ev(), ev()
        e0.record()
        st.step()
        e1.record()
        c, s = st.route_batch(ap, ad)
        e2.record()
        evs.append((e0, e1, e2))
        if t < n_check_ticks:
            outs.append((c, s))
    e_end = ev()
    e_end.record()
    torch.cuda.synchronize()
    D.barrier(group)
    B.check(st.status(), "stream")
    total_ms = e_start.elapsed_time(e_end)
    step_us = np.array([x.elapsed_time(y) for x, y, _ in evs]) * 1e3
    route_us = np.array([y.elapsed_time(z) for _, y, z in evs]) * 1e3
    n_arr = np.array([len(ap) for ap, _ in wl.ticks])
    res = {"total_ms": D.max_over_ranks(total_ms, group, device), "ticks": len(arrs), "arrivals": int(n_arr.sum()),
           "anticipate_us": e_b0.elapsed_time(e_b1) * 1e3, "step_us_median": float(np.median(step_us)),
           "route_call_us_median": float(np.median(route_us)),
           "route_us_per_arrival_median": float(np.median(route_us / np.maximum(n_arr, 1))),
           "table_rows_at_end": int(st.n_requests.item())}
    parity = None
    if n_check_ticks > 0:
        import oracle
        ref = oracle.State.from_workload(wl)
        ref.anticipate()
        parity = True
        for (c, s), (ap, ad) in zip(outs, wl.ticks[:n_check_ticks]):
            ref.step()
            wc, ws = ref.route_batch(ap, ad, fast=True)
            rel = np.abs(s.cpu().numpy() - ws) / np.maximum(np.abs(ws), 1.0)
            parity = parity and bool((c.cpu().numpy() == wc).all()) and float(rel.max()) <= 1e-12
    res["parity_checked"] = parity
    res["parity_ticks"] = n_check_ticks
    st.close()
    return res


def route_scan_roofline(wl, index, t_route_ms, n_arrivals, map_max, layout, route_blocks, clocks, n_sm):
    """The scanning routing kernel against the roof it runs under.  Every arrival scans every cell of every map, but the
    maps are copied into shared memory once per batch (32-bit cells when every value is below 2^32), so the roof
    is the shared-memory bandwidth of the SMs: 128 bytes per clock and SM at the sampled clock."""
    i, h = wl.n_instances, wl.horizon
    resident_bytes = layout[0]
    packed = map_max < (1 << 32) and h % 64 == 0
    cell = 4 if packed else 8
    rows_per_block = -(-i // route_blocks)
    resident_rows_block = min(rows_per_block, resident_bytes // (h * cell))
    resident_rows = min(i, resident_rows_block * route_blocks)
    smem_bytes = cell * resident_rows * h * n_arrivals               # read from shared memory
    l2_bytes = 8 * (i - resident_rows) * h * n_arrivals              # rows that did not fit: streamed from L2
    mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
    peak = n_sm * 128 * mhz * 1e6 / 1e9
    sec = t_route_ms * 1e-3
    achieved = smem_bytes / sec / 1e9
    literal = n_arrivals * (8 * i * h + 16 * h + 16 * i)
    traffic = None
    if index in ROUTE_DRAM_READ:
        traffic = int(ROUTE_DRAM_READ[index] + ROUTE_DRAM_WRITE_PER_ARRIVAL[index] * n_arrivals)
    hbm_peak, kind = measured_peak_gbs()
    return {
        "bound": "smem", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        "peak_kind": f"derived: {n_sm} SMs x 128 B/clk x {mhz:.0f} MHz (SM clock sampled during the timed region)",
        "traffic": traffic, "kernel": "pre_route_persistent", "us_per_arrival": sec * 1e6 / n_arrivals,
        "cells_scanned_per_arrival": i * h, "cell_bytes_in_shared_memory": cell,
        "rows_resident_in_shared_memory": resident_rows, "bytes_streamed_from_l2_per_launch": l2_bytes,
        "scan_equivalent_gbs": literal / sec / 1e9,
        "hbm_frac_of_captured_traffic": None if traffic is None else traffic / sec / 1e9 / hbm_peak,
        "limiter": "latency of the per-arrival exchange between the blocks through L2 (about 1.0-1.5 us from a block's "
                   "publication to every block having read it), not bandwidth",
        "note": "achieved = bytes the kernel reads from shared memory (cell size x resident cells x arrivals) over "
                "time; scan_equivalent_gbs is the literal formulation's 8 bytes per cell and arrival over time, a "
                "convenience number that is not memory traffic; traffic = DRAM bytes of the launch from the ncu "
                f"capture scaled to this batch ({kind} HBM peak {hbm_peak:.0f} GB/s for hbm_frac_of_captured_traffic)"}


def route_summary_roofline(wl, index, t_route_ms, n_arrivals, clocks):
    """The summary routing kernel.  One block on one SM: per arrival it reads the rows' summaries from shared
    memory (8 bytes per instance), reads and rewrites the receiving row in the map (16 bytes per step), and is
    bound by the latency of its rounds (two block barriers and the dependent steps of a decision), not by any
    bandwidth.  Where the instructions per arrival are known from an ncu capture the roof quoted is the instruction
    issue of the ONE SM the block runs on, else that SM's shared-memory bandwidth."""
    i, h = wl.n_instances, wl.horizon
    ip = (i + 31) // 32 * 32
    mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
    peak = 128 * mhz * 1e6 / 1e9
    sec = t_route_ms * 1e-3
    smem_bytes = 8 * ip * n_arrivals
    achieved = smem_bytes / sec / 1e9
    literal = n_arrivals * (8 * i * h + 16 * h + 16 * i)
    traffic = ROUTE_SUMMARY_DRAM_TRAFFIC.get((index, n_arrivals))
    hbm_peak, kind = measured_peak_gbs()
    out = {
        "traffic": traffic, "kernel": "pre_summarise_rows + pre_route_summaries", "us_per_arrival": sec * 1e6 / n_arrivals,
        "bytes_of_shared_memory_read_per_arrival": 8 * ip, "bytes_of_map_read_and_written_per_arrival": 16 * h,
        "smem_gbs": achieved, "smem_peak_gbs_of_the_one_sm": peak, "smem_frac": achieved / peak,
        "scan_equivalent_gbs": literal / sec / 1e9,
        "hbm_frac_of_captured_traffic": None if traffic is None else traffic / sec / 1e9 / hbm_peak,
        "limiter": "latency: every arrival is one round of the block (two block barriers, the scoring pass, the "
                   "dependent steps of the decision); neither a memory nor the instruction issue is saturated",
        "note": "the kernel decides from four numbers per row instead of scanning the maps (identical decisions) and "
                "runs as ONE block; smem_* = bytes of row summaries read from shared memory over time against 128 "
                f"B/clk x {mhz:.0f} MHz of the one SM it occupies; scan_equivalent_gbs is the literal formulation's 8 "
                "bytes per cell and arrival over time, a convenience number that is not memory traffic; traffic = DRAM "
                f"bytes of both kernels from the ncu capture of this batch ({kind} HBM peak {hbm_peak:.0f} GB/s for "
                "hbm_frac_of_captured_traffic)"}
    inst = ROUTE_SUMMARY_WARP_INSTRUCTIONS_PER_ARRIVAL.get(index)
    if inst is not None:
        # not memory-bound: the roof is the instruction issue of the SM the block runs on, 4 warp instructions per clock
        issue_peak = 4 * mhz * 1e6 / 1e9
        issued = inst * n_arrivals / sec / 1e9
        out.update({"bound": "alu", "achieved": issued, "peak": issue_peak, "unit": "G warp-instructions/s",
                    "frac": issued / issue_peak,
                    "peak_kind": f"derived: 1 SM x 4 schedulers x 1 warp instruction per clock x {mhz:.0f} MHz (SM clock "
                                 "sampled during the timed region)",
                    "warp_instructions_per_arrival": inst})
    else:
        out.update({"bound": "smem", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "peak_kind": f"derived: 1 SM x 128 B/clk x {mhz:.0f} MHz (the kernel is one block; SM clock sampled "
                                 "during the timed region)"})
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, choices=[0, 1, 2, 3, 4])
    ap.add_argument("--ref-arrivals", type=int, default=256, help="arrivals routed per step by the reference arm")
    ap.add_argument("--ref-ticks", type=int, default=4, help="ticks per step of the reference arm on the stream")
    ap.add_argument("--cpu-arrivals", type=int, default=600, help="arrivals routed literally by the cpu_baseline leg")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle legs (no parity check either)")
    ap.add_argument("--no-extras", action="store_true", help="skip the separate calls and the per-configuration entries")
    ap.add_argument("--router", default="auto", choices=["auto", "scan"],
                    help="auto: the summary routing kernel where the shape fits it; scan: always the scanning kernel")
    ap.add_argument("--stream-ticks", type=int, default=0, help="shorten the stream to this many ticks (0: all 1,000)")
    ap.add_argument("--arrivals", type=int, default=0,
                    help="route only the first ARRIVALS of the batch (short kernels for profiler captures; "
                         "a line produced with this flag is not a benchmark result)")
    args = ap.parse_args()

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        return spawn_workers(args)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2504_03702_b200 import workloads as W
    wl = W.make_config(args.config, n_ticks=args.stream_ticks or None) if args.config == 4 else W.make_config(args.config)
    if args.impl == "reference":
        if rank == 0:
            run_reference(args, wl, rank)
        return 0

    import torch
    from paper_2504_03702_b200 import binding as B
    from paper_2504_03702_b200 import dist as D

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    group = D.init(world, rank, backend="nccl", device=device)
    n_sm = torch.cuda.get_device_properties(device).multi_processor_count
    peak, peak_kind = measured_peak_gbs()
    oracle_legs = not args.no_cpu_baseline and rank == 0

    if wl.streaming:
        sampler = ClockSampler(local_rank)
        for _ in range(min(args.warmup, 1)):      # one short warm-up stream: the first launches of every kernel
            bench_stream(args, W.make_config(4, n_ticks=8), 4, device, group, 0)
        sampler.start()
        rs = bench_stream(args, wl, 4, device, group, 12 if oracle_legs else 0)
        clocks = sampler.stop()
        if rank != 0:
            D.finish(group)
            return 0
        out = {
            "metric": METRIC_STREAM, "value": world * rs["arrivals"] / (rs["total_ms"] * 1e-3), "unit": "routes/s",
            "n_gpus": world, "steps": rs["ticks"], "warmup": min(args.warmup, 1) * 8,
            "ms_per_step": rs["total_ms"] / rs["ticks"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int64+f64", "data": "synthetic",
            "config": dict(config_dict(wl, 4), parallelism=f"{world} independent replica(s), one per GPU"),
            "ticks_per_s": rs["ticks"] / (rs["total_ms"] * 1e-3), "stream": rs,
            "parity_checked": rs["parity_checked"], "gpu_launches": 3 * rs["ticks"] + 1, "clocks": clocks,
            "roofline": {"bound": "smem", "achieved": None, "peak": None, "unit": "GB/s", "frac": None, "traffic": None,
                         "kernel": "pre_route_persistent",
                         "note": "per-tick batches of about 4,096 arrivals; see the one-shot configurations for the roofs"},
            "e2e": None,
        }
        if oracle_legs:
            tb, tt, routed = oracle_stream_sample(wl, 4)
            out["cpu_baseline"] = {"value": routed / tt, "unit": "routes/s", "cores": 1, "kind": "oracle",
                                   "sample": f"the first 4 ticks ({routed} arrivals) in the oracle's running-maxima mode, "
                                             f"{tt:.2f} s, after anticipate over the initial table ({tb:.2f} s)"}
        print(json.dumps(out))
        D.finish(group)
        return 0

    if args.arrivals > 0:
        wl.ticks = [(wl.ticks[0][0][:args.arrivals].copy(), wl.ticks[0][1][:args.arrivals].copy())]
    n0, a = wl.n_requests, wl.n_arrivals
    res = bench_oneshot(args, wl, args.config, device, group, world, args.steps, args.warmup, True)
    st = res["st"]
    code, route_blocks, tile_rows = B.pre_query(st.ctx)
    _, layout = B.pre_query_layout(st.ctx)

    # what was timed is checked: the state the last timed step left against one whole step of the oracle
    parity, identity = None, None
    if oracle_legs and args.arrivals == 0:
        ref, want_c, want_s, (tb, tr, ts), fast = oracle_full_step(wl)
        parity = compare_with_oracle(st, ref, res["snapshot"][0], res["snapshot"][1], want_c, want_s)
        identity = {"value": a / (tb + tr + ts), "unit": "routes/s", "cores": 1, "kind": "oracle",
                    "sample": f"one whole step, measured in full: anticipate {tb:.2f} s, routing of all {a} arrivals "
                              f"{tr:.2f} s ({'running-maxima' if fast else 'literal'} mode), decode step {ts:.2f} s",
                    "host_cores_available": os.cpu_count(),
                    "routes_per_s_route_call_only": a / tr,
                    "anticipated_request_steps_per_s": wl.n_requests * wl.horizon / tb}

    t_e2e, routed_ok = e2e_leg(res, wl, args.steps, group, device)
    extras = {} if args.no_extras else extras_leg(res, wl, args.config, device)
    if rank != 0:
        D.finish(group)
        return 0

    t_build, t_route, t_dstep, t_step = res["t_build"], res["t_route"], res["t_dstep"], res["t_step"]
    b_build, b_route, b_step = algorithmic_bytes(wl, n0 + a)
    fused = layout[2] > 0 and n0 <= layout[3]
    target = 0.60
    anticipate_roof = roof_hbm(b_build, t_build, 1 if fused else 2,
                               ANTICIPATE_DRAM_TRAFFIC.get(args.config) if fused else None,
                               "pre_build_fused" if fused else "pre_chunk_sort + pre_tile_build")
    anticipate_roof["target_frac"] = target
    anticipate_roof["target_met"] = anticipate_roof["frac"] >= target
    out = {
        "metric": METRIC, "value": world * a / (t_step * 1e-3), "unit": "routes/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int64+f64", "data": "synthetic",
        "config": dict(config_dict(wl, args.config), parallelism=f"{world} independent replica(s), one per GPU",
                       route_blocks=route_blocks, build_tile_rows=tile_rows, build_blocks=layout[2]),
        "parts_ms": {"anticipate": t_build, "route_batch": t_route, "step": t_dstep},
        "anticipated_request_steps_per_s": world * wl.n_requests * wl.horizon / (t_build * 1e-3),
        "routes_per_s_route_call_only": world * a / (t_route * 1e-3),
        "parity_checked": parity,
        "roofline": (route_summary_roofline(wl, args.config, t_route, a, res["clocks"]) if res["route_kernel"] == "summary"
                     else route_scan_roofline(wl, args.config, t_route, a, res["map_max"], layout, route_blocks, res["clocks"], n_sm)),
        "route_kernel": res["route_kernel"],
        "roofline_anticipate": anticipate_roof,
        "roofline_step": roof_hbm(b_step, t_dstep, 2, STEP_DRAM_TRAFFIC.get(args.config),
                                  "pre_step_requests + pre_step_shift",
                                  note="runs right after the routing kernel: part of the maps is served from L2, see traffic"),
        "e2e": {"value": world * a / (t_e2e * 1e-3), "unit": "routes/s", "h2d_bytes_per_step": res["h2d"],
                "d2h_bytes_per_step": res["d2h"], "ms_per_step": t_e2e},
        "gpu_launches": ((4 if fused else 5) + (2 if res["route_kernel"] == "summary" else 0)) * args.steps,
        "clocks": res["clocks"],
        "wall_s_timed_region": res["wall_s"],
        "routed": routed_ok,
    }
    if "route_scan_sample" in extras:
        t_scan, n_scan, scan_max = extras.pop("route_scan_sample")
        out["roofline_route_scan"] = route_scan_roofline(wl, args.config, t_scan, n_scan, scan_max, layout, route_blocks,
                                                         res["clocks"], n_sm)
        out["roofline_route_scan"]["sample"] = f"the first {n_scan} arrivals of the batch through the scanning kernel, one call"
    out.update(extras)
    if args.arrivals > 0:
        out["truncated_batch"] = "profiling run, not a benchmark result"
    if oracle_legs:
        n_route = min(a, args.cpu_arrivals)
        tb, tr, ts = oracle_sample(wl, n_route)
        t_cpu = tb + tr * (a / n_route) + ts
        out["cpu_baseline"] = {
            "value": a / t_cpu, "unit": "routes/s", "cores": 1, "kind": "oracle",
            "sample": f"anticipate over all {n0} requests ({tb:.2f} s), literal routing of the first {n_route} of "
                      f"{a} arrivals ({tr:.2f} s, scaled to the full batch), one decode step ({ts:.2f} s)",
            "host_cores_available": os.cpu_count(),
            "anticipated_request_steps_per_s": wl.n_requests * wl.horizon / tb,
        }
        if identity is not None:
            out["cpu_baseline_identity"] = identity
    st.close()

    # one short entry per configuration (the headline configuration's entry repeats the figures above)
    if not args.no_extras and args.arrivals == 0 and world == 1:
        entries = []
        for idx in range(5):
            if idx == args.config:
                entries.append({"config": idx, "routes_per_s_route_call_only": a / (t_route * 1e-3),
                                "us_per_arrival": t_route * 1e3 / a, "anticipate_us": t_build * 1e3,
                                "step_us": t_dstep * 1e3, "anticipated_request_steps_per_s": n0 * wl.horizon / (t_build * 1e-3),
                                "parity_checked": parity})
                continue
            w2 = W.make_config(idx)
            if w2.streaming:
                bench_stream(args, W.make_config(4, n_ticks=8), 4, device, group, 0)
                rs = bench_stream(args, w2, 4, device, group, 12 if oracle_legs else 0)
                entries.append({"config": 4, "routes_per_s": rs["arrivals"] / (rs["total_ms"] * 1e-3),
                                "ticks_per_s": rs["ticks"] / (rs["total_ms"] * 1e-3), "ticks": rs["ticks"],
                                "arrivals": rs["arrivals"], "anticipate_us": rs["anticipate_us"],
                                "step_us_median": rs["step_us_median"], "route_call_us_median": rs["route_call_us_median"],
                                "us_per_arrival_median": rs["route_us_per_arrival_median"],
                                "parity_checked": rs["parity_checked"], "parity_ticks": rs["parity_ticks"]})
                continue
            r2 = bench_oneshot(args, w2, idx, device, group, world, 3, 3, False)
            p2 = None
            if oracle_legs:
                ref2, wc2, ws2, _, _ = oracle_full_step(w2)
                p2 = compare_with_oracle(r2["st"], ref2, r2["snapshot"][0], r2["snapshot"][1], wc2, ws2)
            entries.append({"config": idx, "routes_per_s_route_call_only": w2.n_arrivals / (r2["t_route"] * 1e-3),
                            "us_per_arrival": r2["t_route"] * 1e3 / w2.n_arrivals, "anticipate_us": r2["t_build"] * 1e3,
                            "step_us": r2["t_dstep"] * 1e3,
                            "anticipated_request_steps_per_s": w2.n_requests * w2.horizon / (r2["t_build"] * 1e-3),
                            "parity_checked": p2})
            r2["st"].close()
        out["configs"] = entries
    print(json.dumps(out))
    D.finish(group)
    return 0


if __name__ == "__main__":
    sys.exit(main())
