#!/usr/bin/env python
"""Benchmark of the whole hot path: build the load-look-ahead maps, route one batch of
arrivals, advance one decode iteration.  One "step" = pre_anticipate + pre_route_batch +
pre_step on the largest one-shot configuration (4,096 instances, H = 2,048, 2,097,152
in-flight requests, 65,536 arrivals), seeded synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 0..3]

Prints ONE JSON line on rank 0.  `--impl reference` times the CPU oracle instead (a
deliberately plain sequential program) on a bounded sample of the same workload.
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


def oracle_sample(wl, n_route):
    """Times the oracle, as it stands, on a bounded sample. Returns seconds per part."""
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


def run_reference(args, wl, rank):
    """The reference arm: the CPU oracle on the host cores; rank 0 only."""
    if rank != 0:
        return
    n_route = min(wl.n_arrivals, args.ref_arrivals)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(wl, min(n_route, 8))
    per_step = []
    for _ in range(args.steps):
        tb, tr, ts = oracle_sample(wl, n_route)
        # whole-step time scaled to the full batch: the build and the decode step run in full,
        # routing cost is linear in the number of arrivals
        per_step.append(tb + tr * (wl.n_arrivals / n_route) + ts)
    t = float(np.mean(per_step))
    value = wl.n_arrivals / t
    sample = (f"per step: anticipate over all {wl.n_requests} requests, literal routing of the first {n_route} of "
              f"{wl.n_arrivals} arrivals (time scaled to the full batch), one decode step")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "routes/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int64+f64", "data": "synthetic",
        "config": dict(config_dict(wl, args), l2="not applicable (host run)",
                       timing="time.perf_counter around the oracle calls; routing time scaled from the sample "
                              "to the full batch"),
        "cpu_baseline": {"value": value, "unit": "routes/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "routes/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


METRIC = "routes/sec over the whole step (anticipate + route batch + decode step)"

# DRAM bytes (read + write) of one pre_route_persistent launch on the full batch of a
# configuration.  From an ncu capture of a 256-arrival batch on the same maps
# (profiles/ncu_dram_route_config3_256_arrivals.txt): 67.31 MB read (the maps, once per launch, whatever
# the batch length) + 655 B written per arrival (folded cells, appended requests), the written part
# scaled to 65,536 arrivals.  A configuration without a capture reports null.
ROUTE_DRAM_TRAFFIC = {3: 67312384 + 655 * 65536}


# DRAM bytes (read + write) of one pre_anticipate call on configuration 3, the two kernels added,
# from the full-set ncu capture (profiles/ncu_full_all_kernels_config3_256_arrivals.txt; the build does
# not depend on the length of the routing batch): pre_chunk_sort 33.61 MB read + 0.41 MB written,
# pre_tile_build 18.98 MB read + 9.24 MB written.  Most of the 64 MiB of maps is still in L2 when
# the call ends, which is why this is below the algorithmic 100.7 MB.
ANTICIPATE_DRAM_TRAFFIC = {3: 33612032 + 408832 + 18977024 + 9237504}


def config_dict(wl, args):
    return {"workload": f"config {args.config} ({wl.name}): {wl.n_instances} instances, H={wl.horizon}, "
                        f"{wl.n_requests} in-flight requests, {wl.n_arrivals} arrivals in one batch",
            "capacity_tokens": wl.capacity_tokens, "t_mem": wl.t_mem, "beta": wl.beta,
            "l2": "flushed between steps by writing a 512 MiB buffer",
            "timing": "CUDA events around each C-ABI call on the launching stream; state reset and L2 flush "
                      "between steps are not timed"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, choices=[0, 1, 2, 3])
    ap.add_argument("--ref-arrivals", type=int, default=256, help="arrivals routed per step by the reference arm")
    ap.add_argument("--cpu-arrivals", type=int, default=1500, help="arrivals routed by the cpu_baseline leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--arrivals", type=int, default=0,
                    help="route only the first ARRIVALS of the batch (short kernels for profiler captures; "
                         "a line produced with this flag is not a benchmark result)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2504_03702_b200 import workloads as W
    if args.impl == "reference":
        if rank == 0:
            run_reference(args, W.make_config(args.config), rank)
        return 0

    import torch
    from paper_2504_03702_b200 import binding as B
    from paper_2504_03702_b200 import dist as D
    from paper_2504_03702_b200.state import DeviceState

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    group = D.init(world, rank, backend="nccl", device=device)

    wl = W.make_config(args.config)
    if args.arrivals > 0:
        wl.ticks = [(wl.ticks[0][0][:args.arrivals].copy(), wl.ticks[0][1][:args.arrivals].copy())]
    n0, a = wl.n_requests, wl.n_arrivals
    arr_p_host, arr_d_host = wl.ticks[0]

    st = DeviceState.from_workload(wl, device=device)
    pristine_generated = st.generated[:n0].clone()
    arr_p = torch.as_tensor(arr_p_host).to(device)
    arr_d = torch.as_tensor(arr_d_host).to(device)
    choice = torch.empty(a, dtype=torch.int32, device=device)
    score = torch.empty(a, dtype=torch.float64, device=device)
    n0_dev = torch.tensor([n0], dtype=torch.int64, device=device)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)

    # pinned host copies for the end-to-end leg
    host_table = [torch.as_tensor(np.ascontiguousarray(x)).pin_memory()
                  for x in (wl.prompt, wl.generated, wl.predicted, wl.instance)]
    host_arr = [torch.as_tensor(np.ascontiguousarray(x)).pin_memory() for x in (arr_p_host, arr_d_host)]
    host_choice = torch.empty(a, dtype=torch.int32).pin_memory()
    host_score = torch.empty(a, dtype=torch.float64).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in host_table + host_arr)
    d2h = host_choice.numel() * 4 + host_score.numel() * 8

    def reset():
        st.generated[:n0].copy_(pristine_generated)
        st.n_requests.copy_(n0_dev)
        st.queued_p.zero_()
        flush.zero_()

    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731

    def one_step(timed):
        reset()
        e = [ev() for _ in range(4)]
        e[0].record()
        B.check(B.pre_anticipate(st.ctx, st.prompt, st.generated, st.predicted, st.instance, n0, st.curves,
                                 st.current_d), "pre_anticipate")
        e[1].record()
        B.check(B.pre_route_batch(st.ctx, arr_p, arr_d, a, st.curves, st.queued_p, st.current_d, st.prompt,
                                  st.generated, st.predicted, st.instance, st.n_requests, choice, score),
                "pre_route_batch")
        e[2].record()
        B.check(B.pre_step(st.ctx, st.prompt, st.generated, st.predicted, st.instance, st.n_requests, st.curves,
                           st.queued_p, st.current_d), "pre_step")
        e[3].record()
        return e

    def one_step_e2e():
        reset()
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
        return e0, e1

    for _ in range(max(args.warmup, 0)):
        one_step(False)
    torch.cuda.synchronize()
    B.check(st.status(), "warm-up")

    sampler = ClockSampler(local_rank)
    D.barrier(group)
    torch.cuda.synchronize()
    sampler.start()
    wall0 = time.perf_counter()
    events = [one_step(True) for _ in range(args.steps)]
    torch.cuda.synchronize()
    D.barrier(group)
    wall1 = time.perf_counter()
    clocks = sampler.stop()
    B.check(st.status(), "timed steps")

    t_build = float(np.mean([e[0].elapsed_time(e[1]) for e in events]))
    t_route = float(np.mean([e[1].elapsed_time(e[2]) for e in events]))
    t_dstep = float(np.mean([e[2].elapsed_time(e[3]) for e in events]))
    t_step_local = t_build + t_route + t_dstep
    t_step = D.max_over_ranks(t_step_local, group, device)

    # end-to-end leg: host buffers in, host results out, copies inside the timed region
    e2e_ms = []
    for k in range(1 + args.steps):
        e0, e1 = one_step_e2e()
        torch.cuda.synchronize()
        if k:  # the first one warms the pinned-copy path
            e2e_ms.append(e0.elapsed_time(e1))
    t_e2e = D.max_over_ranks(float(np.mean(e2e_ms)), group, device)
    B.check(st.status(), "end-to-end steps")
    routed_ok = int((host_choice >= 0).sum())

    # the same batch through the router with its admission queue (Sec. 4.3.3), the paper's overload
    # levels; a separate call, not part of the step
    reset()
    B.check(B.pre_anticipate(st.ctx, st.prompt, st.generated, st.predicted, st.instance, n0, st.curves,
                             st.current_d), "pre_anticipate")
    st.make_queue(4096)
    e0, e1 = ev(), ev()
    e0.record()
    _, adm_choice, _ = st.route_admit(arr_p, arr_d, overload_level=0.95, overload_share=0.10)
    e1.record()
    torch.cuda.synchronize()
    t_admit = e0.elapsed_time(e1)
    adm = {"routed": int((adm_choice >= 0).sum()), "waiting": int((adm_choice == -2).sum()),
           "turned_away": int((adm_choice == -3).sum())}
    B.check(st.status(), "admission call")
    # leave the state as the step leaves it (the calls below continue from there)
    reset()
    B.check(B.pre_anticipate(st.ctx, st.prompt, st.generated, st.predicted, st.instance, n0, st.curves,
                             st.current_d), "pre_anticipate")
    B.check(B.pre_route_batch(st.ctx, arr_p, arr_d, a, st.curves, st.queued_p, st.current_d, st.prompt,
                              st.generated, st.predicted, st.instance, st.n_requests, choice, score),
            "pre_route_batch")
    st.step()

    # scaler signals over the maps (Sec. 4.3.2): a separate, HBM-bound call, not part of the step
    flush.zero_()
    sc_ev = []
    for _ in range(4):
        flush.zero_()
        e0, e1 = ev(), ev()
        e0.record()
        st.scaler_signals()
        e1.record()
        sc_ev.append((e0, e1))
    torch.cuda.synchronize()
    t_scaler = float(np.median([x.elapsed_time(y) for x, y in sc_ev[1:]]))

    # misprediction refinement (Sec. 4.3.1): one pass over the table per tick against real lengths;
    # separate call, timed on four further ticks of the state the steps left behind
    table_actual, tick_actual = W.make_actual(wl, W.BASE_SEED + args.config)
    actual = torch.zeros(wl.max_requests, dtype=torch.int32, device=device)
    actual[:n0] = torch.from_numpy(table_actual).to(device)
    actual[n0:n0 + a] = torch.from_numpy(tick_actual[0][:a]).to(device)
    rf_ev, rf_counts = [], None
    for _ in range(4):
        st.step()
        flush.zero_()
        e0, e1 = ev(), ev()
        e0.record()
        rf_counts = st.refine(actual)
        e1.record()
        rf_ev.append((e0, e1))
    torch.cuda.synchronize()
    t_refine = float(np.median([x.elapsed_time(y) for x, y in rf_ev[1:]]))
    rf_counts = [int(v) for v in rf_counts.cpu().tolist()]
    B.check(st.status(), "refinement ticks")

    # full-width maps kept as a ring (Sec. 4.3.1), routed on the paper's window of 100 iterations:
    # a separate state on the same table and batch; one warm tick, one timed tick
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
    ring_routed = int((ring_choice >= 0).sum())
    ring_st.close()

    if rank != 0:
        D.finish(group)
        return 0

    peak, peak_kind = measured_peak_gbs()
    n_after = n0 + a
    b_build, b_route, b_step = algorithmic_bytes(wl, n_after)

    def roof(nbytes, ms, launches, traffic=None):
        gbs = nbytes / (ms * 1e-3) / 1e9
        return {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                "peak_kind": f"of {peak_kind}", "traffic": traffic, "algorithmic_bytes_per_launch": nbytes,
                "ms_per_launch": ms, "launches_per_step": launches}

    code, route_blocks, tile_rows = B.pre_query(st.ctx)
    out = {
        "metric": METRIC, "value": world * a / (t_step * 1e-3), "unit": "routes/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int64+f64", "data": "synthetic",
        "config": dict(config_dict(wl, args), parallelism=f"{world} independent replica(s), one per GPU",
                       route_blocks=route_blocks, build_tile_rows=tile_rows),
        "parts_ms": {"anticipate": t_build, "route_batch": t_route, "step": t_dstep},
        "anticipated_request_steps_per_s": world * wl.n_requests * wl.horizon / (t_build * 1e-3),
        "routes_per_s_route_call_only": world * a / (t_route * 1e-3),
        "roofline": dict(roof(b_route, t_route, 1, ROUTE_DRAM_TRAFFIC.get(args.config) if args.arrivals == 0 else None),
                         kernel="pre_route_persistent", served_from="shared memory",
                         limiter="latency of the per-arrival exchange between the blocks",
                         note="achieved = bytes of the literal scan (every arrival reads all I*H map cells) over "
                              "time. The maps are copied on chip once per batch (packed to 32-bit cells when they "
                              "fit) and every scan reads them from shared memory, so the figure is a scan-equivalent "
                              "rate, not HBM traffic, and exceeds the HBM peak; 'traffic' is the DRAM traffic of "
                              "the whole launch from an ncu capture scaled to this batch"),
        "roofline_anticipate": dict(roof(b_build, t_build, 2, ANTICIPATE_DRAM_TRAFFIC.get(args.config)),
                                    kernel="pre_chunk_sort + pre_tile_build"),
        "roofline_step": dict(roof(b_step, t_dstep, 2), kernel="pre_step_requests + pre_step_shift"),
        "roofline_scaler_signals": dict(roof(8 * wl.n_instances * wl.horizon + 12 * wl.n_instances, t_scaler, 1),
                                        kernel="pre_scaler_rows", note="separate call, not part of the step"),
        "route_admit": dict(adm, ms=t_admit, decided_per_s=a / (t_admit * 1e-3), kernel="pre_route_persistent<admit>",
                            overload_level=0.95, overload_share=0.10, queue_capacity=4096,
                            note="separate call, not part of the step; same batch, same maps"),
        "roofline_refine": dict(roof(20 * n_after, t_refine, 1), kernel="pre_refine_requests",
                                events_last_tick={"early_finish": rf_counts[0], "extended": rf_counts[1]},
                                note="separate call, not part of the step; bytes = five int32 columns of the "
                                     "table, the read-modify-write of the touched map cells is not counted"),
        "full_width_maps": {
            "width": wl.horizon, "window": ring_window, "routed": ring_routed,
            "tick_ms": {"pre_ring_step": ring_ms[0], "pre_ring_window": ring_ms[1], "pre_route_batch": ring_ms[2],
                        "pre_ring_fold": ring_ms[3]},
            "routes_per_s": a / (sum(ring_ms) * 1e-3),
            "dense_maps_same_tick_ms": {"pre_step": t_dstep, "pre_route_batch": t_route},
            "note": "separate state, not part of the step: maps of the configuration's full width kept as a ring "
                    "over absolute iterations, peaks taken over the next 100 iterations (the paper's l); one "
                    "scheduler tick = decode step + window copy + routing of the batch + real update of the ring"},
        "e2e": {"value": world * a / (t_e2e * 1e-3), "unit": "routes/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": t_e2e},
        "gpu_launches": 5 * args.steps,
        "clocks": clocks,
        "wall_s_timed_region": wall1 - wall0,
        "routed": routed_ok,
    }
    if args.arrivals > 0:
        out["truncated_batch"] = "profiling run, not a benchmark result"
    if not args.no_cpu_baseline:
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
    print(json.dumps(out))
    D.finish(group)
    return 0


if __name__ == "__main__":
    sys.exit(main())
