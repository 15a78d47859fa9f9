#!/usr/bin/env python
"""Benchmark of the EF21 hot path (libef21) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload all|headline|stress|hbm|floor] [--path auto|launches|persistent] [--stress-n N] [--no-cpu] [--no-e2e]

A "step" is one EF21 iteration (Algorithm 2's loop body over all n workers).  The headline
workload is the mushrooms-shaped logistic problem (n = 20, d = 112, N = 8,124, Top-1, gamma = 1/L);
the other named workloads are reported inside the same JSON line under "workloads".
One JSON line is printed by rank 0.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import ef21_inputs as inputs  # noqa: E402

METRIC = "EF21 iterations/sec (all n workers, 1 B200) and achieved HBM GB/s vs peak"
UNIT = "iterations/s"
HEADLINE = 1
FALLBACK_HBM_GBS = 6650.0
# Measured DRAM traffic (ncu: dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel, per launch
# where one launch runs all iterations and per iteration otherwise.  On the on-chip workloads a launch reads the
# shards and the state from DRAM once, whatever the number of iterations (every later iteration finds its rows in
# registers, shared memory or L2), so the per-launch figure holds for any step count.  None: not captured for the
# kernel as it stands.
NCU_TRAFFIC = {
    # persistent_kernel<1,16,REG,256,0>, launches of 2,000 iterations: 3,746,048 B read, 0 B written
    "headline": {"per": "launch", "bytes": 3746048},
    # persistent_kernel<3,4,GMEM,512,0>, launches of 50 iterations: 30,100,547,840 B read + 4,156,416 B written
    "hbm_persistent": {"per": "iteration", "bytes": 602094085},
    # st_collect_kernel<true> captured at n = 16 workers (537.12 MB read + 4.64 MB written per launch), scaled by
    # 64 / 16: the pass reads every vector once, so its traffic grows with the number of workers
    "stress_collect": {"per": "iteration", "bytes": 2167040000},
}


def logistic_bytes_per_iteration(n, d, k, N):
    """Algorithmic bytes one EF21 iteration must move: A and y once, every g_i once, x (read and
    write) and g once, and each (index, value) pair written and read once."""
    return 4 * N * (d + 1) + 4 * n * d + 12 * d + 16 * n * k


def stress_bytes_per_iteration(n, d, k):
    """Supplied-gradient iteration: V and every g_i read once, the dense x/g update (read x, g;
    write x), plus per selected pair the message (8 B written, 8 B read) and the two read-modify-
    writes of one 32-byte sector each on g_i and g."""
    return 8 * n * d + 12 * d + n * k * (16 + 64)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self._thread = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        try:
            for line in self.proc.stdout:
                parts = [p.strip() for p in line.strip().split(",")]
                if len(parts) >= 6:
                    self.rows.append(parts)
        except Exception:
            pass

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "20"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self._thread.start()
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self._thread.join(timeout=5)

    def summary(self):
        if not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm = [float(r[0]) for r in self.rows if r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [nm for i, nm in enumerate(names) if any(r[2 + i].lower().startswith("active") for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(self.rows),
                "window": "the timed runs plus 0.6 s of the same launches repeated (nvidia-smi, 20 ms period)"}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time: what a whole-job throughput has to be divided by."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms_max: float) -> float:
    """Replicas only: every rank processes units_per_rank in at most ms_max milliseconds."""
    return world * units_per_rank / (ms_max * 1e-3)


# ---------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on the host cores
# ---------------------------------------------------------------------------------------------

def time_oracle(w, steps, warmup):
    import oracle
    o = oracle.Oracle("f32")
    st = oracle.State(o, w.n, w.d, w.k, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(0)
    st.step(warmup)
    t0 = time.perf_counter()
    st.step(steps)
    dt = time.perf_counter() - t0
    return steps / dt, dt, st


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def time_oracle_parallel(w, steps, warmup):
    """The same oracle with the node loop of Algorithm 2 ("for all nodes in parallel") spread over
    min(n, cores) host threads: every worker's local gradient is one call of the oracle's own routine (the
    C call runs without the interpreter lock), the message round and the x update stay the oracle's
    single-threaded code.  Returns (iterations/s, seconds, threads)."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    o = oracle.Oracle("f32")
    st = oracle.State(o, w.n, w.d, w.k, w.gamma, w.lam, w.A, w.y, w.row_offsets, w.x0)
    st.init(0)
    threads = max(1, min(w.n, host_cores()))
    shards = [(w.A[w.row_offsets[i]:w.row_offsets[i + 1]], w.y[w.row_offsets[i]:w.row_offsets[i + 1]]) for i in range(w.n)]
    grads = np.empty((w.n, w.d), dtype=np.float32)

    def one(i):
        grads[i] = o.local_grad(shards[i][0], shards[i][1], st.x, w.lam)

    with ThreadPoolExecutor(max_workers=threads) as pool:
        def iterate(count):
            for _ in range(count):
                st.x_update()
                list(pool.map(one, range(w.n)))
                st.round(grads)
        iterate(warmup)
        t0 = time.perf_counter()
        iterate(steps)
        dt = time.perf_counter() - t0
    return steps / dt, dt, threads


def workload_string(w) -> str:
    return f"configs[{HEADLINE}] {w.name}: n={w.n} d={w.d} N={w.N} Top-{w.k} gamma=1/L lambda={w.lam}"


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    w = inputs.config(HEADLINE)
    steps = args.steps if args.steps is not None else 2000
    warmup = args.warmup if args.warmup is not None else 3
    its, dt, _ = time_oracle(w, steps, warmup)
    sample = f"{steps} full iterations of the headline workload (all {w.n} workers, {w.N} rows), single thread"
    line = {
        "impl": "reference", "metric": METRIC, "value": its, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "dtype_note": "state, differences, Top-k, aggregation and x update in fp32 as in the GPU arm; the oracle forms every "
                      "loss and gradient sum in fp64 and rounds it once to fp32",
        "config": {"workload": workload_string(w)},
        "cpu_baseline": {"value": its, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": its, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------------

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2106_05203_b200 import binding as B

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path in libef21)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def slowest(ms: float) -> float:
        return max_over_ranks(ms, world, device)

    peak, peak_kind = measured_peak()
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=device)     # > 126 MB of L2

    def flush_l2():
        flush_buf.fill_(1)

    dev = lambda a: torch.as_tensor(np.ascontiguousarray(a)).to(device)

    def time_stress(n_workers, steps, warmup):
        ws = inputs.config(4)
        n_w = n_workers or ws.n
        V = torch.empty((n_w, ws.d), dtype=torch.float32, device=device)
        for i in range(n_w):
            V[i].copy_(torch.from_numpy(ws.worker_vector(i)))
        hs = B.EF21(n_w, ws.d, ws.k, ws.gamma, device=device)
        hs.init_grads(None, B.INIT_ZERO)
        hs.step_grads(V, max(1, warmup))
        runs = []
        for _ in range(3):
            hs.init_grads(None, B.INIT_ZERO)
            hs.set_x(torch.zeros(ws.d, dtype=torch.float32, device=device))
            flush_l2()
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            l0 = hs.launch_count
            e0.record(); hs.step_grads(V, steps); e1.record()
            barrier()
            runs.append(slowest(e0.elapsed_time(e1)))
        ms = statistics.median(runs)
        b = stress_bytes_per_iteration(n_w, ws.d, ws.k)
        gbs = b * steps / (ms * 1e-3) / 1e9
        return {"workload": f"configs[4] {ws.name}: n={n_w} d={ws.d} Top-{ws.k} supplied gradients (static)",
                "iterations_per_s": steps / (ms * 1e-3), "us_per_iteration": ms / steps * 1e3, "steps": steps,
                "algorithmic_bytes_per_iteration": b, "algorithmic_GBps": gbs, "frac_of_hbm_peak": gbs / peak,
                "launches": hs.launch_count - l0, "fallbacks": hs.fallback_count(), "device_status": hs.poll()}

    if args.workload == "stress":
        r = time_stress(args.stress_n, args.steps if args.steps is not None else 50,
                        args.warmup if args.warmup is not None else 3)
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": world * r["iterations_per_s"], "unit": UNIT, "n_gpus": world,
                              "steps": r["steps"], "ms_per_step": r["us_per_iteration"] / 1e3, "dtype": "f32",
                              "data": "synthetic", "config": {"workload": r["workload"]},
                              "roofline": {"bound": "hbm", "achieved": r["algorithmic_GBps"], "peak": peak, "unit": "GB/s",
                                           "frac": r["frac_of_hbm_peak"], "traffic": NCU_TRAFFIC["stress_collect"]["bytes"], "peak_kind": f"of {peak_kind}",
                                           "kernel": "st_collect_kernel (dominant) + sample/finish/aggregate"},
                              "gpu_launches": r["launches"], "fallbacks": r["fallbacks"]}), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return

    def time_logistic(w, k, steps, warmup, repeats=5, with_clocks=False, variant=0):
        h = B.EF21(w.n, w.d, k, w.gamma, w.lam, total_rows=w.N, device=device)
        h.set_variant(variant)
        if variant == 0:
            h.set_path({"auto": B.PATH_AUTO, "launches": B.PATH_LAUNCHES, "persistent": B.PATH_PERSISTENT}[args.path])
        h.load_shards(dev(w.A), dev(w.y), w.row_offsets)
        h.init(B.INIT_ZERO if variant == B.VARIANT_EF else B.INIT_COMPRESSED)      # Algorithm 4 starts from e_i = 0
        x0, g0, gi0, _, _ = h.get_state()
        h.step(warmup)
        times, launches = [], 0
        sampler = ClockSampler(local_rank) if with_clocks else None
        if sampler:
            sampler.__enter__()
        for _ in range(repeats):
            h.set_state(x0, g0, gi0)
            flush_l2()
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            l0 = h.launch_count
            e0.record()
            h.step(steps)
            e1.record()
            barrier()
            launches = h.launch_count - l0
            times.append(slowest(e0.elapsed_time(e1)))
        if sampler:
            # nvidia-smi cannot resolve a few milliseconds: keep the same launches running for a while
            # longer (untimed) so that the sampler sees the clocks under exactly this load
            t_end = time.perf_counter() + 0.6
            while time.perf_counter() < t_end:
                h.set_state(x0, g0, gi0)
                h.step(steps)
                torch.cuda.synchronize()
            sampler.__exit__()
        status = h.poll()
        f_end = h.eval()[0]
        ms = statistics.median(times)
        return {"ms": ms, "launches": launches, "status": status, "f_end": f_end, "path": h.last_path,
                "shape": h.get_persistent_shape(), "clocks": sampler.summary() if sampler else None, "handle": h}

    def time_floor(w, k, steps, repeats=5):
        """us per iteration of the persistent path's exchange skeleton for this shape (no arithmetic of the method)."""
        h = B.EF21(w.n, w.d, k, w.gamma, w.lam, total_rows=w.N, device=device)
        h.load_shards(dev(w.A), dev(w.y), w.row_offsets)
        h.init(B.INIT_COMPRESSED)
        try:
            h.selftest_exchange_floor(20)
        except B.Ef21Error:
            return None
        times = []
        for _ in range(repeats):
            flush_l2()
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); h.selftest_exchange_floor(steps); e1.record()
            barrier()
            times.append(slowest(e0.elapsed_time(e1)))
        if h.poll() != 0:
            return None
        return statistics.median(times) / steps * 1e3

    def time_hbm_scale(steps, warmup):
        wb = inputs.hbm_scale_logistic()
        rr = time_logistic(wb, wb.k, steps, warmup)
        b = logistic_bytes_per_iteration(wb.n, wb.d, wb.k, wb.N)
        gbs = b * steps / (rr["ms"] * 1e-3) / 1e9
        return {"workload": f"{wb.name}: n={wb.n} d={wb.d} N={wb.N} Top-{wb.k} ({4 * wb.N * wb.d / 1e6:.0f} MB of shards, "
                            "streamed from HBM every iteration)",
                "iterations_per_s": steps / (rr["ms"] * 1e-3), "us_per_iteration": rr["ms"] / steps * 1e3, "steps": steps,
                "algorithmic_bytes_per_iteration": b, "algorithmic_GBps": gbs, "frac_of_hbm_peak": gbs / peak,
                "launches": rr["launches"], "persistent_shape": rr["shape"], "f_end": rr["f_end"], "device_status": rr["status"]}

    if args.workload == "floor":
        steps = args.steps if args.steps is not None else 2000
        rows = []
        for cfg, k in ((1, 1), (2, 1), (2, 4), (2, 16), (3, 1)):
            wk = inputs.config(cfg, k=k)
            rows.append({"workload": f"configs[{cfg}] {wk.name} Top-{k}", "floor_us_per_iteration": time_floor(wk, k, steps)})
        if rank == 0:
            print(json.dumps({"metric": "exchange floor of the persistent path (no arithmetic of the method)", "unit": "us per iteration",
                              "n_gpus": world, "steps": steps, "data": "synthetic", "workloads": rows}), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return

    if args.workload == "hbm":
        r = time_hbm_scale(args.steps if args.steps is not None else 50, max(3, args.warmup if args.warmup is not None else 3))
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": world * r["iterations_per_s"], "unit": UNIT, "n_gpus": world,
                              "steps": r["steps"], "ms_per_step": r["us_per_iteration"] / 1e3, "dtype": "f32",
                              "data": "synthetic", "config": {"workload": r["workload"]},
                              "roofline": {"bound": "hbm", "achieved": r["algorithmic_GBps"], "peak": peak, "unit": "GB/s",
                                           "frac": r["frac_of_hbm_peak"], "traffic": NCU_TRAFFIC["hbm_persistent"]["bytes"] if args.path != "launches" else None,
                                           "peak_kind": f"of {peak_kind}",
                                           "kernel": "persistent_kernel, rows streamed from global memory" if args.path != "launches"
                                                     else "grad_stream_kernel (dominant) + per-stage kernels"},
                              "gpu_launches": r["launches"], "persistent_shape": r["persistent_shape"]}), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- headline ---------------------------------------------------------------------------
    w = inputs.config(HEADLINE)
    steps = args.steps if args.steps is not None else w.T
    warmup = max(3, args.warmup if args.warmup is not None else 20)
    r = time_logistic(w, w.k, steps, warmup, with_clocks=True)
    its = whole_job_rate(steps, world, r["ms"])
    bytes_iter = logistic_bytes_per_iteration(w.n, w.d, w.k, w.N)
    achieved = bytes_iter * steps / (r["ms"] * 1e-3) / 1e9
    path_name = {1: "launch-per-stage kernels", 2: "persistent_kernel (one launch for all iterations)"}.get(r["path"], "?")
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": NCU_TRAFFIC["headline"]["bytes"] if r["path"] == 2 else None,
                "traffic_note": "DRAM bytes of one launch (ncu); the same for any number of iterations per launch: the shards "
                                "and the state are read once, every later iteration finds its rows on chip",
                "peak_kind": f"of {peak_kind}", "kernel": path_name,
                "algorithmic_bytes_per_iteration": bytes_iter, "algorithmic_bytes_per_launch": bytes_iter * steps,
                "note": "latency-bound by design: the 3.6 MB of shards stay on chip, each iteration waits on one "
                        "grid-wide exchange of the n messages; frac relates algorithmic bytes to the HBM copy peak"}

    # ---- end to end: host buffers in, result out, copies inside the timed region -------------
    A_pin = torch.from_numpy(w.A).pin_memory()
    y_pin = torch.from_numpy(w.y).pin_memory()
    e2e_times = []
    xh = gh = np.zeros(w.d, dtype=np.float32)
    for rep in range(0 if args.no_e2e else 3):
        flush_l2()
        barrier()
        t0 = time.perf_counter()
        h2 = B.EF21(w.n, w.d, w.k, w.gamma, w.lam, total_rows=w.N, device=device)
        h2.load_shards_host(A_pin.numpy(), y_pin.numpy(), w.row_offsets)
        h2.init(B.INIT_COMPRESSED)
        h2.step(steps)
        xh, gh, _, _, _ = h2.get_state_host(want_gi=False, messages=False)      # synchronises
        e2e_times.append(slowest((time.perf_counter() - t0) * 1e3))
    e2e_ms = statistics.median(e2e_times) if e2e_times else float("nan")
    e2e = None if args.no_e2e else {"value": whole_job_rate(steps, world, e2e_ms), "unit": UNIT,
           "h2d_bytes_per_step": (w.A.nbytes + w.y.nbytes) / steps, "d2h_bytes_per_step": (xh.nbytes + gh.nbytes) / steps,
           "note": f"create + load_shards_host + init + {steps} iterations + get_state_host, pinned host buffers; "
                   "bytes are per run divided by the iterations of the run"}

    line = {
        "metric": METRIC, "value": its, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": r["ms"] / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_string(w),
                   "l2": "L2 flushed (256 MB written) before each timed run; inside a run the iterations re-read the same "
                         "shards, which is the method's own access pattern",
                   "replicas": "replicas only: each rank runs the whole n-worker problem" if world > 1 else None,
                   "timed_runs": 5, "value_from": "median run"},
        "roofline": roofline, "e2e": e2e, "gpu_launches": r["launches"], "clocks": r["clocks"],
        "device_status": r["status"], "f_end": r["f_end"], "persistent_shape": r["shape"],
        "floor_us_per_iteration": time_floor(w, w.k, max(steps, 200)) if r["path"] == 2 else None,
    }
    if steps != w.T:
        # the same workload at the iteration count its configuration names (one launch runs them all): what a call costs
        # per iteration once the launch and the cold start of the kernel are spread over T iterations
        rT = time_logistic(w, w.k, w.T, warmup)
        gT = bytes_iter * w.T / (rT["ms"] * 1e-3) / 1e9
        line["headline_at_T"] = {"steps": w.T, "us_per_iteration": rT["ms"] / w.T * 1e3, "iterations_per_s": whole_job_rate(w.T, world, rT["ms"]),
                                 "algorithmic_GBps": gT, "frac_of_hbm_peak": gT / peak}

    # ---- CPU baseline (rank 0, N = 1 only) ---------------------------------------------------
    if rank == 0 and world == 1 and not args.no_cpu:
        o_steps = min(steps, 2000)
        o_its, o_dt, st = time_oracle(w, o_steps, 3)
        p_its, p_dt, p_threads = time_oracle_parallel(w, o_steps, 3)
        line["cpu_baseline"] = {"value": o_its, "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": f"{o_steps} full iterations of the headline workload, {o_dt:.1f} s, single thread",
                                "workers_in_parallel": {"value": p_its, "unit": UNIT, "cores": p_threads, "host_cores": host_cores(),
                                                        "sample": f"{o_steps} full iterations, {p_dt:.1f} s; the node loop of Algorithm 2 on "
                                                                  f"{p_threads} threads (one oracle gradient call per worker), the rest single-threaded"}}
    else:
        line["cpu_baseline"] = None

    # ---- the other named workloads (context; not the headline) -------------------------------
    if args.workload == "all" and world == 1:
        others = []
        for cfg, k in ((2, 1), (2, 4), (2, 16), (3, 1)):
            wk = inputs.config(cfg, k=k)
            rr = time_logistic(wk, k, wk.T, 20)
            b = logistic_bytes_per_iteration(wk.n, wk.d, k, wk.N)
            gbs = b * wk.T / (rr["ms"] * 1e-3) / 1e9
            others.append({"workload": f"configs[{cfg}] {wk.name} Top-{k}", "iterations_per_s": wk.T / (rr["ms"] * 1e-3),
                           "us_per_iteration": rr["ms"] / wk.T * 1e3, "algorithmic_bytes_per_iteration": b, "algorithmic_GBps": gbs,
                           "frac_of_hbm_peak": gbs / peak, "floor_us_per_iteration": time_floor(wk, k, wk.T) if rr["path"] == 2 else None,
                           "launches": rr["launches"], "persistent_shape": rr["shape"], "f_end": rr["f_end"]})
        others.append(time_stress(None, 50, 3))
        others.append(time_hbm_scale(50, 3))
        # EF21+ (Algorithm 3) on the headline shapes (persistent_plus_kernel)
        wp = inputs.config(HEADLINE)
        rp = time_logistic(wp, wp.k, 500, 10, variant=B.VARIANT_EF21_PLUS)
        others.append({"workload": f"EF21+ on configs[{HEADLINE}] {wp.name} Top-{wp.k}", "iterations_per_s": 500 / (rp["ms"] * 1e-3),
                       "us_per_iteration": rp["ms"] / 500 * 1e3, "launches": rp["launches"], "f_end": rp["f_end"]})
        # EF, the original error feedback method (Algorithm 4), same shapes
        re_ = time_logistic(wp, wp.k, 500, 10, variant=B.VARIANT_EF)
        others.append({"workload": f"EF (Algorithm 4) on configs[{HEADLINE}] {wp.name} Top-{wp.k}", "iterations_per_s": 500 / (re_["ms"] * 1e-3),
                       "us_per_iteration": re_["ms"] / 500 * 1e3, "launches": re_["launches"], "f_end": re_["f_end"]})
        # stochastic EF21 (Algorithm 5): tau sampled rows per worker and iteration, 500 iterations in one call
        for tau in (32, 128):
            hm = B.EF21(wp.n, wp.d, wp.k, wp.gamma, wp.lam, total_rows=wp.N, device=device)
            hm.load_shards(dev(wp.A), dev(wp.y), wp.row_offsets)
            hm.init(B.INIT_COMPRESSED)
            xm, gm, gim, _, _ = hm.get_state()
            rows = torch.as_tensor(np.stack([inputs.minibatch_rows(9, t, wp.row_offsets, tau) for t in range(500)])).to(device)
            hm.step_minibatches(rows[:20])
            tm, lm = [], 0
            for _ in range(5):
                hm.set_state(xm, gm, gim)
                flush_l2()
                barrier()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                l0 = hm.launch_count
                e0.record(); hm.step_minibatches(rows); e1.record()
                barrier()
                lm = hm.launch_count - l0
                tm.append(slowest(e0.elapsed_time(e1)))
            msm = statistics.median(tm)
            others.append({"workload": f"stochastic EF21 (Algorithm 5) on configs[{HEADLINE}] {wp.name} Top-{wp.k}, tau = {tau}",
                           "iterations_per_s": 500 / (msm * 1e-3), "us_per_iteration": msm / 500 * 1e3, "launches": lm,
                           "device_status": hm.poll(), "f_end": hm.eval()[0]})
        line["workloads"] = others
        line["workloads_note"] = ("frac_of_hbm_peak = algorithmic bytes per iteration / time / measured copy peak (read + write); on the "
                                  "on-chip workloads it is not a DRAM figure (DRAM traffic per launch is the shards once), and a read-only "
                                  "stream can exceed a copy peak slightly")

    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", choices=["all", "headline", "stress", "hbm", "floor"],
                    help="all: headline line with the other workloads attached; headline: only the headline; "
                         "stress: only the supplied-gradient workload; hbm: only the logistic workload whose shards "
                         "exceed L2 (each its own line; for profiling); floor: the exchange skeleton of the persistent "
                         "path on the logistic workloads")
    ap.add_argument("--path", default="auto", choices=["auto", "launches", "persistent"],
                    help="execution path of the logistic workloads (default: the library's own choice)")
    ap.add_argument("--stress-n", type=int, default=None, help="workers of the stress workload (default 64)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end timing")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle timing")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
