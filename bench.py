#!/usr/bin/env python
"""Benchmark: full-batch gradient-descent iterations per second on a synthetic workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3] [--impl ours|reference]

A step is one GD iteration: one pass of the fused loss/gradient kernel over all of X plus the
cross-CTA reduction and parameter update.  The default workload is the 4M x 256 fp32 matrix (4.1 GB,
far larger than L2, so every iteration streams X from HBM).  One JSON line is printed by rank 0.

  value      iterations/s with X, y resident in HBM (CUDA events around one lr_fit call of K steps)
  e2e        the workload's own fit (its configured iteration count) through lr_fit_host: pinned host
             buffers in, parameters out, copies inside the timed region
  roofline   where lr_fit runs as one persistent launch (fp32 matrices of 64 MB and more with narrow rows): that kernel,
             K(4mn + 4m) bytes over its duration; `single_pass` (and every other case): one fused pass alone, from CUDA
             events around each launch
  cpu_baseline  the float64 CPU checker timed on this host on a bounded number of iterations

With --gpus N > 1 (under torchrun) the rows are sharded: every rank holds one workload-sized block of
rows (weak scaling), ranks exchange n+2 sums per iteration over NCCL, and value counts
workload-sized passes per second over all ranks.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# value is the iterations/sec part; the GB/s and the fraction of peak are in `achieved_hbm_gbs_whole_step` and `roofline`
METRIC = "GD iterations/sec and achieved HBM GB/s (fraction of B200 peak) at m\u00d7n fp32"
UNIT = "iterations/s"
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum per row of X, from the ncu captures summarised in profiles/ (taken on a
# smaller row count of the same workload and scaled by rows).  k_stream_rows / k_stream_split: one pass.  k_fit_rows: per
# row and iteration with nothing kept in L2 -- the captures ran three iterations with the default quarter of the L2
# (KEPT_BYTES of X) kept, so two of the three served those bytes from L2; the figure here has them added back, and
# `fit_traffic` takes the kept bytes off again for the iterations after the first.  Keys: workload, with "_bf16" for
# bfloat16 storage.  Remove an entry when its kernel changes.
KEPT_BYTES = 33_030_144                         # a quarter of the 126 MB L2, as lr_set_l2_keep's default for the persistent kernel
NCU_TRAFFIC_BYTES_PER_ROW = {
    "cfg2": {"k_stream_rows": (404.038400e6 + 5.690624e6) / 1_000_000,
             "k_fit_rows": (1.111161e9 + 3.984640e6 + 2 * KEPT_BYTES) / 3 / 1_000_000},
    "cfg5": {"k_stream_rows": (520.023296e6 + 4.371200e6) / 2_000_000,
             "k_fit_rows": (1.445884e9 + 3.818496e6 + 2 * KEPT_BYTES) / 3 / 2_000_000},
    "higgs_like": {"k_stream_rows": (464.071168e6 + 3.365120e6) / 4_000_000,
                   "k_fit_rows": (1.272406e9 + 3.437568e6 + 2 * KEPT_BYTES) / 3 / 4_000_000},
    "cfg3": {"k_stream_rows": (514.070528e6 + 3.252736e6) / 500_000,
             "k_fit_rows": (1.438903e9 + 3.893760e6 + 2 * KEPT_BYTES) / 3 / 500_000},
    "cfg4": {"k_stream_split": (491.682048e6 + 3.577600e6) / 30_000},
    "cfg3_bf16": {"k_stream_rows": (516.026880e6 + 4.308992e6) / 1_000_000,
                  "k_fit_rows": (1.441072e9 + 4.183552e6 + 2 * KEPT_BYTES) / 3 / 1_000_000},
    "cfg4_bf16": {"k_stream_split": (491.803904e6 + 5.702400e6) / 60_000},
}


def fit_traffic(per_row, m, steps, x_bytes, keep_bytes):
    """DRAM bytes of one persistent launch of `steps` iterations over m rows: every iteration after the first finds the kept
    part of X (at most all of it) in L2."""
    return per_row * m * steps - (steps - 1) * min(keep_bytes, x_bytes)


FALLBACK_HBM_GBS = 6650.0


def measured_hbm_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons in the background (100 ms period).

    Every sample carries nvidia-smi's own timestamp; `stop(t0, t1)` keeps the samples taken between the two wall-clock
    times (the timed region), so the sampler can be started early and its start-up time does not eat the region.
    """
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_uuid):
        if not gpu_uuid.startswith("GPU-"):
            gpu_uuid = "GPU-" + gpu_uuid
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", gpu_uuid, f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def wait_first_sample(self, limit_s=5.0):
        """Blocks until nvidia-smi has written its first line (or the limit passes)."""
        t_end = time.time() + limit_s
        while self.p is not None and time.time() < t_end:
            if os.path.getsize(self.f.name) > 0:
                return True
            time.sleep(0.05)
        return False

    @staticmethod
    def parse(text, t0=None, t1=None):
        """Samples of `text` (nvidia-smi csv lines) whose timestamp lies in [t0, t1] (all of them if t0 is None)."""
        import datetime
        rows = []
        for line in text.splitlines():
            t = [x.strip() for x in line.split(",")]
            if len(t) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(t[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                row = (ts, float(t[1]), float(t[2]), float(t[3]), t[4:8])
            except ValueError:
                continue
            if t0 is None or (t0 <= ts <= t1):
                rows.append(row)
        return rows

    @classmethod
    def summarise(cls, rows, in_region):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": len(rows), "in_timed_region": in_region}
        if rows:
            reasons = set()
            for r in rows:
                for name, v in zip(cls.NAMES, r[4]):
                    if v == "Active":
                        reasons.add(name)
            out.update(sm_mhz=statistics.median(r[1] for r in rows), sm_max_mhz=max(r[2] for r in rows),
                       reasons=sorted(reasons), power_w_max=max(r[3] for r in rows))
        return out

    def stop(self, t0, t1):
        """Ends the sampler; summarises the samples taken in the wall-clock window [t0, t1] (time.time() values)."""
        if self.p is None:
            return self.summarise([], True)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        text = self.f.read()
        self.f.close()
        os.unlink(self.f.name)
        rows = self.parse(text, t0, t1)
        if rows:
            return self.summarise(rows, True)
        # a region shorter than the sampling period: fall back to the samples nearest to it (within half a second)
        return self.summarise(self.parse(text, t0 - 0.5, t1 + 0.5), False)


def oracle_rate(X, y, wl, budget_s, max_rows=None):
    """Times the CPU checker as it stands; returns (iterations/s on the full m, description, threads)."""
    import numpy as np
    import oracle
    m = wl.m if max_rows is None else min(wl.m, max_rows)
    Xs, ys = X[:m], y[:m]
    t0 = time.perf_counter()
    oracle.fit(Xs, ys, wl.lr, 1)
    t1 = time.perf_counter() - t0
    k = int(max(2, min(wl.iters, budget_s / max(t1, 1e-9))))
    t0 = time.perf_counter()
    oracle.fit(Xs, ys, wl.lr, k)
    dt = time.perf_counter() - t0
    rate = k / dt * (m / wl.m)
    what = f"{k} of {wl.iters} iterations of oracle.fit on " + ("the full matrix" if m == wl.m else f"the first {m} of {wl.m} rows (rate scaled by rows)")
    return rate, what, oracle.threads()


def run_reference(args, wl):
    """The reference arm: the float64 CPU checker on the host cores, same metric and workload."""
    from paper_2308_10037_b200 import datagen
    import oracle
    steps, warmup = args.steps, args.warmup
    budget_s = 120.0
    # calibrate rows/s on a slice, then size each step's row sample so (steps + warmup) steps fit the budget
    probe_rows = min(wl.m, 200_000)
    Xp, yp, _, _ = datagen.generate(datagen.scaled(wl, probe_rows))
    oracle.fit(Xp, yp, wl.lr, 1)
    t0 = time.perf_counter()
    oracle.fit(Xp, yp, wl.lr, 3)
    rows_per_s = 3 * probe_rows / (time.perf_counter() - t0)
    rows = int(min(wl.m, max(10_000, budget_s * rows_per_s / (steps + warmup))))
    if rows > probe_rows:
        Xp, yp, _, _ = datagen.generate(datagen.scaled(wl, rows))
    else:
        Xp, yp = Xp[:rows], yp[:rows]
    import numpy as np
    w = np.zeros(wl.n)
    w, b, _ = oracle.fit(Xp, yp, wl.lr, warmup)
    t0 = time.perf_counter()
    oracle.fit(Xp, yp, wl.lr, steps, w0=w, b0=b)
    dt = time.perf_counter() - t0
    value = steps / dt * (rows / wl.m)
    sample = f"each step = one oracle iteration over the first {rows} of {wl.m} rows; rate scaled by rows/m"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warmup, "ms_per_step": 1e3 / value, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": workload_config(wl, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def f1_score(labels, y):
    """F1 of uint8 labels against 0/1 targets, 0 when nothing is predicted positive correctly (plain counting)."""
    import numpy as np
    pos = y > 0.5
    pred = labels != 0
    tp = int(np.count_nonzero(pred & pos)); fp = int(np.count_nonzero(pred & ~pos)); fn = int(np.count_nonzero(~pred & pos))
    return (2.0 * tp / (2.0 * tp + fp + fn)) if tp > 0 else 0.0, tp, fp, fn


def workload_config(wl, n_gpus, x_dtype="f32"):
    eb = 2 if x_dtype == "bf16" else 4
    return {"workload": f"{wl.name}: m={wl.m} x n={wl.n} {'bfloat16-stored' if eb == 2 else 'fp32'} row-major, lr={wl.lr}, {wl.iters} iterations"
                        + (f" (per GPU; {n_gpus} row shards)" if n_gpus > 1 else ""),
            "m": wl.m, "n": wl.n, "lr": wl.lr, "iters": wl.iters,
            "l2": (f"no flush needed: X is {wl.m * wl.n * eb / 1e6:.0f} MB per pass against 126 MB of L2"
                   if wl.m * wl.n * eb > 2 * 126e6 else
                   f"X is {wl.m * wl.n * eb / 1e6:.0f} MB, not larger than twice the 126 MB L2: part of every pass is served from L2"
                   if wl.m * wl.n * eb > 126e6 else
                   "X fits in L2: the pass is launch/L2-bound, not HBM-bound"),
            "parallelism": "single GPU" if n_gpus == 1 else f"dp{n_gpus} row-sharded, n+2 fp64 sums exchanged per iteration"}


def run_tol(args, wl):
    """Time to tolerance with the paper's stopping rule (Algorithm 7) on one GPU: `--tol ALPHA,EPS`.

    Trains on the first 90 % of the rows until ||grad||_2 <= EPS (at most --steps updates), scores F1 at threshold 0.5 on
    the held-out 10 %, and times the CPU checker on the same training rows for a bounded number of iterations.
    """
    import numpy as np
    import torch
    import oracle
    from paper_2308_10037_b200 import api, build, datagen
    alpha, eps = (float(v) for v in args.tol.split(","))
    build.build()
    X, y, _, _ = datagen.generate(wl)
    m_tr = int(0.9 * wl.m)
    dX, dy = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
    ctx = api.Context(n_max=wl.n, device=0)
    w = torch.zeros(wl.n, device="cuda")
    b = torch.zeros(1, device="cuda")
    ctx.fit(dX[:m_tr], dy[:m_tr], alpha, args.warmup, w, b)          # warm-up launches, result discarded
    torch.cuda.synchronize()
    w.zero_(); b.zero_()
    launches0 = ctx.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    iters, nrm = ctx.fit_tol(dX[:m_tr], dy[:m_tr], alpha, eps, args.steps, w, b, check_every=64)
    ev1.record()
    torch.cuda.synchronize()
    secs = ev0.elapsed_time(ev1) / 1e3
    labels = ctx.predict(dX[m_tr:], w, b, 0.5).cpu().numpy()
    f1 = f1_score(labels, y[m_tr:])[0]
    k = max(2, min(iters, 40))
    t0 = time.perf_counter()
    oracle.fit(X[:m_tr], y[:m_tr], alpha, k)
    cpu_it_s = k / (time.perf_counter() - t0)
    line = {"metric": "seconds to ||grad||_2 <= eps (Algorithm 7 stopping rule)", "value": secs, "unit": "s", "n_gpus": 1,
            "steps": iters, "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(iters, 1), "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{wl.name}: m={wl.m} x n={wl.n}, first 90 % train / last 10 % test, alpha={alpha}, eps={eps}",
                       "max_updates": args.steps},
            "updates": iters, "grad_norm": nrm, "converged": bool(nrm <= eps), "f1_test": f1,
            "cpu_baseline": {"value": iters / cpu_it_s, "unit": "s", "cores": oracle.threads(), "kind": "oracle",
                             "sample": f"{k} iterations of oracle.fit on the training rows, extrapolated to {iters} updates"},
            "gpu_launches": ctx.launch_count() - launches0}
    print(json.dumps(line))
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rows", type=int, default=0, help="override the workload's row count (profiling on a smaller case)")
    ap.add_argument("--tol", default="", help="ALPHA,EPS: time-to-tolerance mode (Algorithm 7 stopping rule); --steps caps the updates")
    ap.add_argument("--no-persistent", action="store_true", help="force two kernels per iteration in lr_fit")
    ap.add_argument("--force-persistent", action="store_true", help="force the single-launch persistent kernel in lr_fit")
    ap.add_argument("--no-overlap", action="store_true", help="ordinary launches only (no programmatic dependent launches)")
    ap.add_argument("--no-cluster", action="store_true", help="tiny problems: the grid-wide persistent kernel instead of the single-cluster one")
    ap.add_argument("--l2-keep-mb", type=float, default=-1.0, help="MB of X to keep in L2 across iterations (-1: library default, 0: off)")
    ap.add_argument("--x-dtype", default="f32", choices=["f32", "bf16"],
                    help="storage type of X on the device: bf16 runs the bfloat16 entry points on lr_convert_bf16's output "
                         "(half the bytes per pass)")
    ap.add_argument("--fused-exchange", action="store_true",
                    help="--gpus N > 1: exchange the sums inside the persistent kernel (lr_fit_sharded over symmetric memory) "
                         "instead of one NCCL all-gather per iteration")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    from paper_2308_10037_b200 import datagen
    wl = datagen.WORKLOADS[args.workload]
    if args.rows > 0:
        wl = datagen.scaled(wl, args.rows)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, wl)
        return
    if args.tol:
        if rank == 0:
            run_tol(args, wl)
        return

    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2308_10037_b200 import api, build, parallel
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    if rank == 0 or world == 1:
        build.build()
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    api.lib()

    # ---- inputs: generated on the host into pinned memory, then made resident ----
    wl_rank = wl if world == 1 else __import__("dataclasses").replace(wl, seed=wl.seed + rank)
    Xh = torch.empty((wl.m, wl.n), dtype=torch.float32, pin_memory=True)
    X_np, y_np, _, _ = datagen.generate(wl_rank, x_out=Xh.numpy())
    yh = torch.from_numpy(y_np).pin_memory()
    dX = Xh.to("cuda", non_blocking=True)
    dy = yh.to("cuda", non_blocking=True)
    torch.cuda.synchronize()
    ctx = api.Context(n_max=wl.n, device=local_rank)
    if args.no_persistent:
        ctx.set_persistent(False)
    if args.force_persistent:
        ctx.set_persistent(True)
    if args.no_overlap:
        ctx.set_overlap(False)
    if args.no_cluster:
        ctx.set_cluster(False)
    if args.l2_keep_mb >= 0:
        ctx.set_l2_keep(int(args.l2_keep_mb * 1e6))
    w = torch.zeros(wl.n, dtype=torch.float32, device="cuda")
    b = torch.zeros(1, dtype=torch.float32, device="cuda")
    m_total = wl.m * world
    bf16 = args.x_dtype == "bf16"
    if bf16:
        if world > 1:
            raise SystemExit("--x-dtype bf16 is a single-GPU mode")
        dX32 = dX
        dX = ctx.convert_bf16(dX32)                 # the fits below read the bfloat16 matrix only
        torch.cuda.synchronize()
        del dX32
    elem_bytes = 2 if bf16 else 4

    exchange = parallel.ExchangeBuffers(wl.n, torch.device("cuda", local_rank)) if world > 1 and args.fused_exchange else None

    def run_steps(k):
        if world == 1:
            ctx.fit(dX, dy, wl.lr, k, w, b)
        elif exchange is not None:
            parallel.fit_sharded_fused(ctx, dX, dy, m_total, wl.lr, k, w, b, exchange)
        else:
            parallel.fit_sharded_cuda(ctx, dX, dy, m_total, wl.lr, k, w, b)

    # ---- device-resident timing ----
    sampler = ClockSampler(str(torch.cuda.get_device_properties(local_rank).uuid)) if rank == 0 else None
    run_steps(args.warmup)
    torch.cuda.synchronize()
    if sampler:
        sampler.wait_first_sample()                 # nvidia-smi takes a second or so to come up
    if world > 1:
        dist.barrier()
    def timed_region():
        """EXACTLY args.steps steps between two CUDA events, a barrier and a device synchronisation on both sides."""
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        run_steps(args.steps)
        e1.record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        return e0.elapsed_time(e1)

    def max_over_ranks(values):
        if world == 1:
            return list(values)
        t = torch.tensor(values, dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return [float(v) for v in t.tolist()]

    launches0 = ctx.launch_count()
    wall0 = time.time()
    region_ms = max_over_ranks([timed_region()])
    launches = ctx.launch_count() - launches0       # kernels of ONE timed region
    # A region shorter than ~0.2 s says little about sustained clocks (and the clock sampler's period is 0.1 s): repeat it,
    # every repeat again exactly args.steps steps between its own events, for about a second in all, and report the median.
    repeats = 1 if region_ms[0] >= 200.0 else int(min(200, max(3, -(-1000.0 // region_ms[0]))))
    if repeats > 1:
        region_ms += max_over_ranks([timed_region() for _ in range(repeats - 1)])
    wall1 = time.time()
    ms = statistics.median(region_ms)
    clocks = sampler.stop(wall0, wall1) if sampler else None
    status = ctx.device_status()
    if status != 0:
        raise SystemExit(f"device status {status}: {api.status_string(status)}")
    value = args.steps * world / (ms / 1e3)

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- the streaming kernel alone (CUDA events around every launch, on its stream) ----
    k_prof = min(args.steps, 500)
    ctx.profile_enable(True)
    if world == 1:
        ctx.fit(dX, dy, wl.lr, k_prof, w, b)
    else:
        sums = torch.empty(wl.n + 2, dtype=torch.float64, device="cuda")
        for _ in range(k_prof):
            ctx.shard_sums(dX, dy, w, b, sums)
    torch.cuda.synchronize()
    n_l, tot_ms = ctx.profile_read()
    ctx.profile_enable(False)
    k1_ms = tot_ms / max(n_l, 1)
    bytes_per_launch = elem_bytes * wl.m * wl.n + 4 * wl.m
    achieved = bytes_per_launch / (k1_ms * 1e-3) / 1e9
    peak, peak_kind = measured_hbm_peak()
    plan = api.plan_query(wl.m, wl.n, sm_count=torch.cuda.get_device_properties(local_rank).multi_processor_count, bf16=bf16)
    pass_kernel = {0: "k_stream_rows", 1: "k_stream_split", 2: "k_generic", 3: "k_stream_rows"}[plan["variant"]]
    per_row = NCU_TRAFFIC_BYTES_PER_ROW.get(args.workload + ("_bf16" if bf16 else ""), {})
    single_pass = {"kernel": f"{pass_kernel} (one fused loss/gradient pass, two-kernel form of lr_fit)", "achieved": achieved,
                   "unit": "GB/s", "frac": achieved / peak, "bytes_per_launch": bytes_per_launch, "avg_launch_ms": k1_ms,
                   "launches_timed": n_l, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                   "traffic": per_row[pass_kernel] * wl.m if pass_kernel in per_row else None}
    if single_pass["traffic"] is not None:          # the same launch measured in DRAM bytes instead of algorithmic bytes
        single_pass["traffic_gbs"] = single_pass["traffic"] / (k1_ms * 1e-3) / 1e9
    if world == 1 and launches == 1:
        # the timed region was ONE launch of the persistent kernel doing all K iterations (pass + reduction + update)
        ach = bytes_per_launch * args.steps / (ms * 1e-3) / 1e9
        cluster_c = 0 if args.no_cluster else api.cluster_ctas(wl.m, wl.n, bf16=bf16)
        roofline = {"bound": "hbm", "kernel": (f"k_fit_cluster (all timed iterations in one launch on one cluster of {cluster_c} CTAs; X stays in "
                                               "their shared memory, so the algorithmic bytes below never reach HBM after the first pass)"
                                               if cluster_c else "k_fit_rows (persistent: all timed iterations in one cooperative launch)"),
                    "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak, "peak_kind": f"of {peak_kind}",
                    "traffic": (fit_traffic(per_row["k_fit_rows"], wl.m, args.steps, elem_bytes * wl.m * wl.n,
                                            KEPT_BYTES if args.l2_keep_mb < 0 else int(args.l2_keep_mb * 1e6))
                                if "k_fit_rows" in per_row and args.rows == 0 and not cluster_c else None),
                    "bytes_per_launch": bytes_per_launch * args.steps,
                    "avg_launch_ms": ms, "launches_timed": 1, "iterations_per_launch": args.steps,
                    "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS, "single_pass": single_pass}
        if roofline["traffic"] is not None:
            roofline["traffic_gbs"] = roofline["traffic"] / (ms * 1e-3) / 1e9
    else:
        roofline = dict(single_pass, bound="hbm", peak=peak, peak_kind=f"of {peak_kind}")

    # ---- end to end through the host-pointer entry point ----
    e2e = None
    if not args.no_e2e and world == 1:
        wh = torch.zeros(wl.n, dtype=torch.float32).pin_memory()
        bh = torch.zeros(1, dtype=torch.float32).pin_memory()
        times = []
        for rep in range(4):
            wh.zero_(); bh.zero_()
            t0 = time.perf_counter()
            ctx.fit_host(Xh, yh, wl.lr, wl.iters, wh, bh, store_bf16=bf16)
            times.append(time.perf_counter() - t0)
        t_e2e = statistics.median(times[1:])
        e2e = {"value": wl.iters / t_e2e, "unit": UNIT, "h2d_bytes_per_step": (4 * wl.m * wl.n + 4 * wl.m + 4 * wl.n + 4) / wl.iters,
               "d2h_bytes_per_step": (4 * wl.n + 4) / wl.iters, "seconds_per_fit": t_e2e,
               "what": (f"lr_fit_host{'_bf16' if bf16 else ''}: pinned fp32 X, y copied in, "
                        + ("X rounded to bfloat16 on the device, " if bf16 else "") + f"{wl.iters} iterations, w, b copied out; median of 3")}

    # ---- workloads that ask for it: the workload's own fit from zero, then predict at its threshold and F1 against y ----
    predict = None
    if wl.predict_thr is not None and world == 1:
        w.zero_(); b.zero_()
        ctx.fit(dX, dy, wl.lr, wl.iters, w, b)
        for _ in range(3):
            labels = ctx.predict(dX, w, b, wl.predict_thr)
        pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pe0.record()
        for _ in range(10):
            labels = ctx.predict(dX, w, b, wl.predict_thr)
        pe1.record()
        torch.cuda.synchronize()
        p_ms = pe0.elapsed_time(pe1) / 10
        # the confusion counts on the device (lr_f1_counts), timed; the host count over the downloaded labels must agree
        f1, tp, fp, fn = ctx.f1_counts(labels, dy)
        ce0, ce1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        counts = torch.empty(3, dtype=torch.int64, device="cuda")
        ce0.record()
        for _ in range(10):
            ctx.f1_counts_async(labels, dy, counts)
        ce1.record()
        torch.cuda.synchronize()
        c_ms = ce0.elapsed_time(ce1) / 10
        if (f1, tp, fp, fn) != f1_score(labels.cpu().numpy(), y_np):
            raise SystemExit("device confusion counts differ from the host count")
        predict = {"thr": wl.predict_thr, "f1_vs_y": f1, "tp": tp, "fp": fp, "fn": fn, "ms_per_predict": p_ms,
                   "ms_per_f1_counts": c_ms, "f1_counts_gbs": 5 * wl.m / (c_ms * 1e-3) / 1e9,
                   "gbs": (elem_bytes * wl.m * wl.n + wl.m) / (p_ms * 1e-3) / 1e9, "after_iterations": wl.iters}

    # ---- CPU checker on this host's cores (reported baseline, not a target) ----
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        X_cpu = X_np
        if bf16:                                    # the checker runs on the values the device streams: X rounded to bfloat16
            import oracle
            X_cpu = oracle.round_bf16(X_np)[1]
        rate, what, threads = oracle_rate(X_cpu, y_np, wl, budget_s=15.0)
        if bf16:
            what += " (X rounded to bfloat16 by the checker)"
        cpu = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "x_storage": args.x_dtype, "data": "synthetic", "config": workload_config(wl, world, args.x_dtype),
            "achieved_hbm_gbs_whole_step": bytes_per_launch * world * args.steps / (ms * 1e-3) / 1e9,
            "fit_form": ("one launch on one thread-block cluster for all timed iterations"
                         if launches == 1 and args.steps > 1 and not args.no_cluster and api.cluster_ctas(wl.m, wl.n, bf16=bf16) else
                         "one persistent launch for all timed iterations" if launches == 1 and args.steps > 1 else
                         f"{launches // max(args.steps, 1)} kernels per iteration"
                         + ("" if args.no_overlap else ", each the programmatic dependent of the one before")),
            "timed_regions": {"repeats": repeats, "ms_median": ms, "ms_min": min(region_ms), "ms_max": max(region_ms),
                              "what": f"each repeat is exactly {args.steps} steps between its own CUDA events; value uses the median"},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
            "predict": predict}
    print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
