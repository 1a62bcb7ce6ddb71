"""Benchmark of the subsampled Gauss-Newton product path on synthetic data.

One step = one pass of the whole path at the 784-2000-2000-2000-10 network:
    set_subsample (row gather + stored forward pass on S)
    grad          (f and gradient over all l rows, in row batches)
    cg_solve      (n_cg CG steps on the full system: one G^S v each + vector updates)
    cg_solve      (n_cg CG steps on the per-layer systems: one block-diagonal product each)
The metric is Gauss-Newton matrix-vector products per second over whole steps (2 n_cg products per
step); the breakdown gives the product-only rates and FLOP/s.

    python bench.py --gpus N --steps K --warmup W            (N > 1: starts N ranks under torch.distributed.run
                                                              itself unless it already runs under one)
    python bench.py --impl reference ...                      (the float64 CPU checker on a bounded sample)
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import gn_workloads as wl  # noqa: E402

METRIC = "gauss_newton_matvecs_per_s"
UNIT = "matvec/s"
FP32_LANES_PER_SM, SMS = 128, 148
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant GEMM kernel from an ncu capture of the
# kernel as it stands.  Multi-pass counters are only taken on the small case (|S| = 3000), so the figure belongs to
# that workload; for every other workload `traffic` is None and the small-case figure is quoted beside it.
TRAFFIC = {("tf32", "mnist2000_5"): {"bytes_per_launch": 145.1e6, "kernel": "gemm_tf32_2cta_kernel",
                                     "launch": "forward R pass of a hidden layer, 3000 x 2000 x (2000 + 2000); 128 MB algorithmic",
                                     "source": "profiles/gemm_tf32_2cta_mnist2000_5_ncu.md"},
           ("fp32", "mnist2000_5"): {"bytes_per_launch": 144.4e6, "kernel": "gemm_tf32x3_kernel",
                                     "launch": "3000 x 2000 x 2000-class contraction on hi / lo parts",
                                     "source": "profiles/gemm_tf32x3_mnist2000_5_ncu.md"}}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    sm_max_mhz=d.get("sm_max_mhz", 1965.0), src="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, sm_max_mhz=1965.0, src="fallback")


def mac_counts(widths):
    g = [widths[m - 1] * widths[m] for m in range(1, len(widths))]
    L = len(g)
    fwd = sum(g)
    grad = 2 * sum(g) + sum(g[1:])
    full = 2 * g[0] + 4 * sum(g[1:])
    b1 = sum(2 * g[m] + 2 * sum(g[m + 1:]) for m in range(L))
    paper_block = sum(2 * g[m] + 2 * widths[-1] * widths[m + 1] for m in range(L))
    return dict(fwd=fwd, grad=grad, full=full, block_executed=b1, block_paper=paper_block)


def max_over_ranks(value, dist, device):
    """Slowest rank's time: the timed region of a multi-process run ends when the last rank ends."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(products_per_rank, world, ms):
    """Replicas only: every rank does the same number of products; the job's rate uses the slowest rank."""
    return products_per_rank * world / (ms * 1e-3)


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons for one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t0, t1):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [r for t, r in self.rows if t0 <= t <= t1 and len(r) >= 8] or [r for _, r in self.rows if len(r) >= 8]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = sorted(float(r[0]) for r in rows)
        reasons = set()
        for r in rows:
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(rows[0][1]), "samples": len(rows),
                "power_w_max": max(float(r[2]) for r in rows), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ CPU oracle arm
def step_config(args, p, world):
    """The `config` object of the JSON line; both arms print the same keys."""
    return {"workload": args.workload, "widths": p["widths"], "l": p["l"], "S": p["nS"], "C": p["C"], "n_cg": args.n_cg,
            "step": "set_subsample + grad(all rows) + n_cg CG steps full + n_cg CG steps block-diagonal",
            "l2": "per-step working set (activations of S and of the row batches) exceeds the 126 MB L2",
            "parallelism": "replicas only" if world > 1 else "single GPU"}


def oracle_sample_rates(p, sample_rows, n_cg):
    """Times the float64 checker on `sample_rows` rows and scales to the step's row counts."""
    from oracle import gn_oracle as orc
    rows = min(sample_rows, p["nS"])
    XS = p["X"][p["idx"][:rows]]
    th, w, C = p["theta"], p["widths"], p["C"]
    t0 = time.perf_counter(); orc.Gv(th, w, C, XS, p["v"]); t_full = time.perf_counter() - t0
    t0 = time.perf_counter(); orc.Gv_blockdiag(th, w, C, XS, p["v"]); t_blk = time.perf_counter() - t0
    t0 = time.perf_counter(); orc.grad(th, w, C, p["X"][:rows], p["Y"][:rows]); t_grad = time.perf_counter() - t0
    t0 = time.perf_counter(); orc.forward(th, w, XS); t_fwd = time.perf_counter() - t0
    step = (t_fwd * p["nS"] / rows + t_grad * p["l"] / rows + n_cg * (t_full + t_blk) * p["nS"] / rows)
    return dict(value=2 * n_cg / step, step_s=step, rows=rows, t_full=t_full, t_blk=t_blk, t_grad=t_grad,
                Gv_per_s=rows / (t_full * p["nS"]), cpu_s=t_full + t_blk + t_grad + t_fwd)


def oracle_one_core(p, n_cg, rows=128):
    """The same sample with the BLAS pool held to one thread (fewer rows: one core is slow)."""
    try:
        from threadpoolctl import threadpool_limits
    except Exception:
        return None
    with threadpool_limits(limits=1):
        r = oracle_sample_rates(p, rows, n_cg)
    return {"value": r["value"], "Gv_per_s": r["Gv_per_s"], "rows": r["rows"], "cores": 1}


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def run_reference(args):
    """The float64 checker as it stands on the host cores: each step times one bounded row sample of the workload;
    `value` is that rate scaled by row count to the workload's |S| and l, `ms_per_step` is the time actually spent
    per sampled step, and `full_step_ms_extrapolated` is what a whole step would take at that rate."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    p = wl.make(args.workload)
    for _ in range(min(args.warmup, 1)):
        oracle_sample_rates(p, max(64, args.ref_rows // 8), args.n_cg)
    vals, walls = [], []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        vals.append(oracle_sample_rates(p, args.ref_rows, args.n_cg))
        walls.append(time.perf_counter() - t0)
    v = float(np.median([x["value"] for x in vals]))
    cores = blas_threads()
    sample = (f"{vals[0]['rows']} of |S|={p['nS']} rows per product and {vals[0]['rows']} of l={p['l']} rows per gradient "
              f"pass, one of each per step; rates scaled by row count; numpy float64")
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * float(np.median(walls)),
            "full_step_ms_extrapolated": 1e3 * float(np.median([x["step_s"] for x in vals])),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": step_config(args, p, 1),
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "one_core": oracle_one_core(p, args.n_cg)},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------ GPU arm
def free_port():
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def relaunch_with_ranks(args):
    """`--gpus N` given to a plain `python bench.py`: start N ranks (one per GPU) under torch.distributed.run
    with the same arguments and hand back its exit code; rank 0 of that job prints the line."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_dry(args):
    """Launch / aggregation rehearsal without a GPU (`--dry-run`): the ranks join a gloo group, each pretends its
    timed region took 10 ms x (rank + 1), and rank 0 prints what the aggregation makes of it under `dry_run`.
    No kernel runs and no metric value is reported (`value` is null)."""
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    group = None
    if world > 1:
        dist.init_process_group("gloo")
        group = dist
        dist.barrier()
    ms = max_over_ranks(10.0 * (rank + 1), group, torch.device("cpu"))
    rate = whole_job_rate(2 * args.n_cg * args.steps, world, ms)
    if group:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                          "warmup": args.warmup, "scaling": "weak", "data": "none (dry run: no kernel was launched)",
                          "dry_run": {"ms": ms, "rate_from_pretended_times": rate, "backend": "gloo"}}))


def run_ours(args):
    import torch
    import paper_1802_00130_b200 as gn

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    p = wl.make(args.workload)
    mode = gn.GN_TF32 if args.mode == "tf32" else gn.GN_FP32_ACCURATE
    X, Y = torch.from_numpy(p["X"]).to(dev), torch.from_numpy(p["Y"]).to(dev)
    ctx = gn.GnContext(p["widths"], p["C"], X, Y, mode)
    if args.mode == "fp32_fma":
        ctx.set_accurate_method(1)
    theta = torch.from_numpy(p["theta"]).to(dev)
    # a fresh subsample per step, as in the Newton iteration: rotations of one permutation
    rng = np.random.Generator(np.random.PCG64(4242 + rank))
    perm = rng.permutation(p["l"]).astype(np.int32)
    n_sets = args.steps + args.warmup + 2
    idx_host = [np.ascontiguousarray(np.roll(perm, 977 * k)[: p["nS"]]) for k in range(n_sets)]
    idx_dev = [torch.from_numpy(a).to(dev) for a in idx_host]
    g = torch.empty(ctx.n, dtype=torch.float32, device=dev)
    d = torch.empty(ctx.n, dtype=torch.float32, device=dev)
    n_cg = args.n_cg

    def step(k):
        ctx.set_theta(theta)
        ctx.set_subsample(idx_dev[k % n_sets])
        ctx.grad(out=g)
        ctx.cg_solve(g, 1.0, blockdiag=False, max_iter=n_cg, tol=0.0, out=d)
        ctx.cg_solve(g, 1.0, blockdiag=True, max_iter=n_cg, tol=0.0, out=d)

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    for k in range(args.warmup):
        step(k)
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = ctx.kernel_launches
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    e0.record()
    for k in range(args.steps):
        step(args.warmup + k)
    e1.record()
    barrier()
    t_wall1 = time.time()
    ms = e0.elapsed_time(e1)
    launches = ctx.kernel_launches - launches0
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    ms = max_over_ranks(ms, dist, dev)
    # second pass over the same K steps with a CUDA-event pair around every contraction launch (on the context's
    # stream): per-kernel FLOP/s for the roofline.  The headline above is timed without these events.  In this pass
    # everything runs on the one stream, so that no launch's event pair spans time spent waiting behind another stream.
    ctx.debug_option(3, 0)
    ctx.profile(True)
    e0.record()
    for k in range(args.steps):
        step(args.warmup + k)
    e1.record()
    barrier()
    ms_profiled = e0.elapsed_time(e1)
    prof = ctx.profile_read()
    ctx.profile(False)
    matvecs = 2 * n_cg * args.steps * world
    value = whole_job_rate(2 * n_cg * args.steps, world, ms)

    # ---- product-only rates (device-resident, outside the step timing)
    v = torch.from_numpy(p["v"]).to(dev)
    out = torch.empty_like(v)
    breakdown = {}
    macs = mac_counts(p["widths"])
    def timed(fn, reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn(v, out=out)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e-3 / reps

    stored_ok = len(p["widths"]) >= 3 and p["widths"][-1] <= 16
    legs = [("Gv", ctx.Gv, 0, macs["full"], macs["full"]),
            ("Gv_blockdiag_propagate", ctx.Gv_blockdiag, 1, macs["block_executed"], macs["block_paper"])]
    if stored_ok:
        legs.append(("Gv_blockdiag_stored", ctx.Gv_blockdiag, 2, macs["block_paper"], macs["block_paper"]))
    for name, fn, method, mac_exec, mac_alg in legs:
        ctx.set_blockdiag_method(method)
        if method == 2:                       # the once-per-(theta, S) cost of the factors: first product - later ones
            ctx.set_subsample(idx_dev[0])
            torch.cuda.synchronize()
            first = timed(fn, 1)
        for _ in range(3):
            fn(v, out=out)
        torch.cuda.synchronize()
        t = timed(fn, args.product_reps)
        breakdown[name] = {"per_s": 1.0 / t, "ms": 1e3 * t,
                           "executed_tflops": 2.0 * mac_exec * p["nS"] / t / 1e12,
                           "algorithmic_tflops": 2.0 * mac_alg * p["nS"] / t / 1e12}
        if method == 2:
            breakdown[name]["factor_setup_ms"] = 1e3 * max(first - t, 0.0)
    ctx.set_blockdiag_method(0)

    # ---- set_subsample (row gather + stored forward pass) on its own, and amortised over a solve's products
    ts = []
    for k in range(5):
        torch.cuda.synchronize()
        t0s = time.perf_counter()
        ctx.set_subsample(idx_dev[k % n_sets])          # returns after its own synchronisation
        ts.append(time.perf_counter() - t0s)
    t_sub = float(np.median(ts[1:]))
    t_gv = breakdown["Gv"]["ms"] * 1e-3
    breakdown["set_subsample"] = {"ms": 1e3 * t_sub,
                                  "Gv_per_s_amortised": {str(k): k / (t_sub + k * t_gv) for k in (10, 50, 250)}}

    # ---- the same products in FP32-accurate mode (error-compensated tensor-core contractions), for the record of
    # that mode in the default run
    if args.mode == "tf32" and not args.no_fp32_leg:
        ctx32 = gn.GnContext(p["widths"], p["C"], X, Y, gn.GN_FP32_ACCURATE)
        ctx32.set_theta(theta)
        ctx32.set_subsample(idx_dev[0])
        leg = {}
        for name, fn, mac in (("Gv", ctx32.Gv, macs["full"]), ("Gv_blockdiag", ctx32.Gv_blockdiag, macs["block_paper"])):
            for _ in range(2):
                fn(v, out=out)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(max(3, args.product_reps // 2)):
                fn(v, out=out)
            b.record()
            torch.cuda.synchronize()
            t = a.elapsed_time(b) * 1e-3 / max(3, args.product_reps // 2)
            leg[name] = {"per_s": 1.0 / t, "ms": 1e3 * t, "algorithmic_tflops": 2.0 * mac * p["nS"] / t / 1e12}
        breakdown["fp32_accurate_mode"] = leg
        ctx32.close()
        del ctx32

    # ---- a library TF32 product of 8192^3 in the same run: what a plain GEMM sustains on this GPU (context only)
    lib_tf32 = None
    if args.mode == "tf32":
        prev = torch.backends.cuda.matmul.allow_tf32
        torch.backends.cuda.matmul.allow_tf32 = True
        ma = torch.randn(8192, 8192, device=dev); mb = torch.randn(8192, 8192, device=dev); mc = torch.empty_like(ma)
        for _ in range(3):
            torch.matmul(ma, mb, out=mc)
        la, lb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        la.record()
        for _ in range(10):
            torch.matmul(ma, mb, out=mc)
        lb.record()
        torch.cuda.synchronize()
        lib_tf32 = 10 * 2.0 * 8192 ** 3 / (la.elapsed_time(lb) * 1e-3) / 1e12
        torch.backends.cuda.matmul.allow_tf32 = prev
        del ma, mb, mc

    # ---- one Newton iteration of Algorithm 3 (block-diagonal CG capped at n_cg steps), for context
    th_n, dir_n = theta.clone(), torch.zeros_like(theta)
    prm = gn.NewtonParams(lam=1.0, sigma=1e-3, cg_max=n_cg, blockdiag=1)
    ctx.newton_iter(th_n, idx_dev[0], dir_n, prm)
    torch.cuda.synchronize()
    t0n = time.perf_counter()
    rep_n = ctx.newton_iter(th_n, idx_dev[1], dir_n, prm)
    torch.cuda.synchronize()
    breakdown["newton_iter"] = {"ms": 1e3 * (time.perf_counter() - t0n), "cg_iters": rep_n["cg_iters"],
                                "backtracks": rep_n["backtracks"], "f_before": rep_n["f_before"], "f_after": rep_n["f_after"]}

    # ---- end to end through the host-buffer entry points (pinned host memory)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory().numpy()
    h_theta, h_g, h_d = pin(p["theta"]), pin(np.zeros(ctx.n, np.float32)), pin(np.zeros(ctx.n, np.float32))
    h_idx = [pin(a) for a in idx_host]

    def step_host(k):
        ctx.set_theta_host(h_theta)
        ctx.set_subsample_host(h_idx[k % n_sets])
        ctx.grad_host(out=h_g)
        ctx.cg_solve_host(h_g, 1.0, blockdiag=False, max_iter=n_cg, tol=0.0, out=h_d)
        ctx.cg_solve_host(h_g, 1.0, blockdiag=True, max_iter=n_cg, tol=0.0, out=h_d)

    step_host(0)
    barrier()
    e0.record()
    for k in range(args.steps):
        step_host(args.warmup + k)
    e1.record()
    barrier()
    ms_e2e = e0.elapsed_time(e1)
    ms_e2e = max_over_ranks(ms_e2e, dist, dev)
    n4 = 4 * ctx.n
    e2e = {"value": matvecs / (ms_e2e * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": n4 + 4 * p["nS"] + 2 * n4, "d2h_bytes_per_step": n4 + 2 * n4}

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    pk = peaks()
    if args.mode == "tf32":
        peak = pk["bf16_sustained"] / 2.0
        roof = {"bound": "tensor", "unit": "TFLOP/s", "peak": peak,
                "peak_note": f"TF32 = 1/2 of the {pk['src']} sustained bf16 cuBLAS rate ({pk['bf16_sustained']} TFLOP/s)"}
    elif args.mode == "fp32":
        peak = pk["bf16_sustained"] / 6.0
        roof = {"bound": "tensor", "unit": "TFLOP/s", "peak": peak,
                "peak_note": f"FP32-accurate on the tensor cores takes 3 TF32 products per term: 1/3 of the TF32 peak, "
                             f"itself 1/2 of the {pk['src']} sustained bf16 cuBLAS rate ({pk['bf16_sustained']} TFLOP/s)"}
    else:
        peak = SMS * FP32_LANES_PER_SM * 2 * pk["sm_max_mhz"] * 1e6 / 1e12
        roof = {"bound": "alu", "unit": "TFLOP/s", "peak": peak,
                "peak_note": "148 SMs x 128 FP32 lanes x 2 FLOP x max SM clock"}
    main = {"tf32": "tensor", "fp32": "tensor_x3", "fp32_fma": "ffma"}[args.mode]
    kern = prof[main]
    achieved = kern["flop"] / (kern["ms"] * 1e-3) / 1e12 if kern["ms"] > 0 else None
    roof.update({"kernel": {"tensor": "gemm_tf32_2cta_kernel", "tensor_x3": "gemm_tf32x3_kernel",
                            "ffma": "gemm_ffma_kernel"}[main],
                 "achieved": achieved, "frac": achieved / peak if achieved else None,
                 "traffic": (TRAFFIC.get((args.mode, args.workload)) or {}).get("bytes_per_launch"),
                 "traffic_note": TRAFFIC.get((args.mode, args.workload)) or
                                 {"small_case": TRAFFIC.get((args.mode, "mnist2000_5")),
                                  "why_null": "counters of the current kernel were taken on the small case only"},
                 "launches": kern["launches"], "avg_launch_us": 1e3 * kern["ms"] / max(1, kern["launches"]),
                 "share_of_step": kern["ms"] / ms_profiled if ms_profiled > 0 else None,
                 "timing": "CUDA events around every launch of the kernel, on its stream, in a second pass over the same "
                           "K steps with everything on one stream (the headline pass carries no per-launch events and "
                           "runs the bias sums on a side stream); a grouped launch counts the FLOP of all its problems",
                 "ms_per_step_with_events": ms_profiled / args.steps,
                 "library_tf32_8192_tflops": lib_tf32,
                 "frac_of_library": achieved / lib_tf32 if (achieved and lib_tf32) else None,
                 "frac_of_nominal": achieved / 1100.0 if (achieved and args.mode == "tf32") else None,
                 "other_contractions": {name: {"ms": prof[name]["ms"], "launches": prof[name]["launches"]}
                                        for name in ("tensor", "tensor_1cta", "tensor_x3", "ffma", "thin") if name != main}})

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        r = oracle_sample_rates(p, args.ref_rows, n_cg)
        cpu = {"value": r["value"], "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"{r['rows']} rows per product and per gradient pass ({r['cpu_s']:.1f} s of CPU work), "
                         f"scaled by row count to |S|={p['nS']}, l={p['l']}",
               "Gv_per_s": r["Gv_per_s"], "one_core": oracle_one_core(p, n_cg)}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "tf32" if args.mode == "tf32" else "f32", "data": "synthetic",
            "config": step_config(args, p, world),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roof, "cpu_baseline": cpu,
            "breakdown": breakdown}
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mnist2000_20", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--mode", default="tf32", choices=["fp32", "fp32_fma", "tf32"],
                    help="tf32: TF32 contractions; fp32: FP32-accurate mode (error-compensated tensor-core contractions "
                         "where the shape allows); fp32_fma: FP32-accurate mode with every contraction on the FP32 FMA GEMM")
    ap.add_argument("--n-cg", dest="n_cg", type=int, default=10)
    ap.add_argument("--product-reps", type=int, default=10)
    ap.add_argument("--ref-rows", type=int, default=1024)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-fp32-leg", dest="no_fp32_leg", action="store_true",
                    help="skip the FP32-accurate products of the breakdown (they need a second context's workspaces)")
    ap.add_argument("--dry-run", action="store_true",
                    help="rehearse the launch of the ranks and the aggregation over them on CPU (gloo); no kernels, no value")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(relaunch_with_ranks(args))
    elif args.dry_run:
        run_dry(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
