#!/usr/bin/env python
"""Benchmark of the LSAM worker step on B200: worker-samples/s, roofline of the dominant kernel, CPU-oracle baseline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c1|c2|c3|c4|c5] [--impl reference]

A step is one pass of the whole hot path (schedule, gather, ascent gradient, norm, perturbation, descent gradient,
fused update) for all K replicas, plus the centre update whenever the sync trigger fires (every tau steps).
With more than one GPU every rank runs an independent copy of the workload (replicas only, the default: on one GPU
the path has no exchange step), or, with --shard-workers, the ranks form ONE job of N*K workers around a single
centre: K workers per GPU and one all-reduce of the iterate accumulator per sync (Algorithm 2, one worker per device).
Either way the work per GPU is fixed, so scaling is weak.
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
sys.path.insert(0, ROOT)

LSQ, MLP, RESMLP, FLAT = 0, 1, 2, 3

# The five workloads (shapes, replica counts, batch sizes and radii as configured).  Where a workload leaves them open:
# tau = 16 as in the paper's experiments, lambda = lambda0 / (eta tau) with lambda0 = 0.9 from the grid of Appendix D,
# beta = 0.9, eta' = 1.  (With the look-ahead beta = 0.9 and worker momentum 0.9 the worker/centre recursion alone is
# linearly unstable for short sync periods and weak pulls; tau = 16 with lambda0 = 0.9 is in its stable region.)
WORKLOADS = {
    "c1": dict(model=LSQ, widths=(256,), K=4, B=32, n=4096, classes=0, bf16=False, rho=0.05, eta=0.01, tau=4, stale_max=0, lambda0=0.5,
               name="least squares 4096x256, K=4, B=32"),
    "c2": dict(model=MLP, widths=(784, 1024, 10), K=8, B=128, n=60000, classes=10, bf16=False, rho=0.05, eta=0.05, tau=16,
               stale_max=0, name="MLP 784-1024-10 fp32, K=8, B=128"),
    "c3": dict(model=MLP, widths=(3072, 2048, 2048, 2048, 100), K=16, B=128, n=50000, classes=100, bf16=True, rho=0.1,
               eta=0.01, tau=16, stale_max=0, name="MLP 3072-2048x3-100 bf16 GEMM, K=16, B=128"),
    "c4": dict(model=RESMLP, widths=(3072, 4096, 4096, 4096, 4096, 1000), K=32, B=256, n=200000, classes=1000, bf16=True,
               rho=0.1, eta=0.002, tau=16, stale_max=3, head_scale=0.1, res_scale=0.25, name="residual MLP 3072-4096x4-1000 bf16 GEMM, K=32, B=256, staleness [0,3]"),
    "c5": dict(model=FLAT, widths=(), K=8, B=0, n=0, classes=0, bf16=False, rho=0.1, eta=0.05, tau=16, stale_max=0, d=256_000_000,
               name="optimiser-only sweep point d=256M, K=8"),
}
LAMBDA0, MU, BETA, ETA_PRIME, GAMMA = 0.9, 0.9, 0.9, 1.0, 1e-12
NOMINAL_HBM_GBS, FALLBACK_HBM_GBS, FALLBACK_BF16_TF = 8000.0, 6650.0, 1590.0
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12  # SMs x FMA lanes x 2 flop x max SM clock
# ncu counters of one update_kernel launch (dram__bytes_read.sum + dram__bytes_write.sum) at the c4 shape with K = 4
# replicas, see profiles/dram_traffic_c4_k4.md; traffic grows with (20 K + 12) d, so it is scaled to the K of the run.
NCU_UPDATE_TRAFFIC = dict(workload="c4", K=4, bytes=6111971328.0)
# the same for one update8f_kernel launch of the optimiser-only workload at K = 8, d = 25.6M (profiles/stream_kernels_c5_d25m.md);
# traffic grows with (20 K + 12) d, so it is scaled to the d of the run (rows of at least 4 M elements: the same kernel)
NCU_UPDATE_TRAFFIC_C5 = dict(K=8, d=25_600_000, bytes=4351901696.0)


def param_count(w):
    if w["model"] == FLAT:
        return w["d"]
    if w["model"] == LSQ:
        return w["widths"][0]
    ws = w["widths"]
    return sum(ws[i] * ws[i + 1] + ws[i + 1] for i in range(len(ws) - 1))


def max_over_ranks(ms, world, device=None):
    """Time of the slowest rank (the job's time); a plain float when there is one rank."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist

    t = torch.tensor([float(ms)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world, units_per_rank_step, ms_per_step):
    """Aggregate throughput of `world` independent replicas of the workload (weak scaling, no data-path collective)."""
    return world * units_per_rank_step / (ms_per_step * 1e-3)


def wk_bytes(work, name):
    return work[name]["bytes"]


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm=float(j["hbm_gbs"]), bf16=float(j["bf16_tflops"]), bf16_sustained=float(j.get("bf16_tflops_sustained", j["bf16_tflops"])), src="measured")
    return dict(hbm=FALLBACK_HBM_GBS, bf16=FALLBACK_BF16_TF, bf16_sustained=1400.0, src="fallback")


# ---------------------------------------------------------------------------------------------- algorithmic work per step
def work_model(w, tc):
    """Algorithmic bytes / flops per STEP of each kernel class (what the method must move or compute)."""
    K, B, d = w["K"], w["B"], param_count(w)
    op = 2 if w["bf16"] else 4
    out = {}
    out["norm"] = dict(bytes=0.0 if tc else 4.0 * K * d)                     # read g1 (fused into the wgrad epilogue on the tensor-core path)
    out["perturb"] = dict(bytes=(4.0 + (2.0 if tc else 4.0) + op) * K * d)   # read x, g1 (bf16 on the tensor-core path); write x~
    out["update"] = dict(bytes=((2.0 if tc else 4.0) + 8.0 + 8.0 + (2.0 if w["bf16"] else 0.0)) * K * d + 12.0 * d)  # g2 (bf16 on the tensor-core path), x rw, v rw, operand copy; y, acc rw
    if w["model"] in (MLP, RESMLP):
        ws = w["widths"]
        f_fwd = f_dg = f_wg = 0.0
        b_fwd = b_dg = b_wg = 0.0
        for l in range(len(ws) - 1):
            i, o = ws[l], ws[l + 1]
            f_fwd += 2.0 * B * i * o
            b_fwd += op * (i * o + B * i + B * o)
            f_wg += 2.0 * B * i * o
            b_wg += (2.0 if tc else 4.0) * i * o + op * B * (i + o)         # tensor-core path: the gradient is written as bf16
            if l > 0:
                f_dg += 2.0 * B * i * o
                b_dg += op * (i * o + B * i + B * o)
        for name, f, b in (("gemm_fwd", f_fwd, b_fwd), ("gemm_dgrad", f_dg, b_dg), ("gemm_wgrad", f_wg, b_wg)):
            out[name] = dict(flops=2.0 * K * f, bytes=2.0 * K * b)          # two gradient passes per step
    return out


# ---------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "25"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except Exception:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None, reasons=sorted(reasons), samples=len(sm))


# ---------------------------------------------------------------------------------------------- inputs (device, seeded)
def make_inputs(w, dev, seed=0):
    import torch

    g = torch.Generator(device=dev).manual_seed(seed)
    K = w["K"]
    if w["model"] == FLAT:
        d = w["d"]
        x0 = torch.randn(K, d, device=dev, generator=g)
        g1 = torch.randn(K, d, device=dev, generator=g) * 0.1
        g2 = torch.randn(K, d, device=dev, generator=g) * 0.1
        return dict(X=None, Y=None, x0=x0, y0=x0.mean(0), g1=g1, g2=g2)
    n, fin = w["n"], w["widths"][0]
    if w["model"] == LSQ:
        X = torch.randn(n, fin, device=dev, generator=g)
        wstar = torch.randn(fin, device=dev, generator=g)
        Y = X @ wstar + 0.01 * torch.randn(n, device=dev, generator=g)
        w0 = torch.randn(fin, device=dev, generator=g)
    else:
        C = w["classes"]
        means = torch.randn(C, fin, device=dev, generator=g)
        Y = (torch.arange(n, device=dev) % C).to(torch.int32)
        X = torch.randn(n, fin, device=dev, generator=g)
        X += means[Y.long()]
        parts = []
        ws = w["widths"]
        for l in range(len(ws) - 1):
            scale = (2.0 / ws[l]) ** 0.5
            if l == len(ws) - 2:
                scale *= w.get("head_scale", 1.0)       # small head: the initial loss starts near log(classes)
            elif w["model"] == RESMLP and ws[l] == ws[l + 1]:
                scale *= w.get("res_scale", 1.0)        # damped residual branches: no normalisation layers here
            parts.append((torch.randn(ws[l + 1], ws[l], device=dev, generator=g) * scale).reshape(-1))
            parts.append(torch.zeros(ws[l + 1], device=dev))
        w0 = torch.cat(parts)
    x0 = w0.unsqueeze(0).expand(K, -1).contiguous()
    return dict(X=X, Y=Y, x0=x0, y0=w0)


def make_cfg(G, w, flags=0, K_total=0, k_offset=0):
    lam = w.get("lambda0", LAMBDA0) / (w["eta"] * w["tau"])
    return G.make_config(w["model"], widths=w["widths"], K=w["K"], batch=max(w["B"], 1) if w["model"] != FLAT else 0,
                         gemm_dtype=G.GEMM_BF16 if w["bf16"] else G.GEMM_FP32, mu=MU, nesterov=1, gamma=GAMMA, lam=lam, tau=w["tau"],
                         beta=BETA, eta_prime=ETA_PRIME, stale_max=w["stale_max"], seed=0, n_samples=max(w["n"], 1),
                         flat_d=w.get("d", 0), flags=flags, active_num=w.get("active_num", 256),
                         noise_temp=w.get("noise_temp", 0.0), K_total=K_total, k_offset=k_offset)


# ---------------------------------------------------------------------------------------------- CPU oracle leg
def oracle_baseline(w, X, Y, x0_row, budget_s=20.0):
    """Time the oracle, as it stands, on a bounded sample of the workload: a subset of replicas and of each minibatch."""
    import oracle as O

    cores = O.num_threads()
    d = param_count(w)
    lam = w.get("lambda0", LAMBDA0) / (w["eta"] * w["tau"])
    if w["model"] == FLAT:
        Ks, ds = w["K"], min(d, 4_000_000)
        cfg = O.make_config(O.MODEL_FLAT, K=Ks, flat_d=ds, mu=MU, gamma=GAMMA, lam=lam, tau=w["tau"], beta=BETA, eta_prime=ETA_PRIME)
        rng = np.random.default_rng(0)
        x0 = rng.standard_normal((Ks, ds))
        g1 = (0.1 * rng.standard_normal((Ks, ds))).astype(np.float32)
        o = O.Oracle(cfg, None, None, x0, x0.mean(0))
        o.set_external_grads(g1, g1)
        def tick():
            o.step(w["eta"], w["rho"])
            if o.should_couple():
                o.couple()

        tick()
        t0 = time.perf_counter()
        steps = 3
        for _ in range(steps):
            tick()
        dt = (time.perf_counter() - t0) / steps
        return dict(value=36.0 * Ks * ds / dt / 1e9, unit="GB/s (36 B per element-replica)", cores=min(cores, Ks), kind="oracle",
                    sample=f"K={Ks} replicas, d={ds} of {d} elements, {steps} steps"), dt
    # flops per worker-sample (12 per weight: two passes of fwd + dgrad + wgrad) and a measured-free guess of 1.5 GFLOP/s/core
    flop_ws = 12.0 * d
    Ks = min(w["K"], cores)
    Bs = int(max(1, min(w["B"], budget_s * 1.5e9 / flop_ws)))
    cfg = O.make_config(w["model"], widths=w["widths"], K=Ks, batch=Bs, gemm_dtype=O.GEMM_BF16 if w["bf16"] else O.GEMM_FP32, mu=MU,
                        gamma=GAMMA, lam=lam, tau=w["tau"], beta=BETA, eta_prime=ETA_PRIME, stale_max=w["stale_max"], seed=0, n_samples=w["n"])
    x0 = np.repeat(x0_row[None, :].astype(np.float64), Ks, axis=0)
    o = O.Oracle(cfg, X, Y, x0, x0_row.astype(np.float64))
    steps = 1 if flop_ws * Bs > 2e9 else 5
    t0 = time.perf_counter()
    for _ in range(steps):
        o.step(w["eta"], w["rho"])
        if o.should_couple():
            o.couple()
    dt = (time.perf_counter() - t0) / steps
    o.close()
    return dict(value=Ks * Bs / dt, unit="worker-samples/s", cores=min(cores, Ks), kind="oracle",
                sample=f"{Ks} of {w['K']} replicas x {Bs} of {w['B']} samples per minibatch, full model, {steps} step(s)"), dt


def run_reference(args, w, metric, unit):
    """--impl reference: the CPU oracle timed on bounded samples of the same workload (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import torch

    inp = make_inputs(w, torch.device("cpu"), seed=0)
    X = None if inp["X"] is None else inp["X"].numpy()
    Y = None if inp["Y"] is None else inp["Y"].numpy()
    x0_row = inp["y0"].numpy()
    vals, dts = [], []
    per = max(2.0, min(20.0, 120.0 / max(args.steps + args.warmup, 1)))
    for i in range(args.warmup + args.steps):
        cb, dt = oracle_baseline(w, X, Y, x0_row, budget_s=per)
        if i >= args.warmup:
            vals.append(cb["value"])
            dts.append(dt)
    v = float(np.mean(vals))
    cb["value"] = v
    line = dict(impl="reference", metric=metric, value=v, unit=unit, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=float(np.mean(dts) * 1e3), higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64",
                data="synthetic", config=dict(workload=w["name"]), cpu_baseline=cb,
                e2e=dict(value=v, unit=unit, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--workload", default="c4", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--flat-d", type=int, default=None, help="c5 only: vector length of the sweep point")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--replicas", type=int, default=None, help="override K (small cases for profiler captures)")
    ap.add_argument("--noise-temp", type=float, default=0.0, help="Langevin temperature of the sampler (0 = none)")
    ap.add_argument("--active-num", type=int, default=256, help="asynchronous progress: a worker is ready at a tick with probability N/256")
    ap.add_argument("--shard-workers", action="store_true",
                    help="N > 1: one job of N*K workers with a single centre, K workers per GPU, accumulator all-reduce every tau steps "
                         "(default: N independent copies of the workload)")
    ap.add_argument("--cuda-graph", default="auto", choices=["auto", "on", "off"], help="replay each tick as one CUDA graph (auto: when the state fits in L2)")
    args = ap.parse_args()
    w = dict(WORKLOADS[args.workload])
    if args.flat_d and w["model"] == FLAT:
        w["d"] = args.flat_d
        w["name"] = f"optimiser-only sweep point d={args.flat_d}, K=8"
    if args.replicas:
        w["K"] = args.replicas
        w["name"] += f" [K overridden to {args.replicas}]"
    if args.noise_temp > 0.0:
        w["noise_temp"] = args.noise_temp
        w["name"] += f" [Langevin temperature {args.noise_temp}]"
    if args.active_num != 256:
        w["active_num"] = args.active_num
        w["name"] += f" [workers ready with probability {args.active_num}/256 per tick]"
    flat = w["model"] == FLAT
    metric = "fused_update_hbm_gbs" if flat else "lsam_worker_samples_per_s"
    unit = "GB/s" if flat else "worker-samples/s"
    if args.impl == "reference":
        return run_reference(args, w, metric, unit)

    import torch
    import torch.distributed as dist

    from paper_2509_03110_b200 import binding as G

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    shard = bool(args.shard_workers)
    if world > 1 or shard:
        if world == 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29541")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    warm = max(args.warmup, 3)

    # sharded: every rank generates the same dataset and the same initial point (one job); else independent copies
    inp = make_inputs(w, dev, seed=0 if shard else rank)
    # Latency-bound workloads (state resident in L2) replay each tick as one CUDA graph; that needs a capturable stream.
    small = 4.0 * w["K"] * param_count(w) <= 126e6
    # auto: also where the kernels of a step are short (tens of microseconds each), so that launch gaps and the
    # per-launch events of the roofline pass would be a visible share of the step
    short_kernels = 4.0 * w["K"] * param_count(w) <= 1.2e9
    use_graph = (small or short_kernels) if args.cuda_graph == "auto" else args.cuda_graph == "on"
    cfg = make_cfg(G, w, flags=G.FLAG_CUDA_GRAPH if use_graph else 0, K_total=world * w["K"] if shard else 0, k_offset=rank * w["K"] if shard else 0)
    torch.cuda.synchronize()
    work_stream = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(work_stream)
    ctx = G.Lsam(cfg, inp["X"], inp["Y"], inp["x0"], inp["y0"], stream=work_stream)
    d = ctx.d
    inp["x0"] = None
    torch.cuda.empty_cache()
    if flat:
        ctx.set_external_grads(inp["g1"], inp["g2"])
    stream = ctx.stream
    eta, rho = w["eta"], w["rho"]

    if shard:
        from paper_2509_03110_b200 import sharded

    def couple():
        if shard:
            sharded.exchange_and_couple(ctx)  # all-reduce of the iterate accumulator over the ranks, then the centre update
        else:
            ctx.couple()

    def one_step():
        ctx.step(eta, rho)
        if ctx.should_couple():
            couple()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident timing (value), with per-kernel-class events for the roofline
    for _ in range(warm):
        one_step()
    # Per-kernel CUDA events ride inside the timed region when a step is long (working set beyond L2); for the
    # latency-bound workloads they would distort it, so there the shares come from a second, separate run of the same steps.
    events_in_timed = 4.0 * w["K"] * d > 126e6 and not use_graph  # graph replay is off while per-launch events are recorded
    ctx.profile_enable(events_in_timed)
    ctx.profile_read()
    launches0 = ctx.launch_count()
    clocks = ClockSampler(local)
    barrier()
    clocks.start()
    def iterations_done():  # worker iterations since the context was created: every sync closes exactly K tau of them
        _, t_y, t_x = ctx.counters()
        return w["K"] * w["tau"] * t_y + int(t_x.sum())

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    it0 = iterations_done()
    e0.record(stream)
    for _ in range(args.steps):
        one_step()
    e1.record(stream)
    barrier()
    clk = clocks.stop()
    ms = e0.elapsed_time(e1)
    worker_iters_per_step = (iterations_done() - it0) / args.steps  # = K in lock-step mode
    if not events_in_timed:
        launches_timed = ctx.launch_count() - launches0
        ctx.profile_enable(True)
        for _ in range(args.steps):
            one_step()
        barrier()
        launches0 = ctx.launch_count() - launches_timed
    prof = ctx.profile_read()
    ctx.profile_enable(False)
    launches = ctx.launch_count() - launches0
    if ctx.status() != 0:
        raise SystemExit("device status word is not clean after the timed region")
    ms = max_over_ranks(ms, world, dev)
    ms_step = ms / args.steps
    units_step = (36.0 * worker_iters_per_step * d / 1e9) if flat else float(worker_iters_per_step * w["B"])
    value = whole_job_value(world, units_step, ms_step)

    # ---- end to end through the C ABI with host buffers (minibatch H2D and loss D2H inside the timed region)
    e2e = None
    if not flat:
        nst = min(args.steps, 8)
        nb = min(nst, 4)
        fin = w["widths"][0]
        t_now = ctx.counters()[0]
        xbs, ybs = [], []
        for i in range(nb):
            idx, _, _ = ctx.read_schedule(t_now + i, want_ver=False)
            ii = torch.from_numpy(idx.reshape(-1).astype(np.int64)).to(dev)
            xbs.append(inp["X"][ii].reshape(w["K"], w["B"], fin).cpu().pin_memory())
            ybs.append(inp["Y"][ii].reshape(w["K"], w["B"]).cpu().pin_memory())
        loss = np.zeros(w["K"], np.float32)
        ctx.step_batch(eta, rho, xbs[0], ybs[0], loss)
        if ctx.should_couple():
            couple()
        barrier()
        e0.record(stream)
        # every step's minibatch crosses PCIe inside the timed region; the copy of step i+1 is issued on the library's
        # copy stream before step i is enqueued, so it overlaps that step's kernels
        ctx.stage_batch(xbs[0], ybs[0])
        for i in range(nst):
            if i + 1 < nst:
                ctx.stage_batch(xbs[(i + 1) % nb], ybs[(i + 1) % nb])
            ctx.step_staged(eta, rho, loss)
            if ctx.should_couple():
                couple()
        e1.record(stream)
        barrier()
        ems = max_over_ranks(e0.elapsed_time(e1), world, dev)
        e2e = dict(value=whole_job_value(world, w["K"] * w["B"], ems / nst), unit=unit, h2d_bytes_per_step=int(xbs[0].numel() * 4 + ybs[0].numel() * 4),
                   d2h_bytes_per_step=int(4 * w["K"]), steps=nst)
    else:
        # optimiser-only: the gradients are the step's inputs; copy them from pinned host memory every step
        K = w["K"]
        hg = torch.empty(2, K, d, dtype=torch.float32).pin_memory() if d <= 64_000_000 else None
        if hg is not None:
            hg[0].copy_(inp["g1"].cpu())
            hg[1].copy_(inp["g2"].cpu())
            out = np.zeros(d, np.float32)
            barrier()
            nst = min(args.steps, 5)
            e0.record(stream)
            for _ in range(nst):
                inp["g1"].copy_(hg[0], non_blocking=True)
                inp["g2"].copy_(hg[1], non_blocking=True)
                one_step()
                ctx.read_step_info()
            e1.record(stream)
            barrier()
            ems = max_over_ranks(e0.elapsed_time(e1), world, dev)
            e2e = dict(value=whole_job_value(world, units_step, ems / nst), unit=unit, h2d_bytes_per_step=int(8 * K * d), d2h_bytes_per_step=int(12 * K), steps=nst)
        else:
            e2e = dict(value=None, unit=unit, h2d_bytes_per_step=int(8 * K * d), d2h_bytes_per_step=int(12 * K),
                       note="gradient buffers of this sweep point exceed the pinned-memory budget; run --flat-d <= 64000000")

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel class
    pk = peaks()
    work = work_model(w, ctx.uses_tcgen05())
    frac_active = worker_iters_per_step / w["K"]  # waiting replicas are skipped by every kernel
    for wk_ in work.values():
        for key in wk_:
            wk_[key] *= frac_active
    tot_ms = sum(v[0] for v in prof.values())
    top = max(prof, key=lambda k: prof[k][0])
    tms, tn = prof[top]
    per_launch_s = tms / max(tn, 1) * 1e-3
    shares = {k: round(v[0] / tot_ms, 4) for k, v in prof.items() if v[1] > 0}
    wk = work.get(top, {})
    launches_per_step = tn / args.steps
    roof = dict(kernel=top, share_of_kernel_time=shares.get(top), traffic=None, kernel_time_shares=shares)
    if top == "update" and args.workload == NCU_UPDATE_TRAFFIC["workload"] and w["bf16"]:
        roof["traffic"] = NCU_UPDATE_TRAFFIC["bytes"] * (20.0 * w["K"] + 12.0) / (20.0 * NCU_UPDATE_TRAFFIC["K"] + 12.0) if NCU_UPDATE_TRAFFIC["bytes"] else None
        roof["traffic_source"] = "ncu at K=4 scaled by (20K+12)/(20*4+12); algorithmic bytes per launch %.4g" % wk_bytes(work, "update")
    if top == "update" and flat and w["K"] == NCU_UPDATE_TRAFFIC_C5["K"] and d >= (1 << 22) and d % 8 == 0:
        roof["traffic"] = NCU_UPDATE_TRAFFIC_C5["bytes"] * d / NCU_UPDATE_TRAFFIC_C5["d"]
        roof["traffic_source"] = "ncu at d=25.6M scaled by d; algorithmic bytes per launch %.4g" % wk_bytes(work, "update")
    if top in ("gemm_fwd", "gemm_dgrad") and ctx.uses_tcgen05():
        ach = wk["flops"] / launches_per_step / per_launch_s / 1e12
        roof.update(bound="tensor", achieved=ach, peak=pk["bf16_sustained"], unit="TFLOP/s", frac=ach / pk["bf16_sustained"], peak_source=f"{pk['src']} (sustained bf16)")
    elif top.startswith("gemm") and not ctx.uses_tcgen05() and not w["bf16"]:
        ach = wk["flops"] / launches_per_step / per_launch_s / 1e12
        roof.update(bound="alu", achieved=ach, peak=FP32_ALU_TFLOPS, unit="TFLOP/s", frac=ach / FP32_ALU_TFLOPS, peak_source="148 SMs x 128 FMA lanes x 2 x 1.965 GHz")
    elif "bytes" in wk:
        ach = wk["bytes"] / launches_per_step / per_launch_s / 1e9
        roof.update(bound="hbm", achieved=ach, peak=pk["hbm"], unit="GB/s", frac=ach / pk["hbm"], peak_source=f"{pk['src']} copy bandwidth",
                    frac_of_nominal_8TBs=ach / NOMINAL_HBM_GBS)
        if "flops" in wk:
            roof["tflops"] = wk["flops"] / launches_per_step / per_launch_s / 1e12
    else:
        roof.update(bound="latency", achieved=None, peak=None, unit=None, frac=None)
    # the three streaming kernels of the fused update path, always reported
    stream_gbs = {}
    for k in ("norm", "perturb", "update"):
        if prof[k][1] > 0 and work[k]["bytes"] > 0:
            stream_gbs[k] = round(work[k]["bytes"] * args.steps / (prof[k][0] * 1e-3) / 1e9, 1)
    roof["streaming_kernels_gbs"] = stream_gbs
    gemm = {}
    for k in ("gemm_fwd", "gemm_dgrad", "gemm_wgrad"):
        if k in work and prof[k][1] > 0:
            sec = prof[k][0] * 1e-3
            gemm[k] = dict(tflops=round(work[k]["flops"] * args.steps / sec / 1e12, 1), gbs=round(work[k]["bytes"] * args.steps / sec / 1e9, 1),
                           frac_of_bf16_sustained=round(work[k]["flops"] * args.steps / sec / 1e12 / pk["bf16_sustained"], 3) if w["bf16"] else None)
    roof["gemm_classes"] = gemm

    cpu = None
    if not args.no_cpu_baseline:
        X = None if inp["X"] is None else inp["X"].cpu().numpy()
        Y = None if inp["Y"] is None else inp["Y"].cpu().numpy()
        cpu, _ = oracle_baseline(w, X, Y, inp["y0"].cpu().numpy())

    line = dict(metric=metric, value=value, unit=unit, n_gpus=world, steps=args.steps, warmup=warm, ms_per_step=ms_step,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16" if w["bf16"] else "f32", data="synthetic",
                config=dict(workload=w["name"], K=w["K"], batch=w["B"], d=d, gemm="tcgen05" if ctx.uses_tcgen05() else "simt", cuda_graph=bool(use_graph),
                            l2=("working set larger than L2" if not small else "L2-resident state (latency-bound workload)") +
                               ("" if events_in_timed else "; kernel shares and roofline from a separate pass over the same steps with per-launch events"),
                            parallelism=(f"{world * w['K']} workers sharded over {world} GPU(s), one centre, accumulator all-reduce every tau steps" if shard
                                         else ("replicas only" if world > 1 else "1 GPU"))),
                clocks=clk, e2e=e2e, gpu_launches=int(launches), roofline=roof, cpu_baseline=cpu)
    print(json.dumps(line))
    ctx.close()
    if world > 1 or shard:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
