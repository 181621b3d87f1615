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

LSQ, MLP, RESMLP, FLAT, CNN = 0, 1, 2, 3, 4

# The five workloads (shapes, replica counts, batch sizes and radii as configured).  Where a workload leaves them open:
# tau = 16 as in the paper's experiments, lambda = lambda0 / (eta tau) with lambda0 = 0.9 from the grid of Appendix D,
# beta = 0.9, eta' = 1.  (With the look-ahead beta = 0.9 and worker momentum 0.9 the worker/centre recursion alone is
# linearly unstable for short sync periods and weak pulls; tau = 16 with lambda0 = 0.9 is in its stable region.)
WORKLOADS = {
    "c1": dict(model=LSQ, widths=(256,), K=4, B=32, n=4096, classes=0, bf16=False, rho=0.05, eta=0.01, tau=4, stale_max=0,
               name="least squares 4096x256, K=4, B=32"),
    "c2": dict(model=MLP, widths=(784, 1024, 10), K=8, B=128, n=60000, classes=10, bf16=False, rho=0.05, eta=0.05, tau=16,
               stale_max=0, name="MLP 784-1024-10 fp32, K=8, B=128"),
    "c3": dict(model=MLP, widths=(3072, 2048, 2048, 2048, 100), K=16, B=128, n=50000, classes=100, bf16=True, rho=0.1,
               eta=0.01, tau=16, stale_max=0, name="MLP 3072-2048x3-100 bf16 GEMM, K=16, B=128"),
    "c4": dict(model=RESMLP, widths=(3072, 4096, 4096, 4096, 4096, 1000), K=32, B=256, n=200000, classes=1000, bf16=True,
               rho=0.1, eta=0.002, tau=16, stale_max=3, head_scale=0.1, res_scale=0.25, name="residual MLP 3072-4096x4-1000 bf16 GEMM, K=32, B=256, staleness [0,3]"),
    # a convolutional second workload with the image shape of the paper's CIFAR runs (its own conv nets are not reproduced):
    # two 3x3 convolution + ReLU + 2x2 max-pooling layers (3 -> 32 -> 64 channels), then dense 4096 -> 256 -> 10
    "cnn": dict(model=CNN, widths=(3, 32, 64, 256, 10), n_conv=2, img=(32, 32), K=4, B=64, n=50000, classes=10, bf16=False, rho=0.05, eta=0.002, tau=16, head_scale=0.1,
                stale_max=0, name="CNN 3x32x32 conv32-conv64-256-10 fp32, K=4, B=64"),
    "c5": dict(model=FLAT, widths=(), K=8, B=0, n=0, classes=0, bf16=False, rho=0.1, eta=0.05, tau=16, stale_max=0, d=256_000_000,
               name="optimiser-only sweep point d=256M, K=8"),
}
LAMBDA0, MU, BETA, ETA_PRIME, GAMMA = 0.9, 0.9, 0.9, 1.0, 1e-12
NOMINAL_HBM_GBS, FALLBACK_HBM_GBS, FALLBACK_BF16_TF = 8000.0, 6650.0, 1590.0
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12  # SMs x FMA lanes x 2 flop x max SM clock
# ncu DRAM counters of one launch of the two update kernels live beside the summaries they were read from (profiles/);
# they are scaled to the launch that is timed by its algorithmic bytes (20 K + 12) d.
NCU_TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic.json")
# The sample of each workload that the CPU oracle is timed on (fixed, so that the figure is a stable denominator):
# replicas, samples per minibatch, steps.  The full model is always used.
ORACLE_SAMPLE = {"c1": (4, 32, 20), "c2": (8, 16, 2), "c3": (2, 16, 1), "c4": (2, 8, 1), "cnn": (4, 16, 1)}


def ncu_traffic(kernel, K, d):
    """Measured DRAM bytes of one launch of `kernel`, scaled from the captured case to (K, d); None if not on record."""
    try:
        rec = json.load(open(NCU_TRAFFIC_FILE))[kernel]
    except Exception:
        return None, None
    scale = (20.0 * K + 12.0) * d / ((20.0 * rec["K"] + 12.0) * rec["d"])
    return rec["bytes"] * scale, f"ncu capture at K={rec['K']}, d={rec['d']} ({rec['source']}) scaled by (20K+12)d"


def gemm_layers(w):
    """(positions per sample, in, out) of every weight matrix: a dense layer has one position per sample, a 3x3 convolution H x W of them."""
    ws = w["widths"]
    if w["model"] != CNN:
        return [(1, ws[i], ws[i + 1]) for i in range(len(ws) - 1)]
    H, W = w["img"]
    out = []
    for l in range(w["n_conv"]):
        out.append((H * W, ws[l] * 9, ws[l + 1]))
        H, W = H // 2, W // 2
    feat = ws[w["n_conv"]] * H * W
    for l in range(w["n_conv"], len(ws) - 1):
        out.append((1, feat if l == w["n_conv"] else ws[l], ws[l + 1]))
    return out


def param_count(w):
    if w["model"] == FLAT:
        return w["d"]
    if w["model"] == LSQ:
        return w["widths"][0]
    return sum(i * o + o for _, i, o in gemm_layers(w))


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
def work_model(w, tc, grads_bf16=None):
    """Algorithmic bytes / flops per STEP of each kernel class (what the launched kernels must move or compute).
    grads_bf16: the tensor-core path stores both gradients in bf16 (its default), 2 instead of 4 bytes per element."""
    K, B, d = w["K"], w["B"], param_count(w)
    op = 2 if w["bf16"] else 4
    gb = 2.0 if (tc if grads_bf16 is None else grads_bf16) else 4.0
    out = {}
    out["norm"] = dict(bytes=0.0 if tc else 4.0 * K * d)                     # read g1 (fused into the wgrad epilogue on the tensor-core path)
    out["perturb"] = dict(bytes=(4.0 + gb + op) * K * d)                     # read x, g1; write x~
    out["update"] = dict(bytes=(gb + 8.0 + 8.0 + (2.0 if w["bf16"] else 0.0)) * K * d + 12.0 * d)  # g2, x rw, v rw, operand copy; y, acc rw
    if w["model"] in (MLP, RESMLP, CNN):
        f_fwd = f_dg = f_wg = 0.0
        b_fwd = b_dg = b_wg = 0.0
        for l, (pos, i, o) in enumerate(gemm_layers(w)):
            Bp = B * pos                                                    # rows of the GEMM: samples x positions
            f_fwd += 2.0 * Bp * i * o
            b_fwd += op * (i * o + Bp * i + Bp * o)
            f_wg += 2.0 * Bp * i * o
            b_wg += gb * i * o + op * Bp * (i + o)                          # the gradient is written in its storage type
            if l > 0:
                f_dg += 2.0 * Bp * i * o
                b_dg += op * (i * o + Bp * i + Bp * o)
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
    n, fin = w["n"], (w["widths"][0] * w["img"][0] * w["img"][1] if w["model"] == CNN else w["widths"][0])
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
        shapes = gemm_layers(w)
        for l, (_, fan_in, fan_out) in enumerate(shapes):
            scale = (2.0 / fan_in) ** 0.5
            if l == len(shapes) - 1:
                scale *= w.get("head_scale", 1.0)       # small head: the initial loss starts near log(classes)
            elif w["model"] == RESMLP and ws[l] == ws[l + 1]:
                scale *= w.get("res_scale", 1.0)        # damped residual branches: no normalisation layers here
            parts.append((torch.randn(fan_out, fan_in, device=dev, generator=g) * scale).reshape(-1))
            parts.append(torch.zeros(fan_out, device=dev))
        w0 = torch.cat(parts)
    x0 = w0.unsqueeze(0).expand(K, -1).contiguous()
    return dict(X=X, Y=Y, x0=x0, y0=w0)


def make_cfg(G, w, flags=0, K_total=0, k_offset=0, gemm_impl=0):
    lam = w.get("lambda0", LAMBDA0) / (w["eta"] * w["tau"])
    return G.make_config(w["model"], widths=w["widths"], K=w["K"], batch=max(w["B"], 1) if w["model"] != FLAT else 0,
                         gemm_dtype=G.GEMM_BF16 if w["bf16"] else G.GEMM_FP32, mu=MU, nesterov=1, gamma=GAMMA, lam=lam, tau=w["tau"],
                         beta=BETA, eta_prime=ETA_PRIME, stale_max=w["stale_max"], seed=0, n_samples=max(w["n"], 1),
                         flat_d=w.get("d", 0), flags=flags, active_num=w.get("active_num", 256), gemm_impl=gemm_impl,
                         noise_temp=w.get("noise_temp", 0.0), K_total=K_total, k_offset=k_offset,
                         n_conv=w.get("n_conv", 0), img_h=w.get("img", (0, 0))[0], img_w=w.get("img", (0, 0))[1])


# ---------------------------------------------------------------------------------------------- CPU oracle leg
class OracleSample:
    """The oracle, as it stands, on a fixed bounded sample of the workload: a subset of the replicas and of each
    minibatch, the full model.  timed_steps() runs `steps` ticks of it (centre updates included when due) and returns
    the baseline record and the seconds per tick."""

    def __init__(self, w, key, X, Y, x0_row):
        import oracle as O

        self.w, self.O = w, O
        self.cores = O.num_threads()
        d = param_count(w)
        lam = w.get("lambda0", LAMBDA0) / (w["eta"] * w["tau"])
        if w["model"] == FLAT:
            self.Ks, self.ds, self.steps = w["K"], min(d, 4_000_000), 3
            cfg = O.make_config(O.MODEL_FLAT, K=self.Ks, flat_d=self.ds, mu=MU, gamma=GAMMA, lam=lam, tau=w["tau"], beta=BETA, eta_prime=ETA_PRIME)
            rng = np.random.default_rng(0)
            x0 = rng.standard_normal((self.Ks, self.ds))
            g1 = (0.1 * rng.standard_normal((self.Ks, self.ds))).astype(np.float32)
            self.o = O.Oracle(cfg, None, None, x0, x0.mean(0))
            self.o.set_external_grads(g1, g1)
            self.sample = f"K={self.Ks} replicas, d={self.ds} of {d} elements, {self.steps} steps per timing"
        else:
            Ks, Bs, self.steps = ORACLE_SAMPLE[key]
            self.Ks, self.Bs = min(Ks, w["K"]), min(Bs, w["B"])
            cfg = O.make_config(w["model"], widths=w["widths"], K=self.Ks, batch=self.Bs, gemm_dtype=O.GEMM_BF16 if w["bf16"] else O.GEMM_FP32, mu=MU,
                                gamma=GAMMA, lam=lam, tau=w["tau"], beta=BETA, eta_prime=ETA_PRIME, stale_max=w["stale_max"], seed=0, n_samples=w["n"],
                                n_conv=w.get("n_conv", 0), img_h=w.get("img", (0, 0))[0], img_w=w.get("img", (0, 0))[1])
            x0 = np.repeat(x0_row[None, :].astype(np.float64), self.Ks, axis=0)
            self.o = O.Oracle(cfg, X, Y, x0, x0_row.astype(np.float64))
            self.sample = f"{self.Ks} of {w['K']} replicas x {self.Bs} of {w['B']} samples per minibatch, full model, {self.steps} step(s) per timing"

    def timed_steps(self):
        w, o = self.w, self.o
        t0 = time.perf_counter()
        for _ in range(self.steps):
            o.step(w["eta"], w["rho"])
            if o.should_couple():
                o.couple()
        dt = (time.perf_counter() - t0) / self.steps
        if w["model"] == FLAT:
            rec = dict(value=36.0 * self.Ks * self.ds / dt / 1e9, unit="GB/s (36 B per element-replica)")
        else:
            rec = dict(value=self.Ks * self.Bs / dt, unit="worker-samples/s")
        rec.update(cores=min(self.cores, self.Ks), kind="oracle", sample=self.sample)
        return rec, dt

    def close(self):
        self.o.close()


def oracle_baseline(w, key, X, Y, x0_row):
    s = OracleSample(w, key, X, Y, x0_row)
    out = s.timed_steps()
    s.close()
    return out


def run_reference(args, w, metric, unit):
    """--impl reference: the CPU oracle timed on the fixed bounded sample of the same workload (rank 0 only); every
    warm-up or timed step of the run is one timing of that sample, on one oracle run that keeps going."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import torch

    inp = make_inputs(w, torch.device("cpu"), seed=0)
    X = None if inp["X"] is None else inp["X"].numpy()
    Y = None if inp["Y"] is None else inp["Y"].numpy()
    smp = OracleSample(w, args.workload, X, Y, inp["y0"].numpy())
    vals, dts = [], []
    for i in range(args.warmup + args.steps):
        cb, dt = smp.timed_steps()
        if i >= args.warmup:
            vals.append(cb["value"])
            dts.append(dt)
    smp.close()
    v = float(np.mean(vals))
    cb["value"] = v
    line = dict(impl="reference", metric=metric, value=v, unit=unit, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=float(np.mean(dts) * 1e3), higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64",
                data="synthetic", config=workload_config(w), cpu_baseline=cb,
                e2e=dict(value=v, unit=unit, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def workload_config(w):
    """The keys that name the workload; shared by both arms so that their records compare like with like."""
    return dict(workload=w["name"], K=w["K"], batch=w["B"], d=param_count(w))


# ---------------------------------------------------------------------------------------------- one workload on this rank's GPU
def run_workload(key, w, steps, warmup, dev, rank, world, shard=False, cuda_graph="auto", grad_fp32=False, with_e2e=True, with_cpu=True, gemm_impl=0, fused_update=False, pdl=False):
    """Create the context, time `steps` steps after `warmup` untimed ones, and return the record of this workload
    (rank 0; None on the other ranks).  A step is one pass of the whole hot path plus the centre update when it is due."""
    import torch
    import torch.distributed as dist

    from paper_2509_03110_b200 import binding as G

    flat = w["model"] == FLAT
    unit = "GB/s" if flat else "worker-samples/s"
    local = dev.index
    # sharded: every rank generates the same dataset and the same initial point (one job); else independent copies
    inp = make_inputs(w, dev, seed=0 if shard else rank)
    # Each tick is replayed as one CUDA graph (auto: always): the 30-40 launches of a tick leave gaps that are a visible share
    # of the step for the latency-bound workloads (C1: 38.6 -> 25.8 us) and still 1 % at the largest one (16.45 -> 16.26 ms).
    # That needs a capturable stream; the per-kernel shares then come from a second pass over the same steps with per-launch events.
    small = 4.0 * w["K"] * param_count(w) <= 126e6
    use_graph = (not fused_update) if cuda_graph == "auto" else cuda_graph == "on"
    flags = (G.FLAG_CUDA_GRAPH if use_graph else 0) | (G.FLAG_GRAD_FP32 if grad_fp32 else 0) | (G.FLAG_FUSED_UPDATE if fused_update else 0) | (G.FLAG_PDL if pdl else 0)
    cfg = make_cfg(G, w, flags=flags, K_total=world * w["K"] if shard else 0, k_offset=rank * w["K"] if shard else 0, gemm_impl=gemm_impl)
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
    for _ in range(warmup):
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
    for _ in range(steps):
        one_step()
    e1.record(stream)
    barrier()
    clk = clocks.stop()
    ms = e0.elapsed_time(e1)
    worker_iters_per_step = (iterations_done() - it0) / steps  # = K in lock-step mode
    if not events_in_timed:
        launches_timed = ctx.launch_count() - launches0
        ctx.profile_enable(True)
        for _ in range(min(steps, 50)):
            one_step()
        barrier()
        launches0 = ctx.launch_count() - launches_timed
    prof_steps = steps if events_in_timed else min(steps, 50)
    prof = ctx.profile_read()
    ctx.profile_enable(False)
    launches = ctx.launch_count() - launches0
    st = ctx.status()
    if st != 0:
        raise SystemExit(f"{w['name']}: device status word is not clean after the timed region (lsam_status = {st}: {ctx.last_error()})")
    ms = max_over_ranks(ms, world, dev)
    ms_step = ms / steps
    units_step = (36.0 * worker_iters_per_step * d / 1e9) if flat else float(worker_iters_per_step * w["B"])
    value = whole_job_value(world, units_step, ms_step)

    # ---- end to end through the C ABI with host buffers (minibatch H2D and loss D2H inside the timed region)
    e2e = None
    if with_e2e and not flat:
        nst = min(steps, 8)
        nb = min(nst, 4)
        fin = inp["X"].shape[1]
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
    elif with_e2e:
        # optimiser-only: the gradients are the step's inputs; copy them from pinned host memory every step
        K = w["K"]
        hg = torch.empty(2, K, d, dtype=torch.float32).pin_memory() if d <= 64_000_000 else None
        if hg is not None:
            hg[0].copy_(inp["g1"].cpu())
            hg[1].copy_(inp["g2"].cpu())
            barrier()
            nst = min(steps, 5)
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

    uses_tc = ctx.uses_tcgen05()
    x3 = uses_tc and not w.get("bf16", False)  # fp32 GEMMs as six bf16 plane-pair products on the tensor cores
    grads_bf16 = uses_tc and not x3 and not grad_fp32
    if rank != 0:
        ctx.close()
        return None

    # ---- roofline of the dominant kernel class
    pk = peaks()
    work = work_model(w, uses_tc, grads_bf16)
    frac_active = worker_iters_per_step / w["K"]  # waiting replicas are skipped by every kernel
    for wk_ in work.values():
        for k2 in wk_:
            wk_[k2] *= frac_active
    tot_ms = sum(v[0] for v in prof.values())
    top = max(prof, key=lambda k: prof[k][0])
    tms, tn = prof[top]
    per_launch_s = tms / max(tn, 1) * 1e-3
    shares = {k: round(v[0] / tot_ms, 4) for k, v in prof.items() if v[1] > 0}
    wk = work.get(top, {})
    launches_per_step = tn / prof_steps
    roof = dict(kernel=top, share_of_kernel_time=shares.get(top), traffic=None, kernel_time_shares=shares)
    if top == "update" and frac_active == 1.0:
        # which update kernel ran: bf16 gradients (padded rows, always multiples of 8) / long fp32 rows / the 4-per-thread form
        kern = "update8_kernel" if grads_bf16 else ("update8f_kernel" if (flat and d >= (1 << 22) and d % 8 == 0) else None)
        if kern:
            roof["traffic"], roof["traffic_source"] = ncu_traffic(kern, w["K"], d)
    if top.startswith("gemm") and x3:
        # the fp32-equivalent rate against the sustained bf16 rate divided by the six bf16 products each fp32 product costs
        ach = wk["flops"] / launches_per_step / per_launch_s / 1e12
        roof.update(bound="tensor", achieved=ach, peak=pk["bf16_sustained"] / 6, unit="TFLOP/s", frac=ach / (pk["bf16_sustained"] / 6),
                    peak_source=f"{pk['src']} (sustained bf16) / 6 plane-pair products per fp32 product")
    elif top in ("gemm_fwd", "gemm_dgrad") and uses_tc:
        ach = wk["flops"] / launches_per_step / per_launch_s / 1e12
        roof.update(bound="tensor", achieved=ach, peak=pk["bf16_sustained"], unit="TFLOP/s", frac=ach / pk["bf16_sustained"], peak_source=f"{pk['src']} (sustained bf16)")
    elif top.startswith("gemm") and not uses_tc and not w["bf16"]:
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
            gbs = work[k]["bytes"] * prof_steps / (prof[k][0] * 1e-3) / 1e9
            stream_gbs[k] = dict(gbs=round(gbs, 1), frac_of_measured_hbm=round(gbs / pk["hbm"], 3), frac_of_nominal_8TBs=round(gbs / NOMINAL_HBM_GBS, 3))
    roof["streaming_kernels"] = stream_gbs
    gemm = {}
    for k in ("gemm_fwd", "gemm_dgrad", "gemm_wgrad"):
        if k in work and prof[k][1] > 0:
            sec = prof[k][0] * 1e-3
            tf = work[k]["flops"] * prof_steps / sec / 1e12
            gbs = work[k]["bytes"] * prof_steps / sec / 1e9
            gemm[k] = dict(tflops=round(tf, 1), gbs=round(gbs, 1),
                           frac_of_bf16_sustained=round(tf / pk["bf16_sustained"], 3) if w["bf16"] else None,
                           frac_of_bf16_burst=round(tf / pk["bf16"], 3) if w["bf16"] else None,
                           frac_of_measured_hbm=round(gbs / pk["hbm"], 3))
            if w["bf16"]:
                # which roof the shape sits under (flop per algorithmic byte against the ridge of the two measured peaks), and the
                # fraction of that roof: time at the roof / measured time
                t_tensor, t_hbm = tf / pk["bf16_sustained"], gbs / pk["hbm"]
                gemm[k].update(bound="tensor" if t_tensor >= t_hbm else "hbm", frac_of_roofline=round(max(t_tensor, t_hbm), 3))
    roof["gemm_classes"] = gemm
    # the whole step against both roofs: algorithmic bytes and flops of every kernel class over the device-timed step
    # (the kernels run one after another, so the sum of the per-kernel floors, not their maximum, bounds the step)
    step_bytes = sum(v.get("bytes", 0.0) for v in work.values())
    step_flops = sum(v.get("flops", 0.0) for v in work.values())
    if step_bytes > 0 and not small:
        floor_s = sum(max(v.get("bytes", 0.0) / (pk["hbm"] * 1e9), (v.get("flops", 0.0) / (pk["bf16_sustained"] * 1e12)) if (uses_tc and not x3) else 0.0)
                      for v in work.values())
        roof["whole_step"] = dict(bytes=step_bytes, flops=step_flops, gbs=round(step_bytes / (ms_step * 1e-3) / 1e9, 1),
                                  frac_of_measured_hbm=round(step_bytes / (ms_step * 1e-3) / 1e9 / pk["hbm"], 3),
                                  floor_ms=round(floor_s * 1e3, 3), frac_of_floor=round(floor_s * 1e3 / ms_step, 3),
                                  floor="sum over the kernel classes of max(bytes / measured HBM rate, flops / sustained bf16 rate)")

    cpu = None
    if with_cpu:
        X = None if inp["X"] is None else inp["X"].cpu().numpy()
        Y = None if inp["Y"] is None else inp["Y"].cpu().numpy()
        cpu, _ = oracle_baseline(w, key, X, Y, inp["y0"].cpu().numpy())

    cfgd = workload_config(w)
    cfgd.update(gemm=("tcgen05, fp32 as three bf16 planes per operand" if x3 else "tcgen05 (single-CTA kernels only)" if gemm_impl == G.IMPL_TCGEN05_1CTA else "tcgen05") if uses_tc else "simt", cuda_graph=bool(use_graph), pdl=bool(pdl),
                l2=("working set larger than L2" if not small else "L2-resident state (latency-bound workload)") +
                   ("" if events_in_timed else "; kernel shares and roofline from a separate pass over the same steps with per-launch events"),
                parallelism=(f"{world * w['K']} workers sharded over {world} GPU(s), one centre, accumulator all-reduce every tau steps" if shard
                             else ("replicas only" if world > 1 else "1 GPU")))
    if w["bf16"]:
        cfgd["grad_storage"] = "bf16" if grads_bf16 else "fp32"
    rec = dict(metric="fused_update_hbm_gbs" if flat else "lsam_worker_samples_per_s", value=value, unit=unit, ms_per_step=ms_step,
               dtype="bf16" if w["bf16"] else "f32", config=cfgd, clocks=clk, e2e=e2e, gpu_launches=int(launches), roofline=roof, cpu_baseline=cpu)
    ctx.close()
    return rec


# What the default invocation measures after the headline workload, a few hundred milliseconds each, so that one run carries
# the whole metric: the optimiser-only sweep at its five sizes and the three smaller model workloads.
OTHER_WORKLOADS = [("c5", dict(d=1_000_000), 1000), ("c5", dict(d=11_200_000), 300), ("c5", dict(d=25_600_000), 150), ("c5", dict(d=86_000_000), 50),
                   ("c5", dict(d=256_000_000), 20), ("c1", {}, 95), ("c2", {}, 400), ("c3", {}, 100), ("cnn", {}, 100)]


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
    ap.add_argument("--others", default="auto", choices=["auto", "on", "off"],
                    help="also time the sweep sizes and the smaller workloads (auto: on one GPU with the default workload)")
    ap.add_argument("--replicas", type=int, default=None, help="override K (small cases for profiler captures)")
    ap.add_argument("--noise-temp", type=float, default=0.0, help="Langevin temperature of the sampler (0 = none)")
    ap.add_argument("--active-num", type=int, default=256, help="asynchronous progress: a worker is ready at a tick with probability N/256")
    ap.add_argument("--grad-fp32", action="store_true", help="tensor-core path: store the gradients in fp32 instead of bf16")
    ap.add_argument("--fused-update", action="store_true", help="tensor-core path: worker update of the weights inside the descent-pass weight-gradient epilogue")
    ap.add_argument("--gemm-impl", default="auto", choices=["auto", "simt", "tcgen05", "tcgen05-1cta", "tcgen05-pairs"],
                    help="auto: tensor-core GEMMs for the bf16 workloads (CTA pairs where a GEMM is large enough); tcgen05-1cta: single-CTA kernels only")
    ap.add_argument("--shard-workers", action="store_true",
                    help="N > 1: one job of N*K workers with a single centre, K workers per GPU, accumulator all-reduce every tau steps "
                         "(default: N independent copies of the workload)")
    ap.add_argument("--cuda-graph", default="auto", choices=["auto", "on", "off"], help="replay each tick as one CUDA graph (auto: on)")
    ap.add_argument("--pdl", default="on", choices=["on", "off"], help="launch the kernels of a tick with programmatic stream serialization (LSAM_FLAG_PDL)")
    args = ap.parse_args()
    w = dict(WORKLOADS[args.workload])
    modified = False
    if args.flat_d and w["model"] == FLAT:
        w["d"] = args.flat_d
        w["name"] = f"optimiser-only sweep point d={args.flat_d}, K=8"
    if args.replicas:
        w["K"] = args.replicas
        w["name"] += f" [K overridden to {args.replicas}]"
        modified = True
    if args.noise_temp > 0.0:
        w["noise_temp"] = args.noise_temp
        w["name"] += f" [Langevin temperature {args.noise_temp}]"
        modified = True
    if args.active_num != 256:
        w["active_num"] = args.active_num
        w["name"] += f" [workers ready with probability {args.active_num}/256 per tick]"
        modified = True
    flat = w["model"] == FLAT
    metric = "fused_update_hbm_gbs" if flat else "lsam_worker_samples_per_s"
    unit = "GB/s" if flat else "worker-samples/s"
    if args.impl == "reference":
        return run_reference(args, w, metric, unit)

    import torch
    import torch.distributed as dist

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

    rec = run_workload(args.workload, w, args.steps, args.warmup, dev, rank, world, shard=shard, cuda_graph=args.cuda_graph,
                       grad_fp32=args.grad_fp32, with_e2e=True, with_cpu=not args.no_cpu_baseline, fused_update=args.fused_update, pdl=args.pdl == "on",
                       gemm_impl={"auto": 0, "simt": 1, "tcgen05": 2, "tcgen05-1cta": 3, "tcgen05-pairs": 4}[args.gemm_impl])
    others = []
    modified = modified or args.gemm_impl != "auto" or args.grad_fp32 or args.fused_update or args.pdl != "on"
    want_others = args.others == "on" or (args.others == "auto" and world == 1 and args.workload == "c4" and not modified and not shard)
    if want_others and world == 1:
        for key, over, nsteps in OTHER_WORKLOADS:
            torch.cuda.empty_cache()
            ow = dict(WORKLOADS[key])
            ow.update(over)
            if "d" in over:
                ow["name"] = f"optimiser-only sweep point d={over['d']}, K={ow['K']}"
            r = run_workload(key, ow, nsteps, 5, dev, rank, world, cuda_graph="auto", with_e2e=False, with_cpu=False, pdl=args.pdl == "on")
            ro = r["roofline"]
            others.append(dict(workload=r["config"]["workload"], metric=r["metric"], value=r["value"], unit=r["unit"], ms_per_step=r["ms_per_step"], steps=nsteps, warmup=5,
                               config=r["config"], clocks=r["clocks"], gpu_launches=r["gpu_launches"],
                               roofline=dict(kernel=ro["kernel"], bound=ro.get("bound"), achieved=ro.get("achieved"), peak=ro.get("peak"), unit=ro.get("unit"),
                                             frac=ro.get("frac"), traffic=ro.get("traffic"), share_of_kernel_time=ro.get("share_of_kernel_time"),
                                             streaming_kernels=ro.get("streaming_kernels"), gemm_classes=ro.get("gemm_classes"))))
    if rank == 0:
        line = dict(metric=rec["metric"], value=rec["value"], unit=rec["unit"], n_gpus=world, steps=args.steps, warmup=args.warmup, ms_per_step=rec["ms_per_step"],
                    higher_is_better=True, scaling="weak", vs_baseline=None, dtype=rec["dtype"], data="synthetic", config=rec["config"], clocks=rec["clocks"],
                    e2e=rec["e2e"], gpu_launches=rec["gpu_launches"], roofline=rec["roofline"], cpu_baseline=rec["cpu_baseline"])
        if others:
            line["other_workloads"] = others
        print(json.dumps(line))
    if world > 1 or shard:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
