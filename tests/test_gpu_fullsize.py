"""Parity at the full benchmark shapes, in the configuration bench.py times, on outputs the oracle can compute a few
replicas at a time: the CUDA library runs whole ticks (all K replicas, full minibatches, tensor-core GEMMs, bf16
gradient storage); the oracle, which keeps both gradients unrounded, recomputes selected replicas from the same inputs
and schedule.  Between syncs the workers are independent, and before the first sync every centre read is y0, so the
free run of a subset of the workers is exactly what those workers do inside the full job."""
import os
import sys
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

import oracle as O
from harness import BULK_DIVISOR, median_abs_rows, rel_l2
from paper_2509_03110_b200 import binding as G

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402  (workload table and seeded device-side input recipe)

pytestmark = pytest.mark.gpu

# Gradient tolerance of one tick at full size (relative L2 of the whole flat gradient of a replica).  The tensor cores
# accumulate fp32 with truncated alignment, the oracle in double: a pre-activation within ~1e-5 relative of zero takes
# the other ReLU branch, a stored activation within that distance of a bf16 rounding boundary takes the other value, and
# every such difference perturbs the backward signal of its sample, so the error grows from the head towards the first
# layer.  Measured at the 3072-2048x3-100 shape (tick 0, replicas 0 and 15), per weight matrix from the first layer to the
# head: ascent gradient up to 1.9e-2 / 1.4e-2 whole vector; descent gradient (at the perturbed point, a sharper region)
# 3.9e-2, 2.8e-2, 1.7e-2, 2.3e-3 / 2.1e-2 whole vector.  The paper states no per-step figure for bf16 paths; this bound is
# a reading: 1.5 x the trajectory figure it does state (2e-2), which the iterates themselves meet below.  The loss, which
# no flip can move discontinuously, is held to 1e-4 and the gradient norm to 2e-3.
TOL_GRAD_BF16_FULL = 3e-2
TOL_TRAJ_BF16 = 2e-2


def _oracle_cfg(w, K, **over):
    lam = w.get("lambda0", bench.LAMBDA0) / (w["eta"] * w["tau"])
    kw = dict(widths=w["widths"], K=K, batch=w["B"], gemm_dtype=O.GEMM_BF16, mu=bench.MU, gamma=bench.GAMMA, lam=lam, tau=w["tau"],
              beta=bench.BETA, eta_prime=bench.ETA_PRIME, stale_max=w["stale_max"], seed=0, n_samples=w["n"])
    kw.update(over)
    return O.make_config(w["model"], **kw)


def _layer_errors(widths, got, want):
    """Relative L2 error of each weight matrix of the flat gradient (diagnostic for the assertion messages)."""
    out, off = [], 0
    for i, o in zip(widths[:-1], widths[1:]):
        n = i * o
        out.append(round(rel_l2(got[off:off + n], want[off:off + n]), 5))
        off += n + o
    return out


def _inputs(w, dev, K=None):
    import torch

    w = dict(w)
    if K is not None:
        w["K"] = K
    inp = bench.make_inputs(w, dev, seed=0)
    # replicas start apart so that a replica mix-up cannot go unnoticed
    gen = torch.Generator(device=dev).manual_seed(123)
    inp["x0"] += 0.001 * torch.randn(inp["x0"].shape, device=dev, generator=gen)
    return w, inp


def test_c3_full_shape_sixteen_free_running_ticks_of_two_replicas():
    # 3072-2048x3-100, K = 16, B = 128, tau = 16: the library free-runs all 16 workers for one whole sync period; the oracle
    # free-runs workers 0 and 15 (same schedule streams through their global indices).  Per tick: minibatch loss; tick 0:
    # both gradients and the perturbed point; after 16 ticks: iterates, momentum, and the displacement x_16 - x_0.
    import torch

    dev = torch.device("cuda", 0)
    w, inp = _inputs(bench.WORKLOADS["c3"], dev)
    K, ticks = w["K"], w["tau"]
    picks = [0, K - 1]
    x0_rows = np.stack([inp["x0"][k].cpu().numpy().astype(np.float64) for k in picks])
    y0_row = inp["y0"].cpu().numpy().astype(np.float64)
    ctx = G.Lsam(bench.make_cfg(G, w, flags=G.FLAG_KEEP_G1 | G.FLAG_STEP_INFO), inp["X"], inp["Y"], inp["x0"], inp["y0"])
    assert ctx.uses_tcgen05()
    inp["x0"] = None
    torch.cuda.empty_cache()
    gl, gn1, gn2, first = [], [], [], None
    for t in range(ticks):
        ctx.step(w["eta"], w["rho"])
        l, n1, n2 = ctx.read_step_info()
        gl.append(l[picks]); gn1.append(n1[picks]); gn2.append(n2[picks])
        if t == 0:
            first = dict(g1=[ctx.read_grads_replica(1, k) for k in picks], g2=[ctx.read_grads_replica(2, k) for k in picks],
                         xp=[ctx.read_grads_replica(3, k) for k in picks], idx=ctx.read_schedule(0)[0])
    assert ctx.status() == 0 and ctx.should_couple()
    gx = np.stack([ctx.read_params(k) for k in picks]).astype(np.float64)
    gv = ctx.read_state()["v"][picks].astype(np.float64)

    o = O.Oracle(_oracle_cfg(w, len(picks)), inp["X"].cpu().numpy(), inp["Y"].cpu().numpy(), x0_rows, y0_row, replica_ids=picks)
    for t in range(ticks):
        o.step(w["eta"], w["rho"])
        ol, on1, on2 = o.read_step_info()
        # tick 0 starts from the same state: loss 1e-4, gradient norms 2e-3; afterwards the two runs are free and these
        # scalars are functions of iterates that agree to the trajectory tolerance
        np.testing.assert_allclose(gl[t], ol, rtol=1e-4 if t == 0 else TOL_TRAJ_BF16, err_msg=f"loss at tick {t}")
        if t == 0:  # (later gradient norms are steep functions of the iterates in this regime: |g| = 30 ... 60 and a rising loss)
            np.testing.assert_allclose(gn1[t], on1, rtol=2e-3, err_msg="|g1| at tick 0")
            np.testing.assert_allclose(gn2[t], on2, rtol=2e-3, err_msg="|g2| at tick 0")
        if t == 0:
            np.testing.assert_array_equal(o.read_schedule(0)[0], first["idx"][picks])
            og1, og2, oxp = o.read_grads()
            oxp16 = torch.from_numpy(oxp.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()  # stored as the bf16 operand
            for i, k in enumerate(picks):
                for name, got, want in (("g1", first["g1"][i], og1[i]), ("g2", first["g2"][i], og2[i])):
                    e = rel_l2(got, want)
                    assert e <= TOL_GRAD_BF16_FULL, (name, k, e, _layer_errors(w["widths"], got, want))
                assert rel_l2(first["xp"][i], oxp16[i]) <= 1e-3
    assert o.should_couple()
    s = o.read_state()
    lam = w.get("lambda0", bench.LAMBDA0) / (w["eta"] * w["tau"])
    for i, k in enumerate(picks):
        assert rel_l2(gx[i], s["x"][i]) <= TOL_TRAJ_BF16, (k, rel_l2(gx[i], s["x"][i]))
        assert median_abs_rows(gx[i], s["x"][i]) <= TOL_TRAJ_BF16 / BULK_DIVISOR
        # the iterates barely move against their own norm in 16 ticks; the path travelled is the sharper quantity.  It is a
        # sum of gradient steps (and so is the momentum buffer), so it inherits the per-tick gradient bound
        moved = rel_l2(gx[i] - x0_rows[i], s["x"][i] - x0_rows[i])
        assert moved <= TOL_GRAD_BF16_FULL, (k, moved)
        # momentum buffer: a geometric sum (ratio mu) of G = g2 + lambda (x - y), bounded on the scale of its inputs
        scale = (lam * np.linalg.norm(s["x"][i]) + on2[i]) / (1.0 - bench.MU)
        assert np.linalg.norm(gv[i] - s["v"][i]) <= TOL_TRAJ_BF16 * scale, (k, np.linalg.norm(gv[i] - s["v"][i]) / scale)
    ctx.close()
    o.close()


def test_c4_full_widths_two_replicas_sync_every_tick_with_stale_reads():
    # 3072-4096x4-1000 at full widths with K = 2, B = 256, staleness [0, 3] and tau = 1: three ticks with a centre update after
    # each, both replicas in the oracle, so that full-size tiles, lsam_couple at d = 67 M and a stale centre read (s > 0 reaching
    # an older version than the current one) are all checked against the oracle.
    import torch

    dev = torch.device("cuda", 0)
    # lambda0 / 16 keeps the pull strength lambda = lambda0 / (eta tau) of the tau = 16 workload
    w, inp = _inputs(dict(bench.WORKLOADS["c4"], tau=1, lambda0=bench.LAMBDA0 / 16), dev, K=2)
    K, ticks = 2, 3
    x0 = inp["x0"].cpu().numpy().astype(np.float64)
    y0 = inp["y0"].cpu().numpy().astype(np.float64)
    ctx = G.Lsam(bench.make_cfg(G, w, flags=G.FLAG_STEP_INFO), inp["X"], inp["Y"], inp["x0"], inp["y0"])
    assert ctx.uses_tcgen05()
    o = O.Oracle(_oracle_cfg(w, K), inp["X"].cpu().numpy(), inp["Y"].cpu().numpy(), x0, y0)
    stale_hit = False
    for t in range(ticks):
        ctx.step(w["eta"], w["rho"])
        o.step(w["eta"], w["rho"])
        gi, gs, gv = ctx.read_schedule(t)
        oi, os_, ov = o.read_schedule(t)
        np.testing.assert_array_equal(gi, oi)
        np.testing.assert_array_equal(gs, os_)
        np.testing.assert_array_equal(gv, ov)
        stale_hit |= bool((gv < t).any())  # with a sync after every tick the current version is t
        gl, gn1, gn2 = ctx.read_step_info()
        ol, on1, on2 = o.read_step_info()
        np.testing.assert_allclose(gl, ol, rtol=1e-4 if t == 0 else TOL_TRAJ_BF16, err_msg=f"loss at tick {t}")
        if t == 0:
            np.testing.assert_allclose(gn1, on1, rtol=2e-3)
            np.testing.assert_allclose(gn2, on2, rtol=2e-3)
        if t == 0:
            _, og2, _ = o.read_grads()
            for k in range(K):
                got = ctx.read_grads_replica(2, k)
                e = rel_l2(got, og2[k])
                assert e <= TOL_GRAD_BF16_FULL, ("g2", k, e, _layer_errors(w["widths"], got, og2[k]))
        assert ctx.should_couple() and o.should_couple()
        assert ctx.couple() == 0 and o.couple() == 0
    assert stale_hit, "the seeded schedule never read an older centre version in these ticks"
    assert ctx.status() == 0
    s = o.read_state()
    gy = ctx.read_params(-1).astype(np.float64)
    assert rel_l2(gy, s["y"]) <= TOL_TRAJ_BF16
    assert rel_l2(gy - y0, s["y"] - y0) <= TOL_GRAD_BF16_FULL, rel_l2(gy - y0, s["y"] - y0)  # the path travelled: a sum of gradient steps
    assert median_abs_rows(gy, s["y"]) <= TOL_TRAJ_BF16 / BULK_DIVISOR
    for k in range(K):
        gx = ctx.read_params(k).astype(np.float64)
        assert rel_l2(gx, s["x"][k]) <= TOL_TRAJ_BF16
        assert rel_l2(gx - x0[k], s["x"][k] - x0[k]) <= TOL_GRAD_BF16_FULL, (k, rel_l2(gx - x0[k], s["x"][k] - x0[k]))
        assert median_abs_rows(gx, s["x"][k]) <= TOL_TRAJ_BF16 / BULK_DIVISOR
    ctx.close()
    o.close()


def test_c4_full_shape_one_tick_of_all_32_replicas_against_oracle_on_two():
    # the launch configuration bench.py times (K = 32): one whole tick on the device, replicas 0 and 31 recomputed by the
    # oracle's gradient routine from the same minibatches; Eq. 3 and the first update of Algorithm 1 evaluated with the
    # oracle's unrounded gradients
    import torch

    dev = torch.device("cuda", 0)
    w, inp = _inputs(bench.WORKLOADS["c4"], dev)
    K = w["K"]
    picks = [0, K - 1]
    x0_rows = {k: inp["x0"][k].cpu().numpy().astype(np.float64) for k in picks}
    y0_row = inp["y0"].cpu().numpy().astype(np.float64)
    ctx = G.Lsam(bench.make_cfg(G, w, flags=G.FLAG_KEEP_G1 | G.FLAG_STEP_INFO), inp["X"], inp["Y"], inp["x0"], inp["y0"])
    assert ctx.uses_tcgen05()
    inp["x0"] = None
    torch.cuda.empty_cache()
    ctx.step(w["eta"], w["rho"])
    assert ctx.status() == 0
    idx, _, _ = ctx.read_schedule(0)
    loss, n1, n2 = ctx.read_step_info()
    X, Y = inp["X"].cpu().numpy(), inp["Y"].cpu().numpy()
    ocfg = _oracle_cfg(w, 1)
    rho, gam = float(np.float32(w["rho"])), float(np.float32(bench.GAMMA))
    lam = float(np.float32(w.get("lambda0", bench.LAMBDA0) / (w["eta"] * w["tau"])))
    eta, mu = float(np.float32(w["eta"])), float(np.float32(bench.MU))

    def one(k):
        l1, g1 = O.loss_grad(ocfg, X, Y, x0_rows[k], idx[k])
        xp = x0_rows[k] + rho * g1 / (np.linalg.norm(g1) + gam)
        return dict(l1=l1, g1=g1, xp=xp, g2=O.loss_grad(ocfg, X, Y, xp, idx[k])[1])

    with ThreadPoolExecutor(len(picks)) as ex:
        res = list(ex.map(one, picks))
    for k, r in zip(picks, res):
        g1 = ctx.read_grads_replica(1, k)
        assert rel_l2(g1, r["g1"]) <= TOL_GRAD_BF16_FULL, ("g1", k, rel_l2(g1, r["g1"]), _layer_errors(w["widths"], g1, r["g1"]))
        assert abs(loss[k] - r["l1"]) <= 1e-4 * abs(r["l1"]), (k, loss[k], r["l1"])
        assert abs(n1[k] - np.linalg.norm(r["g1"])) <= 2e-3 * np.linalg.norm(r["g1"])
        xp_gpu = ctx.read_grads_replica(3, k)
        want = torch.from_numpy(r["xp"].astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
        assert rel_l2(xp_gpu, want) <= 1e-3
        g2 = ctx.read_grads_replica(2, k)
        assert rel_l2(g2, r["g2"]) <= TOL_GRAD_BF16_FULL, ("g2", k, rel_l2(g2, r["g2"]), _layer_errors(w["widths"], g2, r["g2"]))
        assert abs(n2[k] - np.linalg.norm(r["g2"])) <= 2e-3 * np.linalg.norm(r["g2"])
        # first tick: v = G and the centre read is y0 whatever the staleness, so x_1 = x0 - eta (1 + mu) G with
        # G = g2 + lambda (x0 - y0) from the ORACLE's descent gradient; the displacement is the sharp quantity
        Gs = r["g2"] + lam * (x0_rows[k] - y0_row)
        want_x = x0_rows[k] - eta * (Gs + mu * Gs)
        got_x = ctx.read_params(k).astype(np.float64)
        assert rel_l2(got_x - x0_rows[k], want_x - x0_rows[k]) <= TOL_GRAD_BF16_FULL, (k, rel_l2(got_x - x0_rows[k], want_x - x0_rows[k]))
        assert median_abs_rows(got_x, want_x) <= TOL_TRAJ_BF16 / BULK_DIVISOR
    ctx.close()


@pytest.mark.parametrize("key,K", [("c3", 16), ("c4", 4)])
def test_bench_launch_configuration_is_bitwise_identical_to_plain_launches_at_full_shapes(key, K):
    # bench.py replays each tick as a CUDA graph whose tensor-core GEMMs carry the programmatic-stream-serialization
    # attribute (their blocks become resident while the kernel before drains, and wait for it before touching memory).  At
    # the full layer shapes (several tiles per CTA, CTA pairs, weight-gradient runs) that must not change a bit against
    # plain in-order launches of the same kernels, which the tests above hold against the oracle.
    import torch

    dev = torch.device("cuda", 0)
    w, inp = _inputs(bench.WORKLOADS[key], dev, K=K)
    w["tau"] = 2  # a sync every second tick: the update's stale reads and the centre update are inside the compared run
    torch.cuda.synchronize()  # the inputs were generated on torch's default stream, which a side stream does not wait for
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        ctxs = [G.Lsam(bench.make_cfg(G, w, flags=fl), inp["X"], inp["Y"], inp["x0"], inp["y0"]) for fl in (0, G.FLAG_CUDA_GRAPH | G.FLAG_PDL)]
    assert all(c.uses_tcgen05() for c in ctxs)
    for t in range(5):
        for c in ctxs:
            c.step(w["eta"], w["rho"])
            if c.should_couple():
                assert c.couple() == 0
    a, b = ctxs
    assert a.status() == 0 and b.status() == 0 and a.launch_count() == b.launch_count()
    for k in (0, K - 1):
        np.testing.assert_array_equal(a.read_params(k), b.read_params(k))
    np.testing.assert_array_equal(a.read_params(-1), b.read_params(-1))
    for c in ctxs:
        c.close()
