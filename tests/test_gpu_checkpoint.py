"""Checkpoint and resume: a run saved in the middle of a sync period and loaded into a fresh context continues bit for bit."""
import numpy as np
import pytest

from paper_2509_03110_b200 import binding as G
from paper_2509_03110_b200 import synth

pytestmark = pytest.mark.gpu

HP = dict(tau=3, lam=0.3, seed=23, stale_max=2, mu=0.9, beta=0.9, eta_prime=1.0)


def _make(kind):
    import torch

    if kind == "flat":
        x0, y0, g1, g2 = synth.flat_problem(4, 1001, seed=6)
        dg = [torch.from_numpy(g1).cuda(), torch.from_numpy(g2).cuda()]

        def mk(x_init, flags=0):
            c = G.Lsam(G.make_config(G.MODEL_FLAT, K=4, flat_d=1001, noise_temp=0.05, flags=flags, **HP), None, None, torch.from_numpy(x_init).cuda(), torch.from_numpy(y0).cuda())
            c.set_external_grads(*dg)  # borrowed buffers are the caller's to supply again after a resume
            return c
        return mk, x0
    bf = kind == "resmlp_bf16_tcgen05"
    widths = (64, 128, 128, 16)
    X, labels = synth.gaussian_mixture(300, widths[0], widths[-1], seed=2)
    w0 = synth.mlp_init(widths, seed=2)
    x0 = synth.replicate(w0, 3, jitter=0.01)
    extra = dict(noise_temp=1e-3) if bf else dict(active_num=170)
    dX, dY = torch.from_numpy(X).cuda(), torch.from_numpy(labels).cuda()
    mk = lambda x_init, flags=0: G.Lsam(G.make_config(G.MODEL_RESMLP if bf else G.MODEL_MLP, widths=widths, K=3, batch=48, n_samples=300, flags=flags,
                                             gemm_dtype=G.GEMM_BF16 if bf else G.GEMM_FP32,
                                             gemm_impl=G.IMPL_TCGEN05 if kind == "mlp_fp32_tcgen05_async" else G.IMPL_AUTO, **extra, **HP),
                               dX, dY, torch.from_numpy(x_init).cuda(), torch.from_numpy(w0).cuda())
    return mk, x0


def _run(c, t0, t1):
    for t in range(t0, t1):
        c.step(0.02 + 0.001 * t, 0.0 if t == 5 else 0.03 + 0.002 * t)
        if c.should_couple():
            assert c.couple() == 0


@pytest.mark.parametrize("kind", ["flat", "mlp_fp32_async", "mlp_fp32_tcgen05_async", "resmlp_bf16_tcgen05"])  # the third: operand planes rebuilt from the loaded x
def test_resumed_run_continues_bit_for_bit(kind):
    mk, x0 = _make(kind)
    a = mk(x0)
    _run(a, 0, 8)                      # 8 ticks: past two syncs, in the middle of a period, stale reads pending
    blob = a.save_checkpoint()
    _run(a, 8, 15)
    b = mk(np.zeros_like(x0))          # a fresh context with another starting point: everything must come from the blob
    b.load_checkpoint(blob)
    assert b.counters()[0] == 8
    _run(b, 8, 15)
    np.testing.assert_array_equal(a.read_all_params(), b.read_all_params())
    np.testing.assert_array_equal(a.read_params(-1), b.read_params(-1))
    sa, sb = a.read_state(), b.read_state()
    for key in ("v", "acc", "gprev"):
        np.testing.assert_array_equal(sa[key], sb[key])
    ca, cb = a.counters(), b.counters()
    assert ca[0] == cb[0] and ca[1] == cb[1] and (ca[2] == cb[2]).all()
    for t in (13, 14):                 # centre versions read by the last ticks: the history survived the resume
        np.testing.assert_array_equal(a.read_schedule(t)[2], b.read_schedule(t)[2])
    assert a.status() == 0 and b.status() == 0
    # a blob of another shape is refused, and so is a truncated one
    with pytest.raises(G.LsamError):
        b.load_checkpoint(blob[: blob.size // 2])
    other_mk, other_x0 = _make("flat" if kind != "flat" else "mlp_fp32_async")
    o = other_mk(other_x0)
    with pytest.raises(G.LsamError):
        o.load_checkpoint(np.concatenate([blob, np.zeros(1 << 22, np.uint8)]))
    for c in (a, b, o):
        c.close()


@pytest.mark.parametrize("kind", ["flat", "mlp_fp32_tcgen05_async", "resmlp_bf16_tcgen05"])
def test_resume_into_a_graph_replaying_context(kind):
    # saved by a context that launches its kernels plainly, resumed by one that replays each tick as a CUDA graph with
    # programmatic dependent launch and has already recorded its graphs on another trajectory: tick, centre-version history
    # and budget of the resumed run must reach the recorded graphs, so the two runs end bit for bit equal
    import torch

    mk, x0 = _make(kind)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()  # the default stream cannot be captured
    with torch.cuda.stream(stream):
        a = mk(x0)
        b = mk(x0 * 0.5, G.FLAG_CUDA_GRAPH | G.FLAG_PDL)
    _run(a, 0, 8)
    _run(b, 0, 5)                      # graphs of every tick variant are recorded here
    blob = a.save_checkpoint()
    b.load_checkpoint(blob)
    _run(a, 8, 15)
    _run(b, 8, 15)
    np.testing.assert_array_equal(a.read_all_params(), b.read_all_params())
    np.testing.assert_array_equal(a.read_params(-1), b.read_params(-1))
    np.testing.assert_array_equal(a.read_state()["v"], b.read_state()["v"])
    ca, cb = a.counters(), b.counters()
    assert ca[0] == cb[0] and ca[1] == cb[1] and (ca[2] == cb[2]).all()
    assert a.status() == 0 and b.status() == 0
    a.close()
    b.close()


def test_load_drops_staged_minibatches_and_refuses_inconsistent_counters():
    # a minibatch staged before lsam_load_checkpoint belongs to the run being replaced: the resumed run must not consume it;
    # a blob whose counters describe no reachable state (negative or more than K tau iterations since the last sync, a
    # centre-version history beyond the current version) is refused and leaves the context as it was
    import torch

    widths, K, B = (32, 40, 6), 3, 16
    X, labels = synth.gaussian_mixture(200, 32, 6, seed=1)
    w0 = synth.mlp_init(widths, seed=1)
    x0 = synth.replicate(w0, K)
    dX, dY = torch.from_numpy(X).cuda(), torch.from_numpy(labels).cuda()
    mk = lambda: G.Lsam(G.make_config(G.MODEL_MLP, widths=widths, K=K, batch=B, n_samples=200, tau=2, lam=0.3, seed=9), dX, dY,
                        torch.from_numpy(x0).cuda(), torch.from_numpy(w0).cuda())
    a = mk()
    a.step(0.05, 0.05)
    blob = a.save_checkpoint()
    idx, _, _ = a.read_schedule(1, want_ver=False)
    xb = torch.from_numpy(X[idx.ravel()].reshape(K, B, 32)).pin_memory()
    yb = torch.from_numpy(labels[idx.ravel()].reshape(K, B)).pin_memory()
    a.stage_batch(xb, yb)
    a.load_checkpoint(blob)
    with pytest.raises(G.LsamError) as ei:
        a.step_staged(0.05, 0.05)  # nothing is staged any more
    assert ei.value.code == G.LSAM_ERR_STATE
    hdr = 8 + 8 * 7 + 4 * 16  # magic, seven int64 fields, sixteen int32 history entries
    tx = blob[hdr:hdr + 8 * K].view(np.int64)
    assert tx.tolist() == [1] * K
    for mutate in ("negative", "too_many", "history"):
        bad = blob.copy()
        if mutate == "negative":
            bad[hdr:hdr + 8].view(np.int64)[0] = -1
        elif mutate == "too_many":
            bad[hdr:hdr + 8].view(np.int64)[0] = 100
        else:
            bad[8 + 8 * 7:8 + 8 * 7 + 4].view(np.int32)[0] = 5  # step 0 started at centre version 5 of a run whose version is 0
        with pytest.raises(G.LsamError) as ei:
            a.load_checkpoint(bad)
        assert ei.value.code == G.LSAM_ERR_INVALID
        assert a.counters()[0] == 1 and a.counters()[2].tolist() == [1] * K  # untouched
    b = mk()
    b.load_checkpoint(blob)
    for c in (a, b):
        c.step(0.05, 0.05)
    np.testing.assert_array_equal(a.read_all_params(), b.read_all_params())
    a.close()
    b.close()
