"""Workers sharded over contexts (K_total > K): two contexts on one GPU stand in for two ranks, the accumulator exchange
is done by hand, and the result is compared with the CPU oracle and with one context that holds all workers."""
import os

import numpy as np
import pytest

from harness import max_rel_rows, rel_l2

pytestmark = pytest.mark.gpu

WIDTHS, K_TOTAL, B, TAU, STEPS = (48, 64, 10), 4, 16, 3, 7


def _inputs():
    from paper_2509_03110_b200 import synth

    X, labels = synth.gaussian_mixture(256, WIDTHS[0], WIDTHS[-1], seed=3)
    w0 = synth.mlp_init(WIDTHS, seed=4)
    rng = np.random.default_rng(5)
    x0 = np.stack([w0 + 0.01 * rng.standard_normal(w0.shape) for _ in range(K_TOTAL)]).astype(np.float32)
    return X, labels, x0, w0.astype(np.float32)


HP = dict(mu=0.9, lam=0.7, tau=TAU, beta=0.9, eta_prime=1.0, stale_max=2, seed=11, noise_temp=1e-4)


def _ctx(G, torch, X, labels, x0, y0, k0, K, K_total):
    cfg = G.make_config(G.MODEL_MLP, widths=WIDTHS, K=K, batch=B, n_samples=X.shape[0], K_total=K_total, k_offset=k0, **HP)
    dev = torch.device("cuda")
    return G.Lsam(cfg, torch.from_numpy(X).to(dev), torch.from_numpy(labels.astype(np.int32)).to(dev),
                  torch.from_numpy(x0[k0:k0 + K]).to(dev), torch.from_numpy(y0).to(dev))


def test_two_shards_match_oracle_and_single_context():
    import torch

    import oracle as O
    from paper_2509_03110_b200 import binding as G

    X, labels, x0, y0 = _inputs()
    ocfg = O.make_config(O.MODEL_MLP, widths=WIDTHS, K=K_TOTAL, batch=B, n_samples=X.shape[0], **HP)
    orc = O.Oracle(ocfg, X, labels, x0.astype(np.float64), y0.astype(np.float64))
    single = _ctx(G, torch, X, labels, x0, y0, 0, K_TOTAL, 0)
    shards = [_ctx(G, torch, X, labels, x0, y0, 0, 2, K_TOTAL), _ctx(G, torch, X, labels, x0, y0, 2, 2, K_TOTAL)]
    for t in range(STEPS):
        # the schedule is keyed by the global worker index: bit-exact against the oracle and the single context
        oi, os_, _ = orc.read_schedule(t)
        for r, s in enumerate(shards):
            gi, gs, _ = s.read_schedule(t, want_ver=False)
            np.testing.assert_array_equal(gi, oi[2 * r:2 * r + 2])
            np.testing.assert_array_equal(gs, os_[2 * r:2 * r + 2])
        orc.step(0.05, 0.05)
        single.step(0.05, 0.05)
        for s in shards:
            s.step(0.05, 0.05)
        due = orc.should_couple()
        assert single.should_couple() == due and all(s.should_couple() == due for s in shards)
        if due:
            assert orc.couple() == 0 and single.couple() == 0
            accs = [s.acc_tensor() for s in shards]
            total = accs[0] + accs[1]          # what an all-reduce over the two ranks leaves in both buffers
            for a, s in zip(accs, shards):
                a.copy_(total)
                assert s.couple() == 0
    assert all(s.status() == 0 for s in shards) and single.status() == 0
    ox, oy = orc.read_state()["x"], orc.read_state()["y"]
    sx, sy = single.read_all_params(), single.read_params(-1)
    for r, s in enumerate(shards):
        gx, gy = s.read_all_params(), s.read_params(-1)
        assert max_rel_rows(gx, ox[2 * r:2 * r + 2]) <= 1e-3 and rel_l2(gy, oy) <= 1e-3    # 7-step trajectory, fp32
        assert max_rel_rows(gx, sx[2 * r:2 * r + 2]) <= 1e-5 and rel_l2(gy, sy) <= 1e-5    # differs only in the order of the sum
        assert s.counters()[1] == STEPS // TAU
    np.testing.assert_array_equal(shards[0].read_params(-1), shards[1].read_params(-1))     # identical centres, no broadcast
    for c in shards + [single]:
        c.close()


def test_shard_configuration_is_checked():
    from paper_2509_03110_b200 import binding as G

    ok = G.make_config(G.MODEL_MLP, widths=WIDTHS, K=2, batch=B, n_samples=64, K_total=4, k_offset=2)
    assert G.lsam_workspace_bytes(ok) > 0
    for bad in (dict(K_total=4, k_offset=3), dict(K_total=1, k_offset=0), dict(K_total=0, k_offset=1), dict(K_total=4, k_offset=0, active_num=128)):
        assert G.lsam_workspace_bytes(G.make_config(G.MODEL_MLP, widths=WIDTHS, K=2, batch=B, n_samples=64, **bad)) == 0


def test_exchange_helper_on_a_one_rank_nccl_group():
    """The helper the multi-GPU bench uses, on a process group of one rank: the all-reduce runs on the context's stream."""
    import socket

    import torch
    import torch.distributed as dist

    from paper_2509_03110_b200 import binding as G
    from paper_2509_03110_b200 import sharded

    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        X, labels, x0, y0 = _inputs()
        a = _ctx(G, torch, X, labels, x0, y0, 0, K_TOTAL, K_TOTAL)
        b = _ctx(G, torch, X, labels, x0, y0, 0, K_TOTAL, 0)
        for _ in range(TAU):
            a.step(0.05, 0.05)
            b.step(0.05, 0.05)
        assert a.should_couple() and sharded.exchange_and_couple(a) == 0 and b.couple() == 0
        np.testing.assert_array_equal(a.read_params(-1), b.read_params(-1))
        a.close()
        b.close()
    finally:
        dist.destroy_process_group()
