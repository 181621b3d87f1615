"""Workers sharded over ranks (Algorithm 2 runs one worker per device): the oracle's sharded sync branch against the
single-context oracle, and the exchange helper of the package on two gloo ranks."""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

WIDTHS, K_TOTAL, B, TAU, STEPS = (12, 16, 5), 4, 6, 3, 7


def _inputs():
    from paper_2509_03110_b200 import synth

    X, labels = synth.gaussian_mixture(64, WIDTHS[0], WIDTHS[-1], seed=3)
    w0 = synth.mlp_init(WIDTHS, seed=4)
    rng = np.random.default_rng(5)
    x0 = np.stack([w0 + 0.01 * rng.standard_normal(w0.shape) for _ in range(K_TOTAL)])  # distinct workers
    return X, labels, x0, w0


def _oracle(O, X, labels, x0, y0, ids):
    cfg = O.make_config(O.MODEL_MLP, widths=WIDTHS, K=len(ids), batch=B, mu=0.9, lam=0.7, tau=TAU, beta=0.9, eta_prime=1.0,
                        stale_max=2, seed=11, n_samples=X.shape[0], noise_temp=1e-4)
    return O.Oracle(cfg, X, labels, x0[ids], y0, replica_ids=np.asarray(ids, dtype=np.int32))


def _run_single(O):
    X, labels, x0, y0 = _inputs()
    o = _oracle(O, X, labels, x0, y0, list(range(K_TOTAL)))
    for _ in range(STEPS):
        o.step(0.05, 0.05)
        if o.should_couple():
            assert o.couple() == 0
    st = o.read_state()
    return st["x"], st["y"], o.counters()


def test_sharded_sync_branch_equals_single_context(oracle_mod):
    """Two shards of two workers, accumulators exchanged by hand: same iterates and centre as one context of four."""
    O = oracle_mod
    X, labels, x0, y0 = _inputs()
    shards = [_oracle(O, X, labels, x0, y0, [0, 1]), _oracle(O, X, labels, x0, y0, [2, 3])]
    for _ in range(STEPS):
        for s in shards:
            s.step(0.05, 0.05)
        due = [s.should_couple() for s in shards]
        assert due[0] == due[1]
        if due[0]:
            sums = [s.read_state()["acc"].sum(0) for s in shards]
            total = sums[0] + sums[1]
            for s in shards:
                assert s.couple_sharded(K_TOTAL, total) == 0
    xs, ys, (t, t_y, _) = _run_single(O)
    assert t == STEPS and t_y == STEPS // TAU
    for r, s in enumerate(shards):
        st = s.read_state()
        np.testing.assert_allclose(st["x"], xs[2 * r:2 * r + 2], rtol=0, atol=1e-13)
        np.testing.assert_allclose(st["y"], ys, rtol=0, atol=1e-13)
    # the divisor really is n tau of the whole job: a shard coupled alone (divisor K tau, no exchange) lands elsewhere
    lone = _oracle(O, X, labels, x0, y0, [0, 1])
    for _ in range(TAU):
        lone.step(0.05, 0.05)
    assert lone.couple() == 0
    assert np.abs(lone.read_state()["y"] - ys).max() > 1e-6


class _OracleEngine:
    """Adapter with the interface exchange_and_couple() expects, backed by an oracle shard."""

    def __init__(self, oracle, n_total):
        self.o, self.n_total, self._t = oracle, n_total, None

    def acc_tensor(self):
        import torch

        self._t = torch.from_numpy(self.o.read_state()["acc"].sum(0))
        return self._t

    def couple(self):
        return self.o.couple_sharded(self.n_total, self._t.numpy())


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out):
    import torch.distributed as dist

    import oracle as O
    from paper_2509_03110_b200 import sharded

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    X, labels, x0, y0 = _inputs()
    k0, K = sharded.shard_range(K_TOTAL, rank, world)
    eng = _OracleEngine(_oracle(O, X, labels, x0, y0, list(range(k0, k0 + K))), K_TOTAL)
    syncs = 0
    for _ in range(STEPS):
        eng.o.step(0.05, 0.05)
        if eng.o.should_couple():
            assert sharded.exchange_and_couple(eng) == 0
            syncs += 1
    st = eng.o.read_state()
    out[rank] = (k0, K, syncs, st["x"], st["y"])
    dist.barrier()
    dist.destroy_process_group()


def test_exchange_helper_two_gloo_ranks(oracle_mod):
    port = _free_port()
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank, args=(2, port, out), nprocs=2, join=True)
        res = dict(out)
    xs, ys, _ = _run_single(oracle_mod)
    for rank in (0, 1):
        k0, K, syncs, x, y = res[rank]
        assert (k0, K, syncs) == (2 * rank, 2, STEPS // TAU)
        np.testing.assert_allclose(x, xs[k0:k0 + K], rtol=0, atol=1e-12)
        np.testing.assert_allclose(y, ys, rtol=0, atol=1e-12)
    np.testing.assert_array_equal(res[0][4], res[1][4])  # every rank holds the same centre, bit for bit


def test_shard_range():
    from paper_2509_03110_b200 import sharded

    assert [sharded.shard_range(32, r, 4) for r in range(4)] == [(0, 8), (8, 8), (16, 8), (24, 8)]
    try:
        sharded.shard_range(10, 0, 4)
    except ValueError:
        pass
    else:
        raise AssertionError("uneven shards must be refused")
