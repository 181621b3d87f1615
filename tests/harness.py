"""Builds a CPU-oracle run and a CUDA-library run from the same seeded inputs and compares them."""
import numpy as np

import oracle as O
from paper_2509_03110_b200 import binding as G


def rel_l2(got, want):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    den = np.linalg.norm(want)
    return float(np.linalg.norm(got - want) / den) if den > 0 else float(np.linalg.norm(got - want))


def max_rel_rows(got, want):
    """Max over replicas of the relative L2 error of each row."""
    return max(rel_l2(g, w) for g, w in zip(np.atleast_2d(got), np.atleast_2d(want)))


class Pair:
    """Same configuration and inputs on both sides.  Hyper-parameters are carried as fp32 values on both."""

    def __init__(self, model, widths=(), K=1, batch=1, X=None, Y=None, x0=None, y0=None, flat_d=0, device="cuda", **hp):
        import torch

        self.torch = torch
        n_samples = 1 if X is None else X.shape[0]
        okw = {k: v for k, v in hp.items() if k not in ("gemm_impl", "flags")}
        self.ocfg = O.make_config(model, widths=widths, K=K, batch=batch, n_samples=n_samples, flat_d=flat_d, **okw)
        self.gcfg = G.make_config(model, widths=widths, K=K, batch=batch, n_samples=n_samples, flat_d=flat_d, **hp)
        self.K = K
        x0 = np.ascontiguousarray(x0, dtype=np.float32)
        y0 = np.ascontiguousarray(y0, dtype=np.float32)
        self.oracle = O.Oracle(self.ocfg, X, Y, x0.astype(np.float64), y0.astype(np.float64))
        dev = torch.device(device)
        self.dX = None if X is None else torch.from_numpy(np.ascontiguousarray(X, dtype=np.float32)).to(dev)
        if Y is None:
            self.dY = None
        else:
            ydt = np.float32 if model == G.MODEL_LSQ else np.int32
            self.dY = torch.from_numpy(np.ascontiguousarray(Y, dtype=ydt)).to(dev)
        self.gpu = G.Lsam(self.gcfg, self.dX, self.dY, torch.from_numpy(x0).to(dev), torch.from_numpy(y0).to(dev))
        self.d = self.gpu.d
        assert self.d == self.oracle.d

    def set_external_grads(self, g1, g2):
        t = self.torch
        self.oracle.set_external_grads(g1, g2)
        self.dg1 = t.from_numpy(np.ascontiguousarray(g1, dtype=np.float32)).cuda()
        self.dg2 = t.from_numpy(np.ascontiguousarray(g2, dtype=np.float32)).cuda()
        self.gpu.set_external_grads(self.dg1, self.dg2)

    def step(self, eta, rho):
        self.oracle.step(eta, rho)
        self.gpu.step(eta, rho)

    def couple_if_due(self):
        a, b = self.oracle.should_couple(), self.gpu.should_couple()
        assert a == b
        if a:
            assert self.oracle.couple() == 0
            assert self.gpu.couple() == 0
        return a

    def teacher_force(self):
        """Copy the oracle's iterates, momentum and current centre (rounded to fp32) into the CUDA run."""
        t = self.torch
        s = self.oracle.read_state()
        self.gpu.write_state(t.from_numpy(s["x"].astype(np.float32)).cuda(), t.from_numpy(s["v"].astype(np.float32)).cuda(),
                             t.from_numpy(s["y"].astype(np.float32)).cuda())

    def errors(self):
        s = self.oracle.read_state()
        gx = self.gpu.read_all_params()
        gs = self.gpu.read_state()
        return dict(
            x=max_rel_rows(gx, s["x"]),
            v=max_rel_rows(gs["v"], s["v"]),
            y=rel_l2(self.gpu.read_params(-1), s["y"]),
            acc=rel_l2(gs["acc"], s["acc"].sum(axis=0)) if np.any(s["acc"]) else float(np.abs(gs["acc"]).max()),
        )

    def grad_errors(self):
        g1, g2, xp = self.oracle.read_grads()
        if self.gcfg.gemm_dtype == G.GEMM_BF16:  # the perturbed point is stored as the bf16 matmul operand
            t = self.torch
            xp = t.from_numpy(xp.astype(np.float32)).to(t.bfloat16).to(t.float64).numpy()
        out = dict(g2=max_rel_rows(self.gpu.read_grads(2), g2), xp=max_rel_rows(self.gpu.read_grads(3), xp))
        if self.gcfg.flags & G.FLAG_KEEP_G1 or self.gcfg.model == G.MODEL_FLAT:
            out["g1"] = max_rel_rows(self.gpu.read_grads(1), g1)
        return out

    def close(self):
        self.gpu.close()
        self.oracle.close()
