"""ctypes binding of the CPU oracle (TEST INFRASTRUCTURE ONLY).

The oracle is a plain double-precision restatement of the LSAM worker step and centre update
(Algorithm 2, Eq. 3, Algorithm 1).  Only the test-suite, the smoke check and the benchmark's
CPU-baseline leg may import this module; the CUDA product path never does.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lsam_oracle.cpp")
_HDR = os.path.join(_HERE, "lsam_oracle.h")
_LIB = os.path.join(_HERE, "liblsam_oracle.so")

MODEL_LSQ, MODEL_MLP, MODEL_RESMLP, MODEL_FLAT, MODEL_CNN = 0, 1, 2, 3, 4
GEMM_FP32, GEMM_BF16 = 0, 1
KERNEL_GAUSSIAN, KERNEL_EXP_POWER, KERNEL_CAUCHY, KERNEL_MATERN32 = 0, 1, 2, 3


def build(force=False):
    """Compile the oracle with g++ (OpenMP over replicas only)."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= newest:
        return _LIB
    cmd = ["g++", "-O2", "-std=c++17", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC]
    subprocess.run(cmd, check=True)
    return _LIB


class OracleConfig(C.Structure):
    _fields_ = [
        ("model", C.c_int32), ("n_layers", C.c_int32), ("widths", C.c_int32 * 9), ("K", C.c_int32),
        ("batch", C.c_int32), ("gemm_dtype", C.c_int32), ("nesterov", C.c_int32), ("tau", C.c_int32),
        ("stale_max", C.c_int32), ("active_num", C.c_int32), ("n_samples", C.c_int64), ("flat_d", C.c_int64),
        ("seed", C.c_uint64), ("mu", C.c_double), ("gamma", C.c_double), ("lam", C.c_double),
        ("beta", C.c_double), ("eta_prime", C.c_double), ("noise_temp", C.c_double),
        ("kernel_kind", C.c_int32), ("dp_average", C.c_int32), ("kernel_param", C.c_double),
        ("n_conv", C.c_int32), ("img_h", C.c_int32), ("img_w", C.c_int32),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        vp, i64p, i32p, dp, fp = C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int32), C.POINTER(C.c_double), C.POINTER(C.c_float)
        cfgp = C.POINTER(OracleConfig)
        L.oracle_param_count.restype = C.c_int64
        L.oracle_param_count.argtypes = [cfgp]
        L.oracle_create.restype = vp
        L.oracle_create.argtypes = [cfgp, vp, vp, vp, vp, vp]
        L.oracle_destroy.argtypes = [vp]
        L.oracle_destroy.restype = None
        L.oracle_step.argtypes = [vp, C.c_double, C.c_double]
        L.oracle_should_couple.argtypes = [vp]
        L.oracle_couple.argtypes = [vp]
        L.oracle_couple_sharded.argtypes = [vp, C.c_int32, vp]
        L.oracle_read_params.argtypes = [vp, C.c_int, vp]
        L.oracle_read_state.argtypes = [vp, vp, vp, vp, vp, vp]
        L.oracle_write_state.argtypes = [vp, vp, vp, vp]
        L.oracle_read_schedule.argtypes = [vp, C.c_int64, vp, vp, vp]
        L.oracle_read_step_info.argtypes = [vp, vp, vp, vp]
        L.oracle_read_grads.argtypes = [vp, vp, vp, vp]
        L.oracle_set_external_grads.argtypes = [vp, vp, vp]
        L.oracle_read_counters.argtypes = [vp, vp, vp, vp]
        L.oracle_read_active.argtypes = [vp, vp]
        L.oracle_tag_active.restype = C.c_uint64
        L.oracle_tag_order.restype = C.c_uint64
        L.oracle_loss_grad.argtypes = [cfgp, vp, vp, vp, vp, C.c_int32, vp, vp]
        L.oracle_forward.argtypes = [cfgp, vp, vp, vp, C.c_int32, vp]
        L.oracle_philox4x32_10.restype = None
        L.oracle_philox4x32_10.argtypes = [vp, vp, vp]
        L.oracle_noise4.restype = None
        L.oracle_noise4.argtypes = [C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64, vp]
        L.oracle_kernel_phi.restype = C.c_double
        L.oracle_kernel_phi.argtypes = [C.c_int32, C.c_double, C.c_double, C.c_double]
        L.oracle_kernel_weight.restype = C.c_double
        L.oracle_kernel_weight.argtypes = [C.c_int32, C.c_double, C.c_double, C.c_double]
        L.oracle_read_pull_weights.argtypes = [vp, vp]
        L.oracle_mix64.restype = C.c_uint64
        L.oracle_mix64.argtypes = [C.c_uint64]
        L.oracle_hash.restype = C.c_uint64
        L.oracle_hash.argtypes = [C.c_uint64] * 5
        L.oracle_tag_idx.restype = C.c_uint64
        L.oracle_tag_stale.restype = C.c_uint64
        L.oracle_bf16_round.restype = C.c_float
        L.oracle_bf16_round.argtypes = [C.c_float]
        L.oracle_num_threads.restype = C.c_int
        _lib = L
    return _lib


def make_config(model, widths=(), K=1, batch=1, gemm_dtype=GEMM_FP32, mu=0.9, nesterov=1, gamma=1e-12,
                lam=0.0, tau=4, beta=0.9, eta_prime=1.0, stale_max=0, seed=0, n_samples=1, flat_d=0, active_num=256, noise_temp=0.0,
                kernel_kind=KERNEL_GAUSSIAN, kernel_param=0.0, dp_average=0, n_conv=0, img_h=0, img_w=0):
    """Float hyper-parameters are taken at their fp32 value, the precision the C-ABI carries them in."""
    c = OracleConfig()
    c.model = model
    widths = list(widths)
    c.n_layers = max(len(widths) - 1, 0) if model in (MODEL_MLP, MODEL_RESMLP, MODEL_CNN) else (1 if model == MODEL_LSQ else 0)
    for i, w in enumerate(widths):
        c.widths[i] = int(w)
    c.K, c.batch, c.gemm_dtype, c.nesterov, c.tau = int(K), int(batch), int(gemm_dtype), int(nesterov), int(tau)
    c.stale_max, c.n_samples, c.flat_d, c.seed = int(stale_max), int(n_samples), int(flat_d), int(seed)
    c.active_num = int(active_num)
    f32 = lambda v: float(np.float32(v))
    c.mu, c.gamma, c.lam, c.beta, c.eta_prime = f32(mu), f32(gamma), f32(lam), f32(beta), f32(eta_prime)
    c.noise_temp = f32(noise_temp)
    c.kernel_kind, c.kernel_param, c.dp_average = int(kernel_kind), f32(kernel_param), int(dp_average)
    c.n_conv, c.img_h, c.img_w = int(n_conv), int(img_h), int(img_w)
    return c


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def param_count(cfg):
    return int(lib().oracle_param_count(C.byref(cfg)))


def loss_grad(cfg, X, Y, params, idx):
    """Mean minibatch loss and gradient at `params` (double [d]) for the rows `idx` of X."""
    d = param_count(cfg)
    params = np.ascontiguousarray(params, dtype=np.float64)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    assert params.shape == (d,)
    loss = np.zeros(1, dtype=np.float64)
    grad = np.zeros(d, dtype=np.float64)
    rc = lib().oracle_loss_grad(C.byref(cfg), _ptr(X), _ptr(Y), _ptr(params), _ptr(idx), len(idx), _ptr(loss), _ptr(grad))
    assert rc == 0
    return float(loss[0]), grad


def forward(cfg, X, params, idx):
    params = np.ascontiguousarray(params, dtype=np.float64)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    n_out = 1 if cfg.model == MODEL_LSQ else cfg.widths[cfg.n_layers]
    out = np.zeros((len(idx), n_out), dtype=np.float64)
    rc = lib().oracle_forward(C.byref(cfg), _ptr(X), _ptr(params), _ptr(idx), len(idx), _ptr(out))
    assert rc == 0
    return out


def philox(counter, key):
    c = np.asarray(counter, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return [int(v) for v in out]


def noise4(seed, t, k, seg, group):
    out = np.zeros(4, dtype=np.float64)
    lib().oracle_noise4(seed, t, k, seg, group, _ptr(out))
    return out


def kernel_phi(kind, lam, param, r):
    return float(lib().oracle_kernel_phi(int(kind), float(lam), float(param), float(r)))


def kernel_weight(kind, lam, param, r):
    return float(lib().oracle_kernel_weight(int(kind), float(lam), float(param), float(r)))


def mix64(z):
    return int(lib().oracle_mix64(C.c_uint64(z)))


def hash5(seed, tag, t, k, j):
    return int(lib().oracle_hash(seed, tag, t, k, j))


def bf16_round(v):
    return float(lib().oracle_bf16_round(C.c_float(v)))


def num_threads():
    return int(lib().oracle_num_threads())


class Oracle:
    """One LSAM run on the CPU: K replicas, a centre history, the seeded schedule."""

    def __init__(self, cfg, X, Y, x0, y0, replica_ids=None):
        self.cfg = cfg
        self.K = cfg.K
        self.d = param_count(cfg)
        assert self.d > 0, "invalid oracle configuration"
        self._X = None if X is None else np.ascontiguousarray(X, dtype=np.float32)
        if Y is None:
            self._Y = None
        elif cfg.model == MODEL_LSQ:
            self._Y = np.ascontiguousarray(Y, dtype=np.float32)
        else:
            self._Y = np.ascontiguousarray(Y, dtype=np.int32)
        x0 = np.ascontiguousarray(x0, dtype=np.float64).reshape(self.K, self.d)
        y0 = np.ascontiguousarray(y0, dtype=np.float64).reshape(self.d)
        rid = None if replica_ids is None else np.ascontiguousarray(replica_ids, dtype=np.int32)
        self._h = lib().oracle_create(C.byref(cfg), _ptr(self._X), _ptr(self._Y), _ptr(x0), _ptr(y0), _ptr(rid))
        assert self._h, "oracle_create failed"
        self._keep = []

    def close(self):
        if self._h:
            lib().oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def step(self, eta, rho):
        rc = lib().oracle_step(self._h, float(np.float32(eta)), float(np.float32(rho)))
        assert rc == 0, f"oracle_step rc={rc}"

    def should_couple(self):
        return bool(lib().oracle_should_couple(self._h))

    def couple(self):
        return int(lib().oracle_couple(self._h))

    def couple_sharded(self, n_total, total_acc=None):
        """Sync branch for a shard: total_acc [d] is the summed accumulator of ALL workers of the job (this shard's included)."""
        oa = None if total_acc is None else np.ascontiguousarray(total_acc, dtype=np.float64)
        return int(lib().oracle_couple_sharded(self._h, int(n_total), _ptr(oa)))

    def read_params(self, which):
        out = np.zeros(self.d, dtype=np.float64)
        assert lib().oracle_read_params(self._h, int(which), _ptr(out)) == 0
        return out

    def read_state(self):
        K, d = self.K, self.d
        x, v, acc = (np.zeros((K, d)) for _ in range(3))
        y, gprev = np.zeros(d), np.zeros(d)
        assert lib().oracle_read_state(self._h, _ptr(x), _ptr(v), _ptr(y), _ptr(acc), _ptr(gprev)) == 0
        return dict(x=x, v=v, y=y, acc=acc, gprev=gprev)

    def write_state(self, x=None, v=None, y=None):
        cv = lambda a, shape: None if a is None else np.ascontiguousarray(a, dtype=np.float64).reshape(shape)
        x, v, y = cv(x, (self.K, self.d)), cv(v, (self.K, self.d)), cv(y, (self.d,))
        assert lib().oracle_write_state(self._h, _ptr(x), _ptr(v), _ptr(y)) == 0

    def read_schedule(self, t):
        K, B = self.K, max(self.cfg.batch, 1)
        idx = np.zeros((K, B), dtype=np.int32)
        stale = np.zeros(K, dtype=np.int32)
        ver = np.zeros(K, dtype=np.int32)
        assert lib().oracle_read_schedule(self._h, int(t), _ptr(idx), _ptr(stale), _ptr(ver)) == 0
        return idx, stale, ver

    def read_step_info(self):
        loss, n1, n2 = (np.zeros(self.K) for _ in range(3))
        assert lib().oracle_read_step_info(self._h, _ptr(loss), _ptr(n1), _ptr(n2)) == 0
        return loss, n1, n2

    def read_grads(self):
        g1, g2, xp = (np.zeros((self.K, self.d)) for _ in range(3))
        assert lib().oracle_read_grads(self._h, _ptr(g1), _ptr(g2), _ptr(xp)) == 0
        return g1, g2, xp

    def set_external_grads(self, g1, g2):
        g1 = np.ascontiguousarray(g1, dtype=np.float32).reshape(self.K, self.d)
        g2 = np.ascontiguousarray(g2, dtype=np.float32).reshape(self.K, self.d)
        self._keep = [g1, g2]
        assert lib().oracle_set_external_grads(self._h, _ptr(g1), _ptr(g2)) == 0

    def read_pull_weights(self):
        w = np.zeros(self.K)
        assert lib().oracle_read_pull_weights(self._h, _ptr(w)) == 0
        return w

    def read_active(self):
        a = np.zeros(self.K, dtype=np.int32)
        assert lib().oracle_read_active(self._h, _ptr(a)) == 0
        return a

    def counters(self):
        t = np.zeros(1, dtype=np.int64)
        ty = np.zeros(1, dtype=np.int64)
        tx = np.zeros(self.K, dtype=np.int64)
        assert lib().oracle_read_counters(self._h, _ptr(t), _ptr(ty), _ptr(tx)) == 0
        return int(t[0]), int(ty[0]), tx
