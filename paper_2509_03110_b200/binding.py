"""Thin ctypes binding of the C ABI in include/lsam.h (argument marshalling only).

PyTorch supplies device memory and the CUDA stream; every step of the method runs in the library's kernels.
There is no CPU fallback: loading fails loudly when the shared library cannot be found or built.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liblsam_b200.so")

LSAM_OK, LSAM_ERR_INVALID, LSAM_ERR_WORKSPACE, LSAM_ERR_STATE, LSAM_ERR_CUDA, LSAM_ERR_NONFINITE, LSAM_ERR_TIMEOUT = range(7)
MODEL_LSQ, MODEL_MLP, MODEL_RESMLP, MODEL_FLAT, MODEL_CNN = 0, 1, 2, 3, 4
GEMM_FP32, GEMM_BF16 = 0, 1
IMPL_AUTO, IMPL_SIMT, IMPL_TCGEN05, IMPL_TCGEN05_1CTA, IMPL_TCGEN05_PAIRS = 0, 1, 2, 3, 4
KERNEL_GAUSSIAN, KERNEL_EXP_POWER, KERNEL_CAUCHY, KERNEL_MATERN32 = 0, 1, 2, 3
FLAG_KEEP_G1, FLAG_STEP_INFO, FLAG_CUDA_GRAPH, FLAG_GRAD_FP32, FLAG_FUSED_UPDATE, FLAG_PDL = 1, 2, 4, 8, 16, 32
PROF_CLASSES = ["schedule", "gather", "gemm_fwd", "gemm_dgrad", "gemm_wgrad", "loss", "bias_grad", "lsq_grad", "norm",
                "perturb", "update", "couple", "copy"]

EXPORTS = [
    "lsam_param_count", "lsam_workspace_bytes", "lsam_init", "lsam_step", "lsam_step_batch", "lsam_stage_batch", "lsam_step_staged", "lsam_couple",
    "lsam_should_couple", "lsam_read_params", "lsam_read_schedule", "lsam_read_step_info", "lsam_read_grads", "lsam_read_grads_replica",
    "lsam_set_external_grads", "lsam_write_state", "lsam_read_state", "lsam_read_counters", "lsam_read_active", "lsam_status",
    "lsam_profile_enable", "lsam_profile_read", "lsam_launch_count", "lsam_uses_tcgen05", "lsam_last_error",
    "lsam_destroy", "lsam_schedule_hash", "lsam_row_norms_static", "lsam_acc_buffer", "lsam_selftest_bounded_wait",
    "lsam_checkpoint_bytes", "lsam_save_checkpoint", "lsam_load_checkpoint", "lsam_read_anchor_gap",
]


class LsamConfig(C.Structure):
    _fields_ = [
        ("model", C.c_int32), ("n_layers", C.c_int32), ("widths", C.c_int32 * 9), ("K", C.c_int32), ("batch", C.c_int32),
        ("gemm_dtype", C.c_int32), ("gemm_impl", C.c_int32), ("nesterov", C.c_int32), ("tau", C.c_int32),
        ("stale_max", C.c_int32), ("flags", C.c_int32), ("n_samples", C.c_int64), ("flat_d", C.c_int64),
        ("seed", C.c_uint64), ("mu", C.c_float), ("gamma", C.c_float), ("lam", C.c_float), ("beta", C.c_float),
        ("eta_prime", C.c_float), ("active_num", C.c_int32), ("noise_temp", C.c_float),
        ("K_total", C.c_int32), ("k_offset", C.c_int32), ("kernel_kind", C.c_int32), ("kernel_param", C.c_float), ("dp_average", C.c_int32),
        ("n_conv", C.c_int32), ("img_h", C.c_int32), ("img_w", C.c_int32),
    ]


class LsamError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"lsam error {code}: {msg}")
        self.code = code


_lib = None


def lib():
    """Load liblsam_b200.so (building it with nvcc if it is absent); raises if neither works."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        from . import build as _build

        try:
            _build.build()
        except Exception as e:  # no silent fallback: the CUDA library is the product
            raise RuntimeError(f"liblsam_b200.so is missing and could not be built: {e}") from e
    L = C.CDLL(_LIB_PATH)
    vp, cfgp = C.c_void_p, C.POINTER(LsamConfig)
    L.lsam_param_count.restype = C.c_int64
    L.lsam_param_count.argtypes = [cfgp]
    L.lsam_workspace_bytes.restype = C.c_size_t
    L.lsam_workspace_bytes.argtypes = [cfgp]
    L.lsam_init.argtypes = [C.POINTER(vp), cfgp, vp, vp, vp, vp, vp, C.c_size_t, vp]
    L.lsam_step.argtypes = [vp, C.c_float, C.c_float]
    L.lsam_step_batch.argtypes = [vp, C.c_float, C.c_float, vp, vp, C.c_int, vp]
    L.lsam_stage_batch.argtypes = [vp, vp, vp, C.c_int]
    L.lsam_step_staged.argtypes = [vp, C.c_float, C.c_float, vp]
    L.lsam_couple.argtypes = [vp]
    L.lsam_acc_buffer.argtypes = [vp, C.POINTER(vp), C.POINTER(C.c_int64)]
    L.lsam_should_couple.argtypes = [vp]
    L.lsam_read_params.argtypes = [vp, C.c_int, vp, C.c_int64, C.c_int]
    L.lsam_read_schedule.argtypes = [vp, C.c_int64, vp, vp, vp]
    L.lsam_read_step_info.argtypes = [vp, vp, vp, vp]
    L.lsam_read_grads.argtypes = [vp, C.c_int, vp]
    L.lsam_read_grads_replica.argtypes = [vp, C.c_int, C.c_int, vp]
    L.lsam_set_external_grads.argtypes = [vp, vp, vp]
    L.lsam_write_state.argtypes = [vp, vp, vp, vp]
    L.lsam_read_state.argtypes = [vp, vp, vp, vp]
    L.lsam_read_counters.argtypes = [vp, vp, vp, vp]
    L.lsam_read_active.argtypes = [vp, vp]
    L.lsam_status.argtypes = [vp]
    L.lsam_read_anchor_gap.argtypes = [vp, vp]
    L.lsam_checkpoint_bytes.restype = C.c_size_t
    L.lsam_checkpoint_bytes.argtypes = [vp]
    L.lsam_save_checkpoint.argtypes = [vp, vp, C.c_size_t]
    L.lsam_load_checkpoint.argtypes = [vp, vp, C.c_size_t]
    L.lsam_selftest_bounded_wait.argtypes = [vp, C.c_uint32]
    L.lsam_profile_enable.argtypes = [vp, C.c_int]
    L.lsam_profile_read.argtypes = [vp, vp, vp]
    L.lsam_launch_count.restype = C.c_int64
    L.lsam_launch_count.argtypes = [vp]
    L.lsam_uses_tcgen05.argtypes = [vp]
    L.lsam_last_error.restype = C.c_char_p
    L.lsam_last_error.argtypes = [vp]
    L.lsam_destroy.restype = None
    L.lsam_destroy.argtypes = [vp]
    L.lsam_schedule_hash.restype = C.c_uint64
    L.lsam_schedule_hash.argtypes = [C.c_uint64, C.c_int, C.c_uint64, C.c_uint64, C.c_uint64]
    L.lsam_row_norms_static.argtypes = [vp, C.c_int64, C.c_int64, C.c_int32, vp, vp, C.c_char_p, C.c_size_t]
    _lib = L
    return L


def make_config(model, widths=(), K=1, batch=1, gemm_dtype=GEMM_FP32, gemm_impl=IMPL_AUTO, mu=0.9, nesterov=1,
                gamma=1e-12, lam=0.0, tau=4, beta=0.9, eta_prime=1.0, stale_max=0, seed=0, n_samples=1, flat_d=0, flags=0,
                active_num=256, noise_temp=0.0, K_total=0, k_offset=0, kernel_kind=KERNEL_GAUSSIAN, kernel_param=0.0, dp_average=0, n_conv=0, img_h=0, img_w=0):
    c = LsamConfig()
    c.model = model
    widths = list(widths)
    c.n_layers = max(len(widths) - 1, 0) if model in (MODEL_MLP, MODEL_RESMLP, MODEL_CNN) else (1 if model == MODEL_LSQ else 0)
    for i, w in enumerate(widths):
        c.widths[i] = int(w)
    c.K, c.batch, c.gemm_dtype, c.gemm_impl, c.nesterov, c.tau = int(K), int(batch), int(gemm_dtype), int(gemm_impl), int(nesterov), int(tau)
    c.stale_max, c.flags, c.n_samples, c.flat_d, c.seed = int(stale_max), int(flags), int(n_samples), int(flat_d), int(seed)
    c.mu, c.gamma, c.lam, c.beta, c.eta_prime = mu, gamma, lam, beta, eta_prime
    c.active_num = int(active_num)
    c.noise_temp = noise_temp
    c.K_total, c.k_offset = int(K_total), int(k_offset)
    c.kernel_kind, c.kernel_param, c.dp_average = int(kernel_kind), kernel_param, int(dp_average)
    c.n_conv, c.img_h, c.img_w = int(n_conv), int(img_h), int(img_w)
    return c


def lsam_param_count(cfg):
    return int(lib().lsam_param_count(C.byref(cfg)))


def lsam_workspace_bytes(cfg):
    return int(lib().lsam_workspace_bytes(C.byref(cfg)))


def lsam_schedule_hash(seed, tag, t, k, j):
    return int(lib().lsam_schedule_hash(seed, tag, t, k, j))


STATIC_NORM_MAX_PARTIALS = 262144


def lsam_row_norms_static(g, n, out, stream=None):
    """Row norms of the CUDA tensor g [K, ld] (first n columns) into the CUDA tensor out [K], with no allocation.

    For callers that may not allocate device memory (see include/lsam.h): the partial sums live in an array inside
    the library.  Returns (status, message).  Calls that overlap on one GPU race on that array; the first call on a
    device should be made outside stream capture.
    """
    K, ld = g.shape
    err = C.create_string_buffer(256)
    s = C.c_void_p(stream.cuda_stream) if stream is not None else None
    rc = lib().lsam_row_norms_static(C.c_void_p(g.data_ptr()), ld, int(n), K, C.c_void_p(out.data_ptr()), s, err, 256)
    return int(rc), err.value.decode()


def _np_ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dev_ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


class Lsam:
    """One LSAM context on the current CUDA device.  Tensors passed in are torch CUDA tensors (fp32 / int32)."""

    def __init__(self, cfg, X=None, Y=None, x0=None, y0=None, stream=None):
        import torch

        self._torch = torch
        self.cfg = cfg
        self.K = cfg.K
        self.d = lsam_param_count(cfg)
        if self.d <= 0:
            raise LsamError(LSAM_ERR_INVALID, "invalid configuration")
        nbytes = lsam_workspace_bytes(cfg)
        dev = x0.device
        assert dev.type == "cuda", "x0 must be a CUDA tensor: there is no CPU path"
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=dev)
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 255) // 256 * 256
        self.stream = stream if stream is not None else torch.cuda.current_stream(dev)
        self._keep = [X, Y]
        x0 = x0.contiguous().float()
        y0 = y0.contiguous().float()
        assert x0.numel() == self.K * self.d and y0.numel() == self.d
        h = C.c_void_p()
        rc = lib().lsam_init(C.byref(h), C.byref(cfg), _dev_ptr(X), _dev_ptr(Y), _dev_ptr(x0), _dev_ptr(y0),
                             C.c_void_p(self._ws_ptr), nbytes, C.c_void_p(self.stream.cuda_stream))
        if rc != LSAM_OK:
            raise LsamError(rc, "lsam_init failed")
        self._h = h
        self.stream.synchronize()  # x0 / y0 may be temporaries

    # -- lifetime
    def close(self):
        if getattr(self, "_h", None):
            self.stream.synchronize()
            lib().lsam_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc):
        if rc != LSAM_OK:
            raise LsamError(rc, lib().lsam_last_error(self._h).decode())

    # -- the four calls of the method
    def step(self, eta, rho):
        self._check(lib().lsam_step(self._h, eta, rho))

    def step_batch(self, eta, rho, xb, yb, h_loss=None):
        """xb / yb: pinned host tensors or numpy arrays (on_host) or CUDA tensors; h_loss: numpy float32 [K] or None."""
        torch = self._torch
        on_host = not (isinstance(xb, torch.Tensor) and xb.is_cuda)
        px = C.c_void_p(xb.data_ptr()) if isinstance(xb, torch.Tensor) else _np_ptr(xb)
        py = C.c_void_p(yb.data_ptr()) if isinstance(yb, torch.Tensor) else _np_ptr(yb)
        self._check(lib().lsam_step_batch(self._h, eta, rho, px, py, 1 if on_host else 0, _np_ptr(h_loss)))

    def stage_batch(self, xb, yb):
        """Prefetch a minibatch (pinned host tensors / numpy arrays, or CUDA tensors) into the next staging slot."""
        torch = self._torch
        on_host = not (isinstance(xb, torch.Tensor) and xb.is_cuda)
        px = C.c_void_p(xb.data_ptr()) if isinstance(xb, torch.Tensor) else _np_ptr(xb)
        py = C.c_void_p(yb.data_ptr()) if isinstance(yb, torch.Tensor) else _np_ptr(yb)
        self._check(lib().lsam_stage_batch(self._h, px, py, 1 if on_host else 0))

    def step_staged(self, eta, rho, h_loss=None):
        self._check(lib().lsam_step_staged(self._h, eta, rho, _np_ptr(h_loss)))

    def should_couple(self):
        return bool(lib().lsam_should_couple(self._h))

    def couple(self):
        return int(lib().lsam_couple(self._h))

    def acc_tensor(self):
        """The iterate accumulator as a CUDA fp32 tensor that aliases the workspace (sharded runs all-reduce it in place)."""
        p, n = C.c_void_p(), C.c_int64()
        self._check(lib().lsam_acc_buffer(self._h, C.byref(p), C.byref(n)))
        off = int(p.value) - self.workspace.data_ptr()
        return self.workspace[off:off + 4 * int(n.value)].view(self._torch.float32)

    def read_params(self, which, out=None):
        """Returns a numpy fp32 [d] (host copy) or fills the CUDA tensor `out`."""
        if out is not None:
            self._check(lib().lsam_read_params(self._h, int(which), _dev_ptr(out), out.numel(), 1))
            return out
        dst = np.empty(self.d, dtype=np.float32)
        self._check(lib().lsam_read_params(self._h, int(which), _np_ptr(dst), self.d, 0))
        return dst

    # -- helpers
    def read_all_params(self):
        return np.stack([self.read_params(k) for k in range(self.K)])

    def read_schedule(self, t, want_ver=True):
        K, B = self.K, max(self.cfg.batch, 1)
        idx = np.zeros((K, B), dtype=np.int32)
        stale = np.zeros(K, dtype=np.int32)
        ver = np.zeros(K, dtype=np.int32)
        self._check(lib().lsam_read_schedule(self._h, int(t), _np_ptr(idx), _np_ptr(stale), _np_ptr(ver) if want_ver else None))
        return idx, stale, ver

    def read_step_info(self):
        loss, n1, n2 = (np.zeros(self.K, dtype=np.float32) for _ in range(3))
        self._check(lib().lsam_read_step_info(self._h, _np_ptr(loss), _np_ptr(n1), _np_ptr(n2)))
        return loss, n1, n2

    def read_anchor_gap(self):
        """||x_k - y|| for every worker against the current centre (numpy fp32 [K])."""
        out = np.zeros(self.K, dtype=np.float32)
        self._check(lib().lsam_read_anchor_gap(self._h, _np_ptr(out)))
        return out

    def read_grads(self, which_pass):
        out = np.empty((self.K, self.d), dtype=np.float32)
        self._check(lib().lsam_read_grads(self._h, int(which_pass), _np_ptr(out)))
        return out

    def read_grads_replica(self, which_pass, k):
        out = np.empty(self.d, dtype=np.float32)
        self._check(lib().lsam_read_grads_replica(self._h, int(which_pass), int(k), _np_ptr(out)))
        return out

    def set_external_grads(self, g1, g2):
        self._keep += [g1, g2]
        self._check(lib().lsam_set_external_grads(self._h, _dev_ptr(g1), _dev_ptr(g2)))

    def write_state(self, x=None, v=None, y=None):
        cv = lambda a: None if a is None else a.contiguous().float()
        x, v, y = cv(x), cv(v), cv(y)
        self._check(lib().lsam_write_state(self._h, _dev_ptr(x), _dev_ptr(v), _dev_ptr(y)))
        self.stream.synchronize()

    def read_state(self):
        v = np.empty((self.K, self.d), dtype=np.float32)
        acc = np.empty(self.d, dtype=np.float32)
        gprev = np.empty(self.d, dtype=np.float32)
        self._check(lib().lsam_read_state(self._h, _np_ptr(v), _np_ptr(acc), _np_ptr(gprev)))
        return dict(v=v, acc=acc, gprev=gprev)

    def read_active(self):
        a = np.zeros(self.K, dtype=np.int32)
        self._check(lib().lsam_read_active(self._h, _np_ptr(a)))
        return a

    def counters(self):
        t = np.zeros(1, dtype=np.int64)
        ty = np.zeros(1, dtype=np.int64)
        tx = np.zeros(self.K, dtype=np.int64)
        self._check(lib().lsam_read_counters(self._h, _np_ptr(t), _np_ptr(ty), _np_ptr(tx)))
        return int(t[0]), int(ty[0]), tx

    def status(self):
        return int(lib().lsam_status(self._h))

    def last_error(self):
        return (lib().lsam_last_error(self._h) or b"").decode()

    def save_checkpoint(self):
        """The whole state of the run as a numpy byte array (host)."""
        n = int(lib().lsam_checkpoint_bytes(self._h))
        buf = np.empty(n, dtype=np.uint8)
        self._check(lib().lsam_save_checkpoint(self._h, _np_ptr(buf), n))
        return buf

    def load_checkpoint(self, buf):
        buf = np.ascontiguousarray(buf, dtype=np.uint8)
        self._check(lib().lsam_load_checkpoint(self._h, _np_ptr(buf), buf.size))

    def selftest_bounded_wait(self, polls=2048):
        """Enqueue a wait that is bound to expire (see include/lsam.h); status() then reports LSAM_ERR_TIMEOUT."""
        self._check(lib().lsam_selftest_bounded_wait(self._h, int(polls)))

    def profile_enable(self, on=True):
        self._check(lib().lsam_profile_enable(self._h, 1 if on else 0))

    def profile_read(self):
        ms = np.zeros(len(PROF_CLASSES), dtype=np.float64)
        n = np.zeros(len(PROF_CLASSES), dtype=np.int64)
        self._check(lib().lsam_profile_read(self._h, _np_ptr(ms), _np_ptr(n)))
        return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(PROF_CLASSES)}

    def launch_count(self):
        return int(lib().lsam_launch_count(self._h))

    def uses_tcgen05(self):
        return bool(lib().lsam_uses_tcgen05(self._h))
