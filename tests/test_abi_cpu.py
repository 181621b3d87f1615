"""CPU-only checks of the C-ABI library: it loads, exports what include/lsam.h declares, and its host-only logic."""
import ctypes as C
import os
import re

import numpy as np

import oracle as O
from paper_2509_03110_b200 import binding as G
from paper_2509_03110_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "lsam.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(lsam_[a-z0-9_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    names = _declared()
    assert "lsam_init" in names and "lsam_step" in names and "lsam_couple" in names and "lsam_read_params" in names
    L = G.lib()
    for n in names:
        assert hasattr(L, n), n
    assert sorted(G.EXPORTS) == names


def test_config_struct_matches_header_size(tmp_path):
    # the ctypes mirror of lsam_config against the header itself, as the C compiler lays it out: size and field offsets
    import subprocess

    fields = [f[0] for f in G.LsamConfig._fields_]
    cname = {"lam": "lambda"}
    src = tmp_path / "layout.c"
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "lsam.h"', 'int main(void) {', '  printf("%zu\\n", sizeof(lsam_config));']
    lines += [f'  printf("%zu\\n", offsetof(lsam_config, {cname.get(f, f)}));' for f in fields]
    lines += ['  return 0;', '}']
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    out = [int(v) for v in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()]
    assert C.sizeof(G.LsamConfig) == out[0]
    assert [getattr(G.LsamConfig, f).offset for f in fields] == out[1:]


def test_binding_enumerators_match_the_header(tmp_path):
    # every constant the binding mirrors, printed by a C program that includes the header
    import subprocess

    names = {"LSAM_OK": G.LSAM_OK, "LSAM_ERR_INVALID": G.LSAM_ERR_INVALID, "LSAM_ERR_WORKSPACE": G.LSAM_ERR_WORKSPACE, "LSAM_ERR_STATE": G.LSAM_ERR_STATE,
             "LSAM_ERR_CUDA": G.LSAM_ERR_CUDA, "LSAM_ERR_NONFINITE": G.LSAM_ERR_NONFINITE, "LSAM_ERR_TIMEOUT": G.LSAM_ERR_TIMEOUT}
    for group in ("MODEL_LSQ MODEL_MLP MODEL_RESMLP MODEL_FLAT MODEL_CNN GEMM_FP32 GEMM_BF16 IMPL_AUTO IMPL_SIMT IMPL_TCGEN05 IMPL_TCGEN05_1CTA "
                  "IMPL_TCGEN05_PAIRS KERNEL_GAUSSIAN KERNEL_EXP_POWER KERNEL_CAUCHY KERNEL_MATERN32 FLAG_KEEP_G1 FLAG_STEP_INFO FLAG_CUDA_GRAPH "
                  "FLAG_GRAD_FP32 FLAG_FUSED_UPDATE FLAG_PDL").split():
        names["LSAM_" + group] = getattr(G, group)
    names["LSAM_PROF_CLASSES"] = len(G.PROF_CLASSES)
    for i, cls in enumerate(G.PROF_CLASSES):
        names["LSAM_PROF_" + cls.upper()] = i
    src = tmp_path / "enums.c"
    keys = sorted(names)
    src.write_text("\n".join(['#include <stdio.h>', '#include "lsam.h"', 'int main(void) {'] + [f'  printf("%d\\n", (int){k});' for k in keys] + ['  return 0;', '}']))
    exe = tmp_path / "enums"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    out = [int(v) for v in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()]
    assert dict(zip(keys, out)) == names


def test_param_counts_and_workspace_of_the_five_configs():
    cases = [
        (G.make_config(G.MODEL_LSQ, widths=(256,), K=4, batch=32, n_samples=4096), 256),
        (G.make_config(G.MODEL_MLP, widths=(784, 1024, 10), K=8, batch=128, n_samples=60000), 814090),
        (G.make_config(G.MODEL_MLP, widths=(3072, 2048, 2048, 2048, 100), K=16, batch=128, n_samples=50000, gemm_dtype=G.GEMM_BF16), 14891108),
        (G.make_config(G.MODEL_RESMLP, widths=(3072, 4096, 4096, 4096, 4096, 1000), K=32, batch=256, n_samples=200000, gemm_dtype=G.GEMM_BF16, stale_max=3), 67027944),
        (G.make_config(G.MODEL_FLAT, K=8, flat_d=256_000_000), 256_000_000),
    ]
    for cfg, d in cases:
        assert G.lsam_param_count(cfg) == d
        ws = G.lsam_workspace_bytes(cfg)
        assert ws > 3 * 4 * cfg.K * d  # at least x, v and one more [K, d] fp32 tensor ... FLAT has no gradient buffer
        assert ws < 180e9
    # same parameter counts as the oracle and the input generator
    assert synth.mlp_param_count((784, 1024, 10)) == 814090
    assert O.param_count(O.make_config(O.MODEL_MLP, widths=(784, 1024, 10), K=1, batch=1)) == 814090


def test_invalid_configs_rejected_on_host():
    bad = [
        G.make_config(G.MODEL_FLAT, K=0, flat_d=8),
        G.make_config(G.MODEL_FLAT, K=1, flat_d=8, tau=0),
        G.make_config(G.MODEL_FLAT, K=1, flat_d=8, stale_max=16),
        G.make_config(G.MODEL_FLAT, K=1, flat_d=8, gemm_dtype=G.GEMM_BF16),
        G.make_config(G.MODEL_LSQ, widths=(8,), K=1, batch=0, n_samples=4),
        G.make_config(7, K=1),
    ]
    for cfg in bad:
        assert G.lsam_param_count(cfg) == -1
        assert G.lsam_workspace_bytes(cfg) == 0


def test_host_schedule_hash_matches_oracle():
    rng = np.random.default_rng(0)
    for _ in range(200):
        seed, t = int(rng.integers(0, 2**63)), int(rng.integers(0, 2**40))
        k, j = int(rng.integers(0, 4096)), int(rng.integers(0, 2**20))
        assert G.lsam_schedule_hash(seed, 0, t, k, j) == O.hash5(seed, O.lib().oracle_tag_idx(), t, k, j)
        assert G.lsam_schedule_hash(seed, 1, t, k, 0) == O.hash5(seed, O.lib().oracle_tag_stale(), t, k, 0)


def test_null_context_calls_fail_cleanly():
    L = G.lib()
    assert L.lsam_step(None, 0.1, 0.1) == G.LSAM_ERR_INVALID
    assert L.lsam_couple(None) == G.LSAM_ERR_INVALID
    assert L.lsam_should_couple(None) == 0
    assert L.lsam_status(None) == G.LSAM_ERR_INVALID
    assert L.lsam_launch_count(None) == 0
    L.lsam_destroy(None)
