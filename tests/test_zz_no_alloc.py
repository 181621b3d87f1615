"""The allocation-free row-norm entry point against the norms that lsam_step() itself produces.

Some users of the library cannot allocate device memory at the point where they need a gradient norm: they run
inside a memory pool that already owns the whole GPU, or in a hot loop where cudaMalloc would stall the device.
lsam_row_norms_static() serves them with scratch that is built into the library.  This file is collected last so
that a run which stops at the first failure has already exercised everything else.
"""
import numpy as np
import pytest

from paper_2509_03110_b200 import binding as G
from paper_2509_03110_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,d", [(8, 1_000_000), (3, 1001)])
def test_static_row_norms_match_step_norms_twice_in_a_row(K, d):
    import torch

    x0, y0, g1, g2 = synth.flat_problem(K, d, seed=11)
    dg1, dg2 = torch.from_numpy(g1).cuda(), torch.from_numpy(g2).cuda()
    cfg = G.make_config(G.MODEL_FLAT, K=K, flat_d=d, tau=4, lam=0.1, flags=G.FLAG_STEP_INFO)
    ctx = G.Lsam(cfg, None, None, torch.from_numpy(x0).cuda(), torch.from_numpy(y0).cuda())
    ctx.set_external_grads(dg1, dg2)
    ctx.step(0.05, 0.1)
    _, n1, n2 = ctx.read_step_info()  # the existing path: ||g1_k|| and ||g2_k|| through the workspace
    out = torch.full((K,), -1.0, device="cuda")
    stream = torch.cuda.current_stream()
    mem_before = torch.cuda.memory_allocated()
    # two calls in a row on different data: the second must not see anything of the first
    rc, msg = G.lsam_row_norms_static(dg1, d, out, stream)
    assert rc == G.LSAM_OK, msg
    got1 = out.cpu().numpy().copy()
    rc, msg = G.lsam_row_norms_static(dg2, d, out, stream)
    assert rc == G.LSAM_OK, msg
    got2 = out.cpu().numpy().copy()
    assert torch.cuda.memory_allocated() == mem_before
    np.testing.assert_allclose(got1, n1, rtol=1e-5)
    np.testing.assert_allclose(got2, n2, rtol=1e-5)
    np.testing.assert_allclose(got1, np.linalg.norm(g1.astype(np.float64), axis=1), rtol=1e-5)
    # and once more on the first buffer: same result as before, bit for bit (fixed reduction order)
    rc, msg = G.lsam_row_norms_static(dg1, d, out, stream)
    assert rc == G.LSAM_OK, msg
    np.testing.assert_array_equal(out.cpu().numpy(), got1)
    ctx.close()


def test_static_row_norms_reduce_only_the_first_n_columns_of_padded_rows():
    # rows whose stride is a multiple of 4 but whose length is not: the columns n .. ld-1 hold other data and must not count
    import torch

    K, ld, n = 5, 1004, 1001
    rng = np.random.default_rng(3)
    g = rng.standard_normal((K, ld)).astype(np.float32)
    g[:, n:] = 100.0  # would dominate the norm if it were read
    dg = torch.from_numpy(g).cuda()
    out = torch.full((K,), -1.0, device="cuda")
    for _ in range(2):
        rc, msg = G.lsam_row_norms_static(dg, n, out, torch.cuda.current_stream())
        assert rc == G.LSAM_OK, msg
        np.testing.assert_allclose(out.cpu().numpy(), np.linalg.norm(g[:, :n].astype(np.float64), axis=1), rtol=1e-5)
    # and a row length that IS a multiple of 4 inside a wider stride takes the 128-bit path
    rc, msg = G.lsam_row_norms_static(dg, 1000, out, torch.cuda.current_stream())
    assert rc == G.LSAM_OK, msg
    np.testing.assert_allclose(out.cpu().numpy(), np.linalg.norm(g[:, :1000].astype(np.float64), axis=1), rtol=1e-5)


def test_static_row_norms_reject_oversize_and_bad_arguments():
    import torch

    g = torch.zeros(4, 64, device="cuda")
    out = torch.zeros(4, device="cuda")
    # claim a problem far beyond the built-in scratch (nothing is launched, so the small buffer is never touched)
    err = G.C.create_string_buffer(256)
    rc = G.lib().lsam_row_norms_static(G.C.c_void_p(g.data_ptr()), 10**10, 10**10, 4, G.C.c_void_p(out.data_ptr()), None, err, 256)
    assert rc == G.LSAM_ERR_WORKSPACE and b"exceed" in err.value
    rc = G.lib().lsam_row_norms_static(None, 64, 64, 4, G.C.c_void_p(out.data_ptr()), None, err, 256)
    assert rc == G.LSAM_ERR_INVALID and err.value
    rc = G.lib().lsam_row_norms_static(G.C.c_void_p(g.data_ptr()), 32, 64, 4, G.C.c_void_p(out.data_ptr()), None, None, 0)
    assert rc == G.LSAM_ERR_INVALID
    torch.cuda.synchronize()
