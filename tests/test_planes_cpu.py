"""CPU checks of the arithmetic behind the fp32 GEMMs on the bf16 tensor cores (three bf16 planes per operand).

The library stores an fp32 operand a as p0 = bf16(a), p1 = bf16(a - p0), p2 = bf16(a - p0 - p1) and sums the plane pairs
(i, j) with i + j <= 2.  These tests restate the two facts the design rests on with torch's CPU bfloat16 (round to nearest
even, the conversion the kernels use): the planes add up to a exactly, and the three pairs left out are below fp32 rounding.
"""
import numpy as np
import torch


def planes(a):
    p0 = a.to(torch.bfloat16).to(torch.float32)
    r1 = a - p0
    p1 = r1.to(torch.bfloat16).to(torch.float32)
    r2 = r1 - p1
    p2 = r2.to(torch.bfloat16).to(torch.float32)
    return p0, p1, p2


def test_three_bf16_planes_add_up_to_the_fp32_value_exactly():
    g = torch.Generator().manual_seed(0)
    a = torch.randn(200_000, generator=g) * torch.exp(4 * torch.randn(200_000, generator=g))  # magnitudes over many binades
    a = torch.cat([a, torch.tensor([0.0, 1.0, -1.0, 3.0, 2.0 ** -100, 1.0 + 2.0 ** -23, 1.0 - 2.0 ** -24, 255.5, 65280.0])])
    p0, p1, p2 = planes(a)
    # the residuals are exact in fp32 (Sterbenz-style: each is a difference of nearby fp32 numbers), and 8 + 8 + 8 bits cover the 24
    assert torch.equal((p0 + p1) + p2, a)
    assert torch.equal(p0.double() + p1.double() + p2.double(), a.double())
    # each plane is at most 2^-8 of the one before (round to nearest: half a unit in the last of 8 places)
    nz = a != 0
    assert (p1[nz].abs() <= p0[nz].abs() * 2.0 ** -8).all() and (p2[nz].abs() <= p0[nz].abs() * 2.0 ** -16).all()


def test_the_plane_pairs_left_out_are_below_fp32_rounding():
    g = torch.Generator().manual_seed(1)
    n, kd = 64, 784
    A = torch.randn(n, kd, generator=g)
    B = torch.relu(torch.randn(n, kd, generator=g))
    pa, pb = planes(A), planes(B)
    exact = A.double() @ B.double().T
    kept = sum(pa[i].double() @ pb[j].double().T for i in range(3) for j in range(3) if i + j <= 2)
    dropped = sum(pa[i].double() @ pb[j].double().T for i in range(3) for j in range(3) if i + j > 2)
    np.testing.assert_allclose((kept + dropped).numpy(), exact.numpy(), rtol=0, atol=1e-12)  # nine pairs: the exact product of the planes
    scale = (A.abs().double() @ B.abs().double().T)
    assert (dropped.abs() <= 3 * 2.0 ** -24 * scale).all()  # per term below 2^-24 |a||b|, three pairs
    rel = (kept - exact).norm() / exact.norm()
    assert rel < 1e-7  # an fp32 FMA chain over 784 terms is at 2e-7 - 4e-7
