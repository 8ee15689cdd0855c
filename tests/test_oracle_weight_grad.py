"""Pins for the oracle's weight gradients (Eq. 4-6 and App. A.3 of arXiv 2202.13808)."""
import numpy as np
import pytest
import torch

import dropit_inputs as di
import oracle


def _setup(case):
    xb, dt = oracle.to_bits(di.make_x(case))
    dyb, _ = oracle.to_bits(di.make_dy(case))
    keep, k = oracle.min_k(xb, case.gamma, dt)
    return xb, dyb, keep, dt


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_fc_gamma_zero_is_the_dense_gradient(dtype):
    # Table 2 "0% (Baseline)": nothing dropped, Eq. 6 is the plain GEMM dY^T X
    case = di.small_linear(61, 37, 23, dtype, 0.0, dy_std=1.0)
    xb, dyb, keep, dt = _setup(case)
    assert keep.all()
    dw = oracle.fc_weight_grad(dyb, xb, keep, case.M, case.Ca, case.Cz, dt)
    X = oracle.bits_to_float64(xb, dt).reshape(case.M, case.Ca)
    DY = oracle.bits_to_float64(dyb, dt).reshape(case.M, case.Cz)
    ref = DY.T @ X
    assert dw.shape == (case.Cz, case.Ca)
    np.testing.assert_allclose(dw, ref, rtol=1e-12, atol=1e-12 * np.abs(ref).max())


@pytest.mark.parametrize("gamma", [0.5, 0.9, 1.0])
def test_fc_equals_masked_matmul(gamma):
    # App. A.3: G' = (A o D) x Z
    case = di.small_linear(200, 96, 40, "bf16", gamma, dy_std=1.0)
    xb, dyb, keep, dt = _setup(case)
    dw = oracle.fc_weight_grad(dyb, xb, keep, case.M, case.Ca, case.Cz, dt)
    X = oracle.bits_to_float64(xb, dt).reshape(case.M, case.Ca) * keep.reshape(case.M, case.Ca)
    DY = oracle.bits_to_float64(dyb, dt).reshape(case.M, case.Cz)
    ref = DY.T @ X
    np.testing.assert_allclose(dw, ref, rtol=1e-12, atol=1e-12 * max(np.abs(ref).max(), 1e-300))
    if gamma == 1.0:
        assert not dw.any()


def test_fc_is_a_sum_of_rank_one_updates_over_retained_entries():
    case = di.small_linear(9, 7, 5, "f32", 0.6, dy_std=1.0)
    xb, dyb, keep, dt = _setup(case)
    X = oracle.bits_to_float64(xb, dt).reshape(case.M, case.Ca)
    DY = oracle.bits_to_float64(dyb, dt).reshape(case.M, case.Cz)
    ref = np.zeros((case.Cz, case.Ca))
    for n in range(case.M):
        for c in range(case.Ca):
            if keep[n * case.Ca + c]:
                for j in range(case.Cz):
                    ref[j, c] += DY[n, j] * X[n, c]
    dw = oracle.fc_weight_grad(dyb, xb, keep, case.M, case.Ca, case.Cz, dt)
    np.testing.assert_allclose(dw, ref, rtol=1e-13, atol=1e-13)
    js = np.array([0, 4, 2, 3]); cs = np.array([6, 0, 3, 3])
    ent = oracle.fc_weight_grad_entries(dyb, xb, keep, case.M, case.Ca, case.Cz, dt, js, cs)
    np.testing.assert_allclose(ent, ref[js, cs], rtol=1e-13, atol=1e-13)


def _conv_ref_torch(case, xb, dyb, keep, dt):
    X = torch.from_numpy(oracle.bits_to_float64(xb, dt) * keep).reshape(case.B, case.Ca, case.H, case.W)
    DY = torch.from_numpy(oracle.bits_to_float64(dyb, dt)).reshape(case.B, case.Cz, case.Ho, case.Wo)
    return torch.nn.grad.conv2d_weight(X, (case.Cz, case.Ca, case.R, case.S), DY, stride=case.stride,
                                       padding=case.pad).numpy()


@pytest.mark.parametrize("case", [
    di.small_conv(2, 5, 9, 7, 4, 1, 1, 1, 0, "bf16", 0.8),
    di.small_conv(2, 3, 9, 7, 4, 3, 3, 1, 1, "bf16", 0.8),
    di.small_conv(2, 3, 9, 8, 4, 3, 3, 2, 1, "f32", 0.5),
    di.small_conv(1, 2, 6, 6, 3, 3, 2, 1, 0, "f32", 0.0),
])
def test_conv_against_torch_float64_on_the_masked_input(case):
    xb, dyb, keep, dt = _setup(case)
    dw = oracle.conv_weight_grad(dyb, xb, keep, case.B, case.Ca, case.H, case.W, case.Cz, case.R, case.S, case.stride,
                                 case.pad, dt)
    ref = _conv_ref_torch(case, xb, dyb, keep, dt)
    np.testing.assert_allclose(dw, ref, rtol=1e-11, atol=1e-12 * max(np.abs(ref).max(), 1e-300))
    rng = np.random.default_rng(0)
    js = rng.integers(0, case.Cz, 6); cs = rng.integers(0, case.Ca, 6)
    us = rng.integers(0, case.R, 6); vs = rng.integers(0, case.S, 6)
    ent = oracle.conv_weight_grad_entries(dyb, xb, keep, case.B, case.Ca, case.H, case.W, case.Cz, case.R, case.S,
                                          case.stride, case.pad, dt, js, cs, us, vs)
    np.testing.assert_allclose(ent, dw[js, cs, us, vs], rtol=1e-13, atol=1e-300)


def test_conv_1x1_is_the_fc_gradient_on_the_transposed_view():
    case = di.small_conv(3, 6, 5, 4, 7, 1, 1, 1, 0, "bf16", 0.8)
    xb, dyb, keep, dt = _setup(case)
    dwc = oracle.conv_weight_grad(dyb, xb, keep, case.B, case.Ca, case.H, case.W, case.Cz, 1, 1, 1, 0, dt)
    HW = case.H * case.W
    tr = lambda a, C: a.reshape(case.B, C, HW).transpose(0, 2, 1).reshape(-1).copy()
    dwf = oracle.fc_weight_grad(tr(dyb, case.Cz), tr(xb, case.Ca), tr(keep, case.Ca), case.B * HW, case.Ca, case.Cz, dt)
    np.testing.assert_allclose(dwc.reshape(case.Cz, case.Ca), dwf, rtol=1e-13, atol=1e-300)


def test_conv_tiny_brute_force_python_loops():
    case = di.small_conv(1, 2, 4, 3, 2, 3, 3, 1, 1, "f32", 0.5)
    xb, dyb, keep, dt = _setup(case)
    X = (oracle.bits_to_float64(xb, dt) * keep).reshape(1, 2, 4, 3)
    DY = oracle.bits_to_float64(dyb, dt).reshape(1, 2, 4, 3)
    ref = np.zeros((2, 2, 3, 3))
    for j in range(2):
        for c in range(2):
            for u in range(3):
                for v in range(3):
                    for y in range(4):
                        for x in range(3):
                            yi, xi = y + u - 1, x + v - 1
                            if 0 <= yi < 4 and 0 <= xi < 3:
                                ref[j, c, u, v] += DY[0, j, y, x] * X[0, c, yi, xi]
    dw = oracle.conv_weight_grad(dyb, xb, keep, 1, 2, 4, 3, 2, 3, 3, 1, 1, dt)
    np.testing.assert_allclose(dw, ref, rtol=1e-13, atol=1e-300)
