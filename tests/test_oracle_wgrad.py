"""Pins for the oracle's per-example weight gradients (not the CUDA path).

Each pin is something other than the oracle's own formula: PyTorch float64 autograd
run one example at a time, a finite difference of the linear functional <dY, conv(X,W)>,
the 1x1 special case as a matrix product, brute-force python loops on a tiny case and
the invariant that per-example gradients sum to the batch gradient.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_2109_12191_b200 import synth

CASES = [
    # Cin, Kout, R, stride, pad, H, W
    (3, 4, 3, 1, 1, 6, 6),
    (5, 7, 3, 2, 1, 9, 8),
    (4, 6, 1, 1, 0, 5, 7),
    (3, 8, 7, 2, 3, 18, 18),
    (2, 3, 3, 2, 1, 7, 7),
    (6, 5, 1, 2, 0, 8, 8),
    (2, 2, 5, 1, 0, 6, 9),
]


def _draw(B, H, W, Cin, Kout, R, stride, pad, seed):
    OH = (H + 2 * pad - R) // stride + 1
    OW = (W + 2 * pad - R) // stride + 1
    X = synth.normal_f32((B, H, W, Cin), 900, seed, 0)
    dY = synth.normal_f32((B, OH, OW, Kout), 900, seed, 1)
    return X, dY


def _torch_per_example(X, dY, R, stride, pad):
    """dW_n by autograd of sum(dY_n * conv2d(X_n, W)) one example at a time."""
    B, H, W, Cin = X.shape
    Kout = dY.shape[-1]
    out_w, out_b = [], []
    for n in range(B):
        x = torch.from_numpy(X[n:n + 1].astype(np.float64)).permute(0, 3, 1, 2)
        g = torch.from_numpy(dY[n:n + 1].astype(np.float64)).permute(0, 3, 1, 2)
        w = torch.zeros(Kout, Cin, R, R, dtype=torch.float64, requires_grad=True)
        b = torch.zeros(Kout, dtype=torch.float64, requires_grad=True)
        (F.conv2d(x, w, b, stride=stride, padding=pad) * g).sum().backward()
        out_w.append(w.grad.permute(0, 2, 3, 1).numpy().copy())   # [Kout,R,S,Cin]
        out_b.append(b.grad.numpy().copy())
    return np.stack(out_w), np.stack(out_b)


@pytest.mark.parametrize("case", CASES)
def test_conv_matches_autograd_per_example(case):
    Cin, Kout, R, stride, pad, H, W = case
    X, dY = _draw(3, H, W, Cin, Kout, R, stride, pad, sum(case))
    dW, db = oracle.conv_wgrad(X, dY, R, R, stride, pad, bias=True)
    tw, tb = _torch_per_example(X, dY, R, stride, pad)
    np.testing.assert_allclose(dW, tw, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(db, tb, rtol=1e-12, atol=1e-12)


def test_conv_finite_difference():
    """L(W) = <dY_n, conv(X_n, W)> is linear in W, so a central difference is exact up to rounding."""
    Cin, Kout, R, stride, pad, H, W = 3, 4, 3, 2, 1, 7, 6
    X, dY = _draw(2, H, W, Cin, Kout, R, stride, pad, 11)
    dW, _ = oracle.conv_wgrad(X, dY, R, R, stride, pad, bias=False)
    rng = np.random.default_rng(5)
    W0 = rng.standard_normal((Kout, Cin, R, R))

    def loss(n, Wt):
        x = torch.from_numpy(X[n:n + 1].astype(np.float64)).permute(0, 3, 1, 2)
        y = F.conv2d(x, torch.from_numpy(Wt), stride=stride, padding=pad)
        return float((y.permute(0, 2, 3, 1).numpy() * dY[n:n + 1]).sum())

    for n in range(2):
        for _ in range(12):
            k, c, r, s = rng.integers(Kout), rng.integers(Cin), rng.integers(R), rng.integers(R)
            E = np.zeros_like(W0)
            E[k, c, r, s] = 0.5
            fd = loss(n, W0 + E) - loss(n, W0 - E)
            assert abs(fd - dW[n, k, r, s, c]) < 1e-10 * max(1.0, abs(fd))


def test_conv_1x1_is_a_matrix_product():
    B, H, W, Cin, Kout = 3, 5, 6, 7, 4
    X, dY = _draw(B, H, W, Cin, Kout, 1, 1, 0, 3)
    dW, _ = oracle.conv_wgrad(X, dY, 1, 1, 1, 0, bias=False)
    for n in range(B):
        ref = dY[n].reshape(-1, Kout).astype(np.float64).T @ X[n].reshape(-1, Cin).astype(np.float64)
        np.testing.assert_allclose(dW[n, :, 0, 0, :], ref, rtol=1e-12, atol=1e-12)


def test_conv_brute_force_tiny():
    """Six nested python loops straight from the definition, on a tiny case."""
    B, H, W, Cin, Kout, R, stride, pad = 2, 5, 4, 2, 3, 3, 2, 1
    X, dY = _draw(B, H, W, Cin, Kout, R, stride, pad, 4)
    OH, OW = dY.shape[1:3]
    ref = np.zeros((B, Kout, R, R, Cin))
    Xp = np.zeros((B, H + 2 * pad, W + 2 * pad, Cin))
    Xp[:, pad:pad + H, pad:pad + W] = X
    for n in range(B):
        for k in range(Kout):
            for r in range(R):
                for s in range(R):
                    for c in range(Cin):
                        for oh in range(OH):
                            for ow in range(OW):
                                ref[n, k, r, s, c] += float(dY[n, oh, ow, k]) * Xp[n, oh * stride + r, ow * stride + s, c]
    dW, db = oracle.conv_wgrad(X, dY, R, R, stride, pad)
    np.testing.assert_allclose(dW, ref, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(db, dY.astype(np.float64).sum(axis=(1, 2)), rtol=1e-12, atol=1e-12)


def test_per_example_grads_sum_to_batch_gradient():
    Cin, Kout, R, stride, pad, H, W = 4, 5, 3, 1, 1, 8, 8
    B = 6
    X, dY = _draw(B, H, W, Cin, Kout, R, stride, pad, 21)
    dW, db = oracle.conv_wgrad(X, dY, R, R, stride, pad)
    x = torch.from_numpy(X.astype(np.float64)).permute(0, 3, 1, 2)
    g = torch.from_numpy(dY.astype(np.float64)).permute(0, 3, 1, 2)
    w = torch.zeros(Kout, Cin, R, R, dtype=torch.float64, requires_grad=True)
    b = torch.zeros(Kout, dtype=torch.float64, requires_grad=True)
    (F.conv2d(x, w, b, stride=stride, padding=pad) * g).sum().backward()
    np.testing.assert_allclose(dW.sum(0), w.grad.permute(0, 2, 3, 1).numpy(), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(db.sum(0), b.grad.numpy(), rtol=1e-11, atol=1e-11)


def test_dense_matches_autograd_and_rank1_norm():
    B, Cin, Kout = 5, 13, 7
    X = synth.normal_f32((B, Cin), 901, 0)
    dY = synth.normal_f32((B, Kout), 901, 1)
    dW, db = oracle.dense_wgrad(X, dY)
    for n in range(B):
        w = torch.zeros(Kout, Cin, dtype=torch.float64, requires_grad=True)
        b = torch.zeros(Kout, dtype=torch.float64, requires_grad=True)
        y = F.linear(torch.from_numpy(X[n:n + 1].astype(np.float64)), w, b)
        (y * torch.from_numpy(dY[n:n + 1].astype(np.float64))).sum().backward()
        np.testing.assert_allclose(dW[n], w.grad.numpy(), rtol=1e-13, atol=1e-13)
        np.testing.assert_allclose(db[n], b.grad.numpy(), rtol=1e-13, atol=1e-13)
    # closed form: ||dY_n^T X_n||_F^2 = ||dY_n||^2 ||X_n||^2
    closed = (dY.astype(np.float64) ** 2).sum(1) * (X.astype(np.float64) ** 2).sum(1)
    np.testing.assert_allclose(oracle.sqnorm(dW), closed, rtol=1e-12)
    np.testing.assert_allclose(oracle.sqnorm(db), (dY.astype(np.float64) ** 2).sum(1), rtol=1e-12)


def test_dense_equals_conv_on_a_1x1_image():
    B, Cin, Kout = 4, 6, 5
    X = synth.normal_f32((B, Cin), 902, 0)
    dY = synth.normal_f32((B, Kout), 902, 1)
    dW, db = oracle.dense_wgrad(X, dY)
    cW, cb = oracle.conv_wgrad(X.reshape(B, 1, 1, Cin), dY.reshape(B, 1, 1, Kout), 1, 1, 1, 0)
    np.testing.assert_array_equal(dW, cW.reshape(B, Kout, Cin))
    np.testing.assert_array_equal(db, cb)


def test_norm_affine_matches_autograd():
    B, H, W, C = 3, 4, 5, 6
    xhat = synth.normal_f32((B, H, W, C), 903, 0)
    dY = synth.normal_f32((B, H, W, C), 903, 1)
    dg, dbeta = oracle.norm_affine_wgrad(xhat, dY)
    for n in range(B):
        gamma = torch.ones(C, dtype=torch.float64, requires_grad=True)
        beta = torch.zeros(C, dtype=torch.float64, requires_grad=True)
        y = torch.from_numpy(xhat[n].astype(np.float64)) * gamma + beta
        (y * torch.from_numpy(dY[n].astype(np.float64))).sum().backward()
        np.testing.assert_allclose(dg[n], gamma.grad.numpy(), rtol=1e-13, atol=1e-13)
        np.testing.assert_allclose(dbeta[n], beta.grad.numpy(), rtol=1e-13, atol=1e-13)


def test_bf16_rounding_helper_is_round_to_nearest_even():
    a = np.array([1.0, 1.00390625, 1.01171875, -1.00390625, 3.0e-39, 65504.0, 1.0 + 2 ** -7], dtype=np.float32)
    bits, wide = synth.round_to_bf16(a)
    ref = torch.from_numpy(a).to(torch.bfloat16)
    np.testing.assert_array_equal(wide, ref.to(torch.float32).numpy())
    np.testing.assert_array_equal(bits.view(np.int16), ref.view(torch.int16).numpy())
    big = synth.normal_f32((4096,), 904)
    b2, w2 = synth.round_to_bf16(big)
    np.testing.assert_array_equal(w2, torch.from_numpy(big).to(torch.bfloat16).to(torch.float32).numpy())
