"""Pins for the oracle's operators: each is checked against something that is not itself -
a literal brute-force loop on tiny tensors, a library routine it does not use, a closed form."""
import itertools

import numpy as np
import pytest
import torch
import torch.nn.functional as F


def brute_conv(x, w, stride, pad):
    """The definition, as seven literal loops over Python floats."""
    N, C, H, W = x.shape
    K, _, R, S = w.shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    y = np.zeros((N, K, P, Q))
    for n in range(N):
        for k in range(K):
            for p in range(P):
                for q in range(Q):
                    acc = 0.0
                    for c in range(C):
                        for r in range(R):
                            for s in range(S):
                                ih, iw = p * stride + r - pad, q * stride + s - pad
                                if 0 <= ih < H and 0 <= iw < W:
                                    acc += x[n, c, ih, iw] * w[k, c, r, s]
                    y[n, k, p, q] = acc
    return y


@pytest.mark.parametrize("R,stride,pad", [(1, 1, 0), (1, 2, 0), (3, 1, 1), (3, 2, 1), (3, 1, 0), (3, 2, 0),
                                          (5, 2, 2), (7, 2, 3), (3, 1, 2)])
def test_conv_brute_force(fpo, R, stride, pad):
    rng = np.random.default_rng(R * 100 + stride * 10 + pad)
    for (N, C, K, H, W) in [(2, 3, 4, 5, 4), (1, 1, 1, 7, 7), (2, 4, 2, 8, 5)]:
        if H + 2 * pad < R or W + 2 * pad < R:
            continue
        x = rng.standard_normal((N, C, H, W))
        w = rng.standard_normal((K, C, R, R))
        got = fpo.conv2d(x, w, stride, pad)
        ref = brute_conv(x, w, stride, pad)
        assert got.shape == ref.shape
        np.testing.assert_allclose(got, ref, rtol=0, atol=1e-13)


def test_conv_asymmetric_values_catch_transposition(fpo):
    # one-hot input and filter: the only non-zero output sits where the definition puts it
    x = np.zeros((1, 2, 5, 6)); x[0, 1, 3, 4] = 2.0
    w = np.zeros((3, 2, 3, 3)); w[2, 1, 0, 2] = 5.0
    y = fpo.conv2d(x, w, 1, 1)
    # y[p,q] = x[p+r-1, q+s-1] * w[r,s]  =>  p = 3-0+1 = 4, q = 4-2+1 = 3
    expect = np.zeros_like(y); expect[0, 2, 4, 3] = 10.0
    np.testing.assert_array_equal(y, expect)


@pytest.mark.parametrize("stride,pad,R", [(1, 1, 3), (2, 1, 3), (2, 3, 7), (1, 0, 1), (2, 0, 1)])
def test_conv_vs_library(fpo, stride, pad, R):
    rng = np.random.default_rng(3)
    x = rng.standard_normal((3, 5, 13, 11))
    w = rng.standard_normal((6, 5, R, R))
    ref = F.conv2d(torch.from_numpy(x), torch.from_numpy(w), stride=stride, padding=pad).numpy()
    np.testing.assert_allclose(fpo.conv2d(x, w, stride, pad), ref, rtol=1e-12, atol=1e-12)


def test_conv_1x1_is_matrix_product(fpo):
    rng = np.random.default_rng(4)
    x = rng.standard_normal((2, 7, 4, 3))
    w = rng.standard_normal((5, 7, 1, 1))
    ref = np.einsum("kc,nchw->nkhw", w[:, :, 0, 0], x)
    np.testing.assert_allclose(fpo.conv2d(x, w, 1, 0), ref, rtol=1e-13, atol=1e-13)


def test_identity_convolution_returns_input(fpo):
    # Sec. IV-B.1: the auxiliary operator's weights are identity matrices, x = xconv(x, W~)
    rng = np.random.default_rng(5)
    x = rng.standard_normal((2, 6, 5, 5))
    I = fpo._identity_filters(6, 6, 3, 3)
    assert I.sum() == 6 and np.count_nonzero(I) == 6
    np.testing.assert_array_equal(fpo.conv2d(x, I, 1, 1), x)
    # stride-2 centre tap of a 3x3/pad-1 filter reads the pixel a 1x1/stride-2 filter reads
    np.testing.assert_array_equal(fpo.conv2d(x, I, 2, 1), x[:, :, ::2, ::2])


def test_padded_1x1_equals_3x3(fpo):
    # Sec. IV-B.1: a 1x1 convolution padded with zeros to 3x3 produces the same output
    rng = np.random.default_rng(6)
    x = rng.standard_normal((2, 4, 6, 6))
    w = rng.standard_normal((3, 4, 1, 1))
    for stride in (1, 2):
        a = fpo.conv2d(x, w, stride, 0)
        b = fpo.conv2d(x, fpo._pad_to(w, 3, 3), stride, 1)
        np.testing.assert_allclose(a, b, rtol=0, atol=1e-14)


def test_bn_affine_form(fpo):
    # Eq. 3-5: BN(x) = omega*x + lambda with omega = gamma/sqrt(var+eps), lambda = beta - omega*mean
    rng = np.random.default_rng(7)
    x = rng.standard_normal((2, 5, 3, 4))
    g, b, m = rng.uniform(0.5, 1.5, 5), rng.standard_normal(5), rng.standard_normal(5)
    v, eps = rng.uniform(0.5, 1.5, 5), 1e-5
    omega = g / np.sqrt(v + eps)
    lam = b - omega * m
    ref = omega[None, :, None, None] * x + lam[None, :, None, None]
    np.testing.assert_allclose(fpo.batchnorm(x, g, b, m, v, eps), ref, rtol=1e-13, atol=1e-13)
    lib = F.batch_norm(torch.from_numpy(x), torch.from_numpy(m), torch.from_numpy(v), torch.from_numpy(g),
                       torch.from_numpy(b), False, 0.0, eps).numpy()
    np.testing.assert_allclose(fpo.batchnorm(x, g, b, m, v, eps), lib, rtol=1e-12, atol=1e-12)


def test_fold_equals_conv_then_bn(fpo):
    rng = np.random.default_rng(8)
    x = rng.standard_normal((2, 4, 6, 6))
    w = rng.standard_normal((5, 4, 3, 3))
    g, b, m, v = rng.uniform(0.5, 1.5, 5), rng.standard_normal(5), rng.standard_normal(5), rng.uniform(0.5, 1.5, 5)
    ref = fpo.batchnorm(fpo.conv2d(x, w, 1, 1), g, b, m, v, 1e-5)
    W, lam, _ = fpo.fold64(w, g, b, m, v, 1e-5)
    got = fpo.add_bias(fpo.conv2d(x, W, 1, 1), lam)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)
    # the single-precision fold follows the same map to fp32 accuracy
    W32, lam32, om32 = fpo.fold32(w.astype(np.float32), g, b, m, v, 1e-5)
    np.testing.assert_allclose(W32, W, rtol=3e-6, atol=1e-7)
    np.testing.assert_allclose(lam32, lam, rtol=1e-5, atol=1e-6)


def test_fold32_operation_order_bits():
    # each step is one rounded fp32 operation: reproduce with numpy float32 scalars
    from oracle import fpo
    rng = np.random.default_rng(9)
    w = rng.standard_normal((3, 2, 3, 3)).astype(np.float32)
    g, b, m, v = (rng.uniform(0.5, 1.5, 3).astype(np.float32) for _ in range(4))
    eps = np.float32(1e-5)
    W32, lam32, om32 = fpo.fold32(w, g, b, m, v, 1e-5)
    for k in range(3):
        t = np.float32(v[k] + eps)
        r = np.float32(np.sqrt(t))
        om = np.float32(g[k] / r)
        assert om == om32[k]
        np.testing.assert_array_equal(W32[k], (om * w[k]).astype(np.float32))
        assert lam32[k] == np.float32(b[k] - np.float32(om * m[k]))


def test_relu_add(fpo):
    a = np.array([[-1.0, 0.0, 2.5, -0.0]])
    np.testing.assert_array_equal(fpo.relu(a), np.array([[0.0, 0.0, 2.5, 0.0]]))
    np.testing.assert_array_equal(fpo.add(a, a), 2 * a)


def test_maxpool_vs_library(fpo):
    rng = np.random.default_rng(10)
    for H, W in [(8, 8), (7, 9), (5, 5)]:
        x = rng.standard_normal((2, 3, H, W)) - 3.0   # all-negative regions: padding must not win
        ref = F.max_pool2d(torch.from_numpy(x), 3, 2, 1).numpy()
        np.testing.assert_array_equal(fpo.maxpool(x, 3, 2, 1), ref)


def test_gavgpool_fc(fpo):
    rng = np.random.default_rng(11)
    x = rng.standard_normal((3, 4, 5, 6))
    np.testing.assert_allclose(fpo.gavgpool(x), x.mean(axis=(2, 3)), rtol=1e-13, atol=1e-14)
    v = rng.standard_normal((3, 4)); w = rng.standard_normal((5, 4)); b = rng.standard_normal(5)
    np.testing.assert_allclose(fpo.fc(v, w, b), v @ w.T + b, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(fpo.fc(v, w), v @ w.T, rtol=1e-13, atol=1e-13)


def test_shortcut_a(fpo):
    rng = np.random.default_rng(12)
    x = rng.standard_normal((2, 4, 6, 6))
    y = fpo.shortcut_a(x, 8, 2, 0)
    ref = np.zeros((2, 8, 3, 3)); ref[:, :4] = x[:, :, ::2, ::2]
    np.testing.assert_array_equal(y, ref)
    y = fpo.shortcut_a(x, 8, 2, 2)
    ref = np.pad(x[:, :, ::2, ::2], ((0, 0), (2, 2), (0, 0), (0, 0)))
    np.testing.assert_array_equal(y, ref)
    np.testing.assert_array_equal(fpo.shortcut_a(x, 4, 1, 0), x)
