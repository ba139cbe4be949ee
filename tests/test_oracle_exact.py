"""Pins of the oracle's exact filter gradient against things other than itself."""
import itertools

import numpy as np
import pytest
import torch

from oracle import oracle

GEOMS = [
    # n c h w k r s st_h st_w pad_h pad_w
    oracle.Shape(2, 3, 6, 5, 4, 3, 3, 1, 1, 1, 1),
    oracle.Shape(1, 2, 7, 7, 3, 3, 3, 2, 2, 1, 1),
    oracle.Shape(3, 2, 8, 6, 2, 5, 5, 1, 1, 2, 2),
    oracle.Shape(2, 2, 5, 5, 2, 1, 1, 1, 1, 0, 0),
    oracle.Shape(4, 1, 6, 6, 2, 3, 3, 2, 1, 0, 2),
    oracle.Shape(2, 3, 4, 4, 2, 3, 3, 1, 1, 0, 0),
    oracle.Shape(1, 2, 9, 8, 2, 5, 3, 2, 2, 2, 1),
]


def _rand(g, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((g.n, g.c, g.h, g.w)), rng.standard_normal((g.n, g.k, g.p, g.q))


def forward_conv(x, w, g):
    """y = conv(x, w) written independently of the oracle: explicit zero-padded copy, then windows."""
    xp = np.pad(x, ((0, 0), (0, 0), (g.pad_h, g.pad_h), (g.pad_w, g.pad_w)))
    y = np.zeros((g.n, g.k, g.p, g.q))
    for p in range(g.p):
        for q in range(g.q):
            win = xp[:, :, p * g.stride_h:p * g.stride_h + g.r, q * g.stride_w:q * g.stride_w + g.s]
            y[:, :, p, q] = np.einsum("ncrs,kcrs->nk", win, w)
    return y


@pytest.mark.parametrize("g", GEOMS)
def test_finite_differences_linear_loss(g):
    """L(W) = <conv(X,W), G> is linear in W, so a central difference is exact up to rounding."""
    x, gy = _rand(g, 1)
    dw, _ = oracle.dw_exact(x, gy, g)
    rng = np.random.default_rng(2)
    w0 = rng.standard_normal((g.k, g.c, g.r, g.s))
    eps = 0.5
    for k, c, r, s in itertools.product(range(g.k), range(g.c), range(g.r), range(g.s)):
        e = np.zeros_like(w0); e[k, c, r, s] = eps
        fd = (np.sum(forward_conv(x, w0 + e, g) * gy) - np.sum(forward_conv(x, w0 - e, g) * gy)) / (2 * eps)
        assert abs(fd - dw[k, c, r, s]) <= 1e-10 * max(1.0, abs(fd))


@pytest.mark.parametrize("g", GEOMS[:3])
def test_finite_differences_quadratic_loss(g):
    """L(W) = 0.5 ||conv(X,W)||^2 has dL/dY = Y; its W-derivative must be dW(X, Y)."""
    x, _ = _rand(g, 3)
    rng = np.random.default_rng(4)
    w0 = rng.standard_normal((g.k, g.c, g.r, g.s)) * 0.3
    y0 = forward_conv(x, w0, g)
    dw, _ = oracle.dw_exact(x, y0, g)
    eps = 1e-5
    for k, c, r, s in itertools.islice(itertools.product(range(g.k), range(g.c), range(g.r), range(g.s)), 0, None, 3):
        e = np.zeros_like(w0); e[k, c, r, s] = eps
        lp = 0.5 * np.sum(forward_conv(x, w0 + e, g) ** 2); lm = 0.5 * np.sum(forward_conv(x, w0 - e, g) ** 2)
        fd = (lp - lm) / (2 * eps)
        assert abs(fd - dw[k, c, r, s]) <= 1e-6 * max(1.0, abs(fd))


@pytest.mark.parametrize("g", GEOMS)
def test_brute_force_seven_loops(g):
    x, dy = _rand(g, 5)
    alpha = -0.75
    dw, dn = oracle.dw_exact(x, dy, g, alpha)
    ref = np.zeros_like(dw); refn = np.zeros_like(dw)
    for k in range(g.k):
        for c in range(g.c):
            for r in range(g.r):
                for s in range(g.s):
                    for n in range(g.n):
                        for p in range(g.p):
                            for q in range(g.q):
                                hh = p * g.stride_h + r - g.pad_h; ww = q * g.stride_w + s - g.pad_w
                                if 0 <= hh < g.h and 0 <= ww < g.w:
                                    ref[k, c, r, s] += alpha * x[n, c, hh, ww] * dy[n, k, p, q]
                                    refn[k, c, r, s] += abs(alpha * x[n, c, hh, ww] * dy[n, k, p, q])
    np.testing.assert_allclose(dw, ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(dn, refn, rtol=1e-12, atol=1e-12)
    v, nrm = oracle.dw_exact_at(x, dy, g, g.k - 1, g.c - 1, g.r - 1, 0, alpha)
    assert v == dw[g.k - 1, g.c - 1, g.r - 1, 0] and nrm == dn[g.k - 1, g.c - 1, g.r - 1, 0]


@pytest.mark.parametrize("g", [GEOMS[0], GEOMS[1], GEOMS[2], GEOMS[6]])
def test_delta_inputs_closed_form(g):
    """One non-zero in X and one in dY: dW has one non-zero, at r = h0 - p0*st + pad (same for s)."""
    for (h0, w0, p0, q0) in [(0, 0, 0, 0), (g.h - 1, g.w - 1, g.p - 1, g.q - 1), (2, 1, 1, 0), (3, 3, 1, 1)]:
        x = np.zeros((g.n, g.c, g.h, g.w)); dy = np.zeros((g.n, g.k, g.p, g.q))
        n0, c0, k0 = g.n - 1, g.c - 1, 0
        x[n0, c0, h0, w0] = 2.0; dy[n0, k0, p0, q0] = -3.0
        dw, _ = oracle.dw_exact(x, dy, g)
        want = np.zeros_like(dw)
        r0 = h0 - p0 * g.stride_h + g.pad_h; s0 = w0 - q0 * g.stride_w + g.pad_w
        if 0 <= r0 < g.r and 0 <= s0 < g.s:
            want[k0, c0, r0, s0] = -6.0
        np.testing.assert_array_equal(dw, want)


def test_pointwise_filter_is_a_matrix_product():
    g = oracle.Shape(3, 5, 4, 6, 7, 1, 1)
    x, dy = _rand(g, 6)
    dw, _ = oracle.dw_exact(x, dy, g)
    ref = dy.transpose(1, 0, 2, 3).reshape(g.k, -1) @ x.transpose(1, 0, 2, 3).reshape(g.c, -1).T
    np.testing.assert_allclose(dw[:, :, 0, 0], ref, rtol=0, atol=1e-12)


def test_full_window_filter_is_a_matrix_product():
    g = oracle.Shape(4, 3, 5, 6, 2, 5, 6)
    assert (g.p, g.q) == (1, 1)
    x, dy = _rand(g, 7)
    dw, _ = oracle.dw_exact(x, dy, g)
    ref = np.einsum("nk,nchw->kchw", dy[:, :, 0, 0], x)
    np.testing.assert_allclose(dw, ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("g", GEOMS)
def test_against_torch_float64_weight_gradient(g):
    x, dy = _rand(g, 8)
    dw, _ = oracle.dw_exact(x, dy, g)
    ref = torch.nn.grad.conv2d_weight(torch.from_numpy(x), (g.k, g.c, g.r, g.s), torch.from_numpy(dy),
                                      stride=(g.stride_h, g.stride_w), padding=(g.pad_h, g.pad_w)).numpy()
    np.testing.assert_allclose(dw, ref, rtol=0, atol=1e-11)


def test_rejects_inconsistent_shape():
    with pytest.raises((ValueError, AssertionError)):
        oracle.dw_exact(np.zeros((1, 1, 2, 2)), np.zeros((1, 1, 1, 1)), oracle.Shape(1, 1, 2, 2, 1, 5, 5))
