"""Pins of the oracle's layer definitions against things other than itself."""
import itertools
import os

import numpy as np
import pytest

import oracle as O

rng = np.random.default_rng(7)
HERE = os.path.dirname(os.path.abspath(__file__))


# ---------------------------------------------------------------- brute force (Python loops)
def brute_conv(x, w, stride, pad):
    n, h, wd, c = x.shape
    k, kr, ks, _ = w.shape
    ho, wo = (h + 2 * pad - kr) // stride + 1, (wd + 2 * pad - ks) // stride + 1
    z = np.zeros((n, ho, wo, k))
    for b, i, j, o, r, s, ci in itertools.product(range(n), range(ho), range(wo), range(k),
                                                  range(kr), range(ks), range(c)):
        hi, wi = i * stride - pad + r, j * stride - pad + s
        if 0 <= hi < h and 0 <= wi < wd:
            z[b, i, j, o] += x[b, hi, wi, ci] * w[o, r, s, ci]
    return z


def brute_conv_grads(x, w, dz, stride, pad):
    n, h, wd, c = x.shape
    k, kr, ks, _ = w.shape
    _, ho, wo, _ = dz.shape
    dx, dw = np.zeros_like(x), np.zeros_like(w)
    for b, i, j, o, r, s, ci in itertools.product(range(n), range(ho), range(wo), range(k),
                                                  range(kr), range(ks), range(c)):
        hi, wi = i * stride - pad + r, j * stride - pad + s
        if 0 <= hi < h and 0 <= wi < wd:
            dx[b, hi, wi, ci] += dz[b, i, j, o] * w[o, r, s, ci]
            dw[o, r, s, ci] += dz[b, i, j, o] * x[b, hi, wi, ci]
    return dx, dw


CONV_CASES = [(2, 5, 6, 3, 4, 3, 1, 1), (1, 7, 5, 2, 3, 3, 2, 1), (2, 4, 4, 3, 2, 1, 1, 0),
              (1, 6, 7, 2, 2, 1, 2, 0), (1, 5, 5, 1, 2, 3, 1, 0), (1, 8, 8, 2, 2, 3, 2, 0)]


@pytest.mark.parametrize("n,h,w,c,k,ks,stride,pad", CONV_CASES)
def test_conv_matches_brute_force(n, h, w, c, k, ks, stride, pad):
    x = rng.standard_normal((n, h, w, c))
    wt = rng.standard_normal((k, ks, ks, c))
    z = O.conv2d_forward(x, wt, stride, pad)
    zb = brute_conv(x, wt, stride, pad)
    assert z.shape == zb.shape
    np.testing.assert_allclose(z, zb, rtol=0, atol=1e-12)
    dz = rng.standard_normal(z.shape)
    dx, dw = O.conv2d_backward(x, wt, dz, stride, pad)
    dxb, dwb = brute_conv_grads(x, wt, dz, stride, pad)
    np.testing.assert_allclose(dx, dxb, rtol=0, atol=1e-12)
    np.testing.assert_allclose(dw, dwb, rtol=0, atol=1e-12)


@pytest.mark.parametrize("stride", [1, 2])
def test_depthwise_is_dense_conv_with_diagonal_weights(stride):
    c = 5
    x = rng.standard_normal((2, 7, 6, c))
    wd = rng.standard_normal((c, 3, 3))
    dense = np.zeros((c, 3, 3, c))
    for ch in range(c):
        dense[ch, :, :, ch] = wd[ch]
    z = O.dwconv2d_forward(x, wd, stride, 1)
    np.testing.assert_allclose(z, brute_conv(x, dense, stride, 1), atol=1e-12)
    dz = rng.standard_normal(z.shape)
    dx, dw = O.dwconv2d_backward(x, wd, dz, stride, 1)
    dxb, dwb = brute_conv_grads(x, dense, dz, stride, 1)
    np.testing.assert_allclose(dx, dxb, atol=1e-12)
    np.testing.assert_allclose(dw, np.stack([dwb[ch, :, :, ch] for ch in range(c)]), atol=1e-12)


def test_pointwise_conv_is_a_matrix_product():
    x = rng.standard_normal((3, 4, 5, 6))
    w = rng.standard_normal((7, 1, 1, 6))
    z = O.conv2d_forward(x, w, 1, 0)
    ref = np.einsum("nhwc,kc->nhwk", x, w[:, 0, 0, :])
    np.testing.assert_allclose(z, ref, atol=1e-12)


def test_delta_kernel_shifts():
    x = rng.standard_normal((1, 6, 6, 1))
    for r, s in itertools.product(range(3), range(3)):
        w = np.zeros((1, 3, 3, 1))
        w[0, r, s, 0] = 1.0
        z = O.conv2d_forward(x, w, 1, 1)
        ref = np.zeros_like(x)
        for i, j in itertools.product(range(6), range(6)):
            hi, wi = i - 1 + r, j - 1 + s
            if 0 <= hi < 6 and 0 <= wi < 6:
                ref[0, i, j, 0] = x[0, hi, wi, 0]
        np.testing.assert_array_equal(z, ref)


@pytest.mark.parametrize("stride,pad,ks", [(1, 1, 3), (2, 1, 3), (2, 0, 1)])
def test_conv_adjoint_identity(stride, pad, ks):
    x = rng.standard_normal((2, 9, 8, 3))
    w = rng.standard_normal((4, ks, ks, 3))
    z = O.conv2d_forward(x, w, stride, pad)
    u = rng.standard_normal(z.shape)
    dx, dw = O.conv2d_backward(x, w, u, stride, pad)
    assert abs((z * u).sum() - (x * dx).sum()) < 1e-10 * abs((z * u).sum()) + 1e-10
    assert abs((z * u).sum() - (w * dw).sum()) < 1e-10 * abs((z * u).sum()) + 1e-10


# ---------------------------------------------------------------- finite differences
def fd_grad(f, a, h=1e-6):
    g = np.zeros_like(a)
    it = np.nditer(a, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        old = a[i]
        a[i] = old + h
        fp = f()
        a[i] = old - h
        fm = f()
        a[i] = old
        g[i] = (fp - fm) / (2 * h)
    return g


def assert_close_rel(a, b, tol=1e-6):
    scale = max(np.abs(b).max(), 1e-12)
    assert np.abs(a - b).max() / scale < tol, np.abs(a - b).max() / scale


def test_bn_forward_closed_forms():
    z = rng.standard_normal((3, 4, 5, 6)) * 3 + 2
    gamma, beta = rng.standard_normal(6), rng.standard_normal(6)
    y, (mu, var, xhat) = O.bn_forward(z, gamma, beta, 1e-5)
    np.testing.assert_allclose(y.mean(axis=(0, 1, 2)), beta, atol=1e-12)
    np.testing.assert_allclose(y.var(axis=(0, 1, 2)), gamma ** 2 * var / (var + 1e-5), rtol=1e-12)
    np.testing.assert_allclose(mu, z.reshape(-1, 6).mean(0), atol=1e-13)
    np.testing.assert_allclose(var, z.reshape(-1, 6).var(0), rtol=1e-12)    # numpy var: biased
    yc, _ = O.bn_forward(np.full((2, 3, 3, 6), 4.2), gamma, beta, 1e-5)
    np.testing.assert_allclose(yc, np.broadcast_to(beta, yc.shape), atol=1e-12)


def test_bn_backward_invariants_and_fd():
    z = rng.standard_normal((2, 3, 3, 4))
    gamma, beta = rng.standard_normal(4) + 1.5, rng.standard_normal(4)
    u = rng.standard_normal(z.shape)
    y, cache = O.bn_forward(z, gamma, beta, 1e-5)
    dz, dg, db = O.bn_backward(u, cache, gamma, 1e-5)
    np.testing.assert_allclose(dz.sum(axis=(0, 1, 2)), 0, atol=1e-12)
    # sum(xhat^2) = N var/(var+eps), hence sum(dz*xhat) = gamma/sqrt(var+eps) * dgamma * eps/(var+eps)
    var = cache[1]
    np.testing.assert_allclose((dz * cache[2]).sum(axis=(0, 1, 2)),
                               gamma / np.sqrt(var + 1e-5) * dg * 1e-5 / (var + 1e-5), atol=1e-12)
    f = lambda: (O.bn_forward(z, gamma, beta, 1e-5)[0] * u).sum()
    assert_close_rel(dz, fd_grad(f, z))
    assert_close_rel(dg, fd_grad(f, gamma))
    assert_close_rel(db, fd_grad(f, beta))


@pytest.mark.parametrize("kind", ["relu6", "relu"])
def test_activation_values_kinks_and_fd(kind):
    pre = np.array([-1.0, 0.0, 0.5, 5.999, 6.0, 7.5])
    y = O.act_forward(kind, pre)
    d = O.act_backward(kind, np.ones_like(pre), pre)
    if kind == "relu6":
        np.testing.assert_array_equal(y, [0, 0, 0.5, 5.999, 6, 6])
        np.testing.assert_array_equal(d, [0, 0, 1, 1, 0, 0])     # zero gradient exactly at both kinks
    else:
        np.testing.assert_array_equal(y, [0, 0, 0.5, 5.999, 6, 7.5])
        np.testing.assert_array_equal(d, [0, 0, 1, 1, 1, 1])
    a = rng.uniform(-3, 9, size=50)
    a = a[(np.abs(a) > 1e-3) & (np.abs(a - 6) > 1e-3)]
    f = lambda: O.act_forward(kind, a).sum()
    assert_close_rel(O.act_backward(kind, np.ones_like(a), a), fd_grad(f, a))


def test_conv_dw_linear_gap_fd():
    x = rng.standard_normal((2, 5, 4, 3))
    w = rng.standard_normal((2, 3, 3, 3))
    u = rng.standard_normal(O.conv2d_forward(x, w, 2, 1).shape)
    f = lambda: (O.conv2d_forward(x, w, 2, 1) * u).sum()
    dx, dw = O.conv2d_backward(x, w, u, 2, 1)
    assert_close_rel(dx, fd_grad(f, x)); assert_close_rel(dw, fd_grad(f, w))
    wd = rng.standard_normal((3, 3, 3))
    u = rng.standard_normal(O.dwconv2d_forward(x, wd, 2, 1).shape)
    f = lambda: (O.dwconv2d_forward(x, wd, 2, 1) * u).sum()
    dx, dw = O.dwconv2d_backward(x, wd, u, 2, 1)
    assert_close_rel(dx, fd_grad(f, x)); assert_close_rel(dw, fd_grad(f, wd))
    a = rng.standard_normal((3, 4)); W = rng.standard_normal((5, 4)); b = rng.standard_normal(5)
    u = rng.standard_normal((3, 5))
    f = lambda: (O.linear_forward(a, W, b) * u).sum()
    da, dW, db = O.linear_backward(a, W, u)
    assert_close_rel(da, fd_grad(f, a)); assert_close_rel(dW, fd_grad(f, W)); assert_close_rel(db, fd_grad(f, b))
    np.testing.assert_allclose(O.linear_forward(a, W, b), np.array([[W[j] @ a[n] + b[j] for j in range(5)] for n in range(3)]), atol=1e-13)
    g = O.gap_forward(x)
    np.testing.assert_allclose(g[:, 0, 0, :], x.reshape(2, -1, 3).mean(1), atol=1e-13)
    u = rng.standard_normal(g.shape)
    f = lambda: (O.gap_forward(x) * u).sum()
    assert_close_rel(O.gap_backward(u, 5, 4), fd_grad(f, x))


def test_mse_special_cases_and_fd():
    y = rng.standard_normal((2, 3, 3, 2))
    L, d = O.mse_loss(y, y.copy())
    assert L == 0 and not d.any()
    t = rng.standard_normal(y.shape)
    L, d = O.mse_loss(y, t)
    assert abs(L - sum((a - b) ** 2 for a, b in zip(y.ravel(), t.ravel())) / y.size) < 1e-13
    assert_close_rel(d, fd_grad(lambda: O.mse_loss(y, t)[0], y))


def test_softmax_xent_special_cases_and_fd():
    labels = np.array([3, 0, 999, 17])
    L, d = O.softmax_xent_loss(np.zeros((4, 1000)), labels)
    assert abs(L - np.log(1000)) < 1e-12
    logits = rng.standard_normal((4, 1000)) * 5
    L, d = O.softmax_xent_loss(logits, labels)
    np.testing.assert_allclose(d.sum(axis=1), 0, atol=1e-15)
    # shift invariance and no overflow for huge logits
    L2, d2 = O.softmax_xent_loss(logits + 1e4, labels)
    assert abs(L - L2) < 1e-9 and np.isfinite(d2).all()
    # a confident correct prediction has near-zero loss
    big = np.full((1, 10), -50.0); big[0, 4] = 50.0
    assert O.softmax_xent_loss(big, np.array([4]))[0] < 1e-12
    lg = rng.standard_normal((3, 7)); lb = np.array([1, 6, 0])
    assert_close_rel(O.softmax_xent_loss(lg, lb)[1], fd_grad(lambda: O.softmax_xent_loss(lg, lb)[0], lg))


def test_sgd_momentum_closed_forms():
    w = rng.standard_normal(10); g = rng.standard_normal(10)
    lr, mu, M = 0.01, 0.9, 4
    w1, v1 = O.sgd_momentum_step(w, np.zeros(10), g * M, M, lr, mu)
    np.testing.assert_allclose(w1, w - lr * g, atol=1e-15)             # first step from v=0
    w2, v2 = O.sgd_momentum_step(w1, v1, g * M, M, lr, mu)
    np.testing.assert_allclose(w2, w - lr * (2 + mu) * g, atol=1e-15)  # two steps, same gradient
    np.testing.assert_allclose(v2, (1 + mu) * g, atol=1e-15)


def test_warmup_forwards_matches_paper_example():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "warmup_forwards.txt")) if not l.startswith("#")]
    assert len(rows) == 3
    for P, p, k in rows:
        assert O.warmup_forwards(int(P), int(p)) == int(k)
    assert O.warmup_forwards(1, 0) == 1          # a single stage keeps one micro-batch resident
    assert O.stage_memory(10, 4, 7, 5) == 10 + 4 + 5 * 7      # Eq. (3)


def test_silu_values_and_fd():
    x = np.array([-30.0, -1.0, 0.0, 1.0, 30.0])
    y = O.act_forward("silu", x)
    assert abs(y[0]) < 1e-10 and y[2] == 0.0 and abs(y[4] - 30.0) < 1e-10
    assert np.allclose(y[[1, 3]], [-1.0 / (1.0 + np.e), 1.0 / (1.0 + 1.0 / np.e)], rtol=0, atol=1e-15)       # x * sigmoid(x) at -1 and 1
    assert np.allclose(O.act_forward("silu", x) - O.act_forward("silu", -x), x, rtol=0, atol=1e-12)           # silu(x) - silu(-x) = x
    rng = np.random.default_rng(3)
    pre = rng.normal(size=(2, 3, 3, 4)) * 3
    dy = rng.normal(size=pre.shape)
    g = fd_grad(lambda: float((O.act_forward("silu", pre) * dy).sum()), pre)
    assert_close_rel(O.act_backward("silu", dy, pre), g)
    assert O.act_backward("silu", np.ones(1), np.zeros(1))[0] == 0.5                                            # derivative at 0


def test_squeeze_excite_closed_forms_and_fd():
    rng = np.random.default_rng(4)
    n, h, w, c, k = 2, 3, 4, 5, 2
    x = rng.normal(size=(n, h, w, c))
    w1, b1, w2, b2 = rng.normal(size=(k, c)), rng.normal(size=k), rng.normal(size=(c, k)), rng.normal(size=c)
    out, cache = O.se_forward(x, w1, b1, w2, b2)
    # hand loop of the definition
    for nn in range(n):
        s = [sum(x[nn, i, j, cc] for i in range(h) for j in range(w)) / (h * w) for cc in range(c)]
        hid = []
        for q in range(k):
            p = sum(w1[q, cc] * s[cc] for cc in range(c)) + b1[q]
            hid.append(p / (1.0 + np.exp(-p)))
        for cc in range(c):
            p2 = sum(w2[cc, q] * hid[q] for q in range(k)) + b2[cc]
            g = 1.0 / (1.0 + np.exp(-p2))
            assert np.allclose(out[nn, :, :, cc], x[nn, :, :, cc] * g, rtol=0, atol=1e-14)
    # zero second-layer weights: the gate is sigmoid(b2), the same for every sample
    o0, _ = O.se_forward(x, w1, b1, np.zeros_like(w2), b2)
    assert np.allclose(o0, x * (1.0 / (1.0 + np.exp(-b2))), rtol=0, atol=1e-14)
    dout = rng.normal(size=out.shape)
    dx, dw1, db1, dw2, db2 = O.se_backward(x, w1, w2, cache, dout)
    L = lambda: float((O.se_forward(x, w1, b1, w2, b2)[0] * dout).sum())       # fd_grad perturbs its array in place
    for got, arr in ((dx, x), (dw1, w1), (db1, b1), (dw2, w2), (db2, b2)):
        assert_close_rel(got, fd_grad(L, arr))
