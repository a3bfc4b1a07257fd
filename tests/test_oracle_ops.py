"""Pins for the oracle's operators: brute force, adjoint identities, closed forms, finite differences.

None of these tests re-types an oracle formula: each compares against an independently written
scalar loop, a mathematical identity, a library routine on a special case, or a stored value.
"""
import math
import os

import numpy as np
import pytest

from oracle import lp_oracle as O
from workloads import gen

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rnd(name, shape, seed=11):
    return gen.normal(seed, name, shape)


# -- (i) convolution: scatter-form brute force, written independently -----------------------
def conv_scatter(x, w, stride, pad):
    """Every input pixel pushes its contribution to the outputs it touches (scalar loops)."""
    n, h, wd, ci = x.shape
    co, R, S, _ = w.shape
    oh = (h + 2 * pad - R) // stride + 1
    ow = (wd + 2 * pad - S) // stride + 1
    y = np.zeros((n, oh, ow, co))
    for b in range(n):
        for ih in range(h):
            for iw in range(wd):
                for r in range(R):
                    for s in range(S):
                        th, tw = ih + pad - r, iw + pad - s
                        if th % stride or tw % stride:
                            continue
                        o_h, o_w = th // stride, tw // stride
                        if 0 <= o_h < oh and 0 <= o_w < ow:
                            for c in range(ci):
                                y[b, o_h, o_w, :] += x[b, ih, iw, c] * w[:, r, s, c]
    return y


CONV_CASES = [(3, 1, 1, 5, 6), (3, 2, 1, 6, 6), (1, 1, 0, 4, 5), (1, 2, 0, 6, 4), (7, 2, 3, 9, 10),
              (3, 2, 1, 5, 7)]


@pytest.mark.parametrize("R,stride,pad,h,w", CONV_CASES)
def test_conv_fwd_bruteforce(R, stride, pad, h, w):
    x = rnd("x", (2, h, w, 3))
    wt = rnd("w", (4, R, R, 3))
    np.testing.assert_allclose(O.conv_fwd(x, wt, stride, pad), conv_scatter(x, wt, stride, pad),
                               rtol=1e-12, atol=1e-12)


def test_conv_1x1_is_matmul_and_delta_is_identity():
    x = rnd("x", (2, 5, 4, 6))
    w = rnd("w", (3, 1, 1, 6))
    np.testing.assert_allclose(O.conv_fwd(x, w, 1, 0), (x.reshape(-1, 6) @ w.reshape(3, 6).T).reshape(2, 5, 4, 3),
                               rtol=1e-13, atol=1e-13)
    delta = np.zeros((6, 3, 3, 6))
    for c in range(6):
        delta[c, 1, 1, c] = 1.0
    np.testing.assert_array_equal(O.conv_fwd(x, delta, 1, 1), x)
    shift = np.zeros((6, 3, 3, 6))           # tap (0,2) reads x[h-1, w+1]
    for c in range(6):
        shift[c, 0, 2, c] = 1.0
    y = O.conv_fwd(x, shift, 1, 1)
    np.testing.assert_array_equal(y[:, 1:, :-1, :], x[:, :-1, 1:, :])
    assert np.all(y[:, 0, :, :] == 0) and np.all(y[:, :, -1, :] == 0)


@pytest.mark.parametrize("R,stride,pad,h,w", CONV_CASES)
def test_conv_adjoint_identities(R, stride, pad, h, w):
    """<conv(x,w), y> = <x, dgrad(y,w)> = <w, wgrad(x,y)> exactly (bilinearity)."""
    x = rnd("x", (2, h, w, 3))
    wt = rnd("w", (4, R, R, 3))
    y = O.conv_fwd(x, wt, stride, pad)
    dy = rnd("dy", y.shape)
    lhs = float((y * dy).sum())
    dx = O.conv_dgrad(dy, wt, stride, pad, x.shape)
    dw = O.conv_wgrad(x, dy, wt.shape, stride, pad)
    assert dx.shape == x.shape and dw.shape == wt.shape
    assert abs(lhs - float((x * dx).sum())) < 1e-10 * max(1, abs(lhs))
    assert abs(lhs - float((wt * dw).sum())) < 1e-10 * max(1, abs(lhs))


def test_conv_grads_elementwise_by_unit_vectors():
    """dgrad/wgrad entries equal <conv(e_i), dy>: pins every index, not only the inner product."""
    x = rnd("x", (1, 4, 5, 2))
    wt = rnd("w", (3, 3, 3, 2))
    for stride in (1, 2):
        y = O.conv_fwd(x, wt, stride, 1)
        dy = rnd("dy", y.shape)
        dx = O.conv_dgrad(dy, wt, stride, 1, x.shape)
        dw = O.conv_wgrad(x, dy, wt.shape, stride, 1)
        for idx in [(0, 0, 0, 0), (0, 3, 4, 1), (0, 2, 1, 0), (0, 1, 3, 1)]:
            e = np.zeros_like(x)
            e[idx] = 1.0
            assert abs(dx[idx] - (conv_scatter(e, wt, stride, 1) * dy).sum()) < 1e-12
        for idx in [(0, 0, 0, 0), (2, 2, 2, 1), (1, 0, 2, 0), (2, 1, 0, 1)]:
            e = np.zeros_like(wt)
            e[idx] = 1.0
            assert abs(dw[idx] - (conv_scatter(x, e, stride, 1) * dy).sum()) < 1e-12


# -- batch normalisation -----------------------------------------------------------------
def test_bn_forward_moments_and_affine():
    x = 3.0 + 2.0 * rnd("x", (4, 5, 6, 3))
    g = np.array([1.5, -0.5, 2.0])
    b = np.array([0.1, 0.2, -0.3])
    eps = 1e-5
    y, (xhat, rstd) = O.bn_fwd(x, g, b, eps)
    var = x.reshape(-1, 3).var(axis=0)          # numpy's biased variance
    np.testing.assert_allclose(xhat.reshape(-1, 3).mean(axis=0), 0, atol=1e-12)
    np.testing.assert_allclose(xhat.reshape(-1, 3).var(axis=0), var / (var + eps), rtol=1e-12)
    np.testing.assert_allclose(y, g * xhat + b, rtol=1e-13)
    np.testing.assert_allclose(rstd, 1 / np.sqrt(var + eps), rtol=1e-12)


def fd_grad(f, x, idxs, h=1e-6):
    out = []
    for idx in idxs:
        xp, xm = x.copy(), x.copy()
        xp[idx] += h
        xm[idx] -= h
        out.append((f(xp) - f(xm)) / (2 * h))
    return np.array(out)


def test_bn_backward_invariants_and_fd():
    x = rnd("x", (3, 4, 4, 2))
    g = np.array([1.3, 0.7])
    b = np.array([0.2, -0.1])
    dy = rnd("dy", x.shape)
    eps = 1e-5
    y, cache = O.bn_fwd(x, g, b, eps)
    dx, dg, db = O.bn_bwd(dy, cache, g)
    np.testing.assert_allclose(dx.reshape(-1, 2).sum(axis=0), 0, atol=1e-12)
    # sum(dx * xhat) = gamma*rstd*dgamma*eps/(var+eps): zero in the limit eps -> 0
    var = x.reshape(-1, 2).var(axis=0)
    np.testing.assert_allclose((dx * cache[0]).reshape(-1, 2).sum(axis=0),
                               g * cache[1] * dg * eps / (var + eps), rtol=1e-9, atol=1e-13)
    dx0, _, _ = O.bn_bwd(dy, O.bn_fwd(x, g, b, 0.0)[1], g)
    np.testing.assert_allclose((dx0 * O.bn_fwd(x, g, b, 0.0)[1][0]).reshape(-1, 2).sum(axis=0), 0, atol=1e-12)
    f = lambda xx: float((O.bn_fwd(xx, g, b, eps)[0] * dy).sum())
    idxs = [(0, 0, 0, 0), (2, 3, 1, 1), (1, 2, 2, 0)]
    np.testing.assert_allclose([dx[i] for i in idxs], fd_grad(f, x, idxs), rtol=1e-6, atol=1e-8)
    fg = lambda gg: float((O.bn_fwd(x, gg, b, eps)[0] * dy).sum())
    np.testing.assert_allclose(dg, fd_grad(fg, g, [(0,), (1,)]), rtol=1e-6)
    fb = lambda bb: float((O.bn_fwd(x, g, bb, eps)[0] * dy).sum())
    np.testing.assert_allclose(db, fd_grad(fb, b, [(0,), (1,)]), rtol=1e-6)


def test_conv_bn_scale_invariance():
    """BN(conv(x, a*w)) does not depend on a (eps -> 0), hence <w, dL/dw> = 0: pins wgrad with BN-bwd."""
    x = rnd("x", (3, 6, 6, 4))
    w = rnd("w", (5, 3, 3, 4))
    g, b = np.ones(5) * 1.2, np.zeros(5)
    dy = rnd("dy", (3, 6, 6, 5))
    y = O.conv_fwd(x, w, 1, 1)
    _, cache = O.bn_fwd(y, g, b, 0.0)
    dconv, _, _ = O.bn_bwd(dy, cache, g)
    dw = O.conv_wgrad(x, dconv, w.shape, 1, 1)
    for c in range(5):
        assert abs((w[c] * dw[c]).sum()) < 1e-10


# -- softmax cross-entropy -----------------------------------------------------------------
def test_ce_uniform_is_log_classes_golden():
    rows = [l.split() for l in open(os.path.join(GOLD, "log_classes.txt")) if not l.startswith("#")]
    for classes, value in rows:
        classes, value = int(classes), float(value)
        labels = gen.uniform_int(3, "lab", (7,), classes)
        loss, g = O.softmax_ce(np.zeros((7, classes)), labels)
        assert abs(loss - value) < 1e-12
        assert abs(value - math.log(classes)) < 1e-12


def test_ce_gradient_rows_sum_to_zero_and_fd():
    z = rnd("z", (5, 7))
    labels = gen.uniform_int(3, "lab", (5,), 7)
    loss, g = O.softmax_ce(z, labels)
    np.testing.assert_allclose(g.sum(axis=1), 0, atol=1e-14)
    # independent scalar evaluation
    ref = 0.0
    for i in range(5):
        ref += -(z[i, labels[i]] - math.log(sum(math.exp(v) for v in z[i])))
    assert abs(loss - ref / 5) < 1e-12
    f = lambda zz: O.softmax_ce(zz, labels)[0]
    idxs = [(0, 0), (1, int(labels[1])), (4, 6)]
    np.testing.assert_allclose([g[i] for i in idxs], fd_grad(f, z, idxs), rtol=1e-6, atol=1e-9)
    # large logits do not overflow
    big, _ = O.softmax_ce(z + 1000.0, labels)
    assert abs(big - loss) < 1e-9


# -- pooling ------------------------------------------------------------------------------
def test_maxpool_bruteforce_ties_and_mass():
    x = np.round(rnd("x", (2, 7, 6, 3)) * 2) / 2       # coarse values: ties do occur
    y, cache = O.maxpool_fwd(x)
    n, h, w, c = x.shape
    oh, ow = (h + 2 - 3) // 2 + 1, (w + 2 - 3) // 2 + 1
    assert y.shape == (n, oh, ow, c)
    dy = rnd("dy", y.shape)
    dx_ref = np.zeros_like(x)
    for b in range(n):
        for i in range(oh):
            for j in range(ow):
                for ch in range(c):
                    best, arg = -math.inf, None
                    for r in range(3):
                        for s in range(3):
                            ih, iw = 2 * i + r - 1, 2 * j + s - 1
                            if 0 <= ih < h and 0 <= iw < w and x[b, ih, iw, ch] > best:
                                best, arg = x[b, ih, iw, ch], (ih, iw)
                    assert y[b, i, j, ch] == best
                    dx_ref[b, arg[0], arg[1], ch] += dy[b, i, j, ch]
    dx = O.maxpool_bwd(dy, cache)
    np.testing.assert_allclose(dx, dx_ref, atol=1e-14)
    assert abs(dx.sum() - dy.sum()) < 1e-10


def test_avgpool_and_linear():
    x = rnd("x", (3, 4, 5, 2))
    p = O.avgpool_fwd(x)
    for b in range(3):
        for c in range(2):
            assert abs(p[b, c] - sum(x[b, i, j, c] for i in range(4) for j in range(5)) / 20) < 1e-13
    d = rnd("d", (3, 2))
    dx = O.avgpool_bwd(d, x.shape)
    assert abs((dx * x).sum() - (d * p).sum()) < 1e-12           # adjoint identity
    w, bias = rnd("w", (6, 2)), rnd("b", (6,))
    y = O.linear_fwd(p, w, bias)
    assert abs(y[1, 4] - (p[1, 0] * w[4, 0] + p[1, 1] * w[4, 1] + bias[4])) < 1e-13


def test_relu_zero_derivative_at_zero():
    x = np.array([-1.0, 0.0, 2.0])
    assert list(O.relu(x)) == [0.0, 0.0, 2.0]
    assert list(O.relu_bwd(np.ones(3), x)) == [0.0, 0.0, 1.0]


# -- local loss: stored hand computation -----------------------------------------------------
def test_local_loss_handmade_golden():
    vals = {}
    for line in open(os.path.join(GOLD, "local_loss_handmade.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        vals[k] = np.array([float(t) for t in v])
    out = np.array([1.0, -2.0, 0.5, 3.0])
    xn = np.array([0.5, -1.0, 0.5, 1.0])
    kap = np.array([0.2, -0.1, 0.4, 0.0])
    lp, rn2, r, sp = O.local_loss(out, xn, None, 0.5)
    la, _, _, sa = O.local_loss(out, xn, kap, 0.5)
    assert abs(rn2 - vals["rnorm2"][0]) < 1e-14
    assert abs(lp - vals["loss_penalty"][0]) < 1e-14
    assert abs(la - vals["loss_al"][0]) < 1e-14
    np.testing.assert_allclose(sp, vals["seed_penalty"], atol=1e-15)
    np.testing.assert_allclose(sa, vals["seed_al"], atol=1e-15)


def test_updates_closed_form():
    p = np.array([1.0, 2.0, -3.0])
    g = np.array([0.5, -1.0, 2.0])
    newp, v = O.sgd_update(p, g, 0.1)
    np.testing.assert_allclose(newp, [0.95, 2.1, -3.2], atol=1e-15)
    newp, v = O.sgd_update(p, g, 0.1, momentum=0.9, weight_decay=0.01)
    np.testing.assert_allclose(newp, p - 0.1 * (g + 0.01 * p), atol=1e-15)
    newp2, v2 = O.sgd_update(newp, g, 0.1, momentum=0.9, weight_decay=0.01, velocity=v)
    np.testing.assert_allclose(newp2, newp - 0.1 * (0.9 * v + g + 0.01 * newp), atol=1e-15)
    np.testing.assert_allclose(O.kappa_update(np.array([1.0, 0.0]), np.array([2.0, -1.0]), 0.5), [2.0, -0.5])
