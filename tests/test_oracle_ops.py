"""Pins for the oracle's ops: brute force, library special cases, closed forms, invariants and
central finite differences.  None of these re-types the oracle's own formula."""
import itertools

import numpy as np
import pytest

from oracle import ops

RNG = np.random.default_rng(7)


# ---- forward: brute force and library special cases -------------------------------------------
def conv_loops(x, w, bias, st, ph, pw):
    n, h, wd, cin = x.shape
    kh, kw, _, cout = w.shape
    ho, wo = (h + 2 * ph - kh) // st + 1, (wd + 2 * pw - kw) // st + 1
    y = np.zeros((n, ho, wo, cout))
    for b, i, j, co in itertools.product(range(n), range(ho), range(wo), range(cout)):
        acc = 0.0 if bias is None else bias[co]
        for r, s, ci in itertools.product(range(kh), range(kw), range(cin)):
            hi, wi = i * st - ph + r, j * st - pw + s
            if 0 <= hi < h and 0 <= wi < wd:
                acc += x[b, hi, wi, ci] * w[r, s, ci, co]
        y[b, i, j, co] = acc
    return y


@pytest.mark.parametrize("h,w,kh,kw,st,ph,pw", [(4, 4, 3, 3, 1, 1, 1), (5, 4, 3, 3, 2, 1, 1),
                                               (1, 9, 1, 5, 1, 0, 2), (3, 3, 1, 1, 1, 0, 0),
                                               (4, 5, 3, 3, 1, 0, 0)])
def test_conv_brute_force(h, w, kh, kw, st, ph, pw):
    x = RNG.standard_normal((2, h, w, 3))
    k = RNG.standard_normal((kh, kw, 3, 4))
    b = RNG.standard_normal(4)
    assert np.allclose(ops.conv_fwd(x, k, b, st, ph, pw), conv_loops(x, k, b, st, ph, pw), atol=1e-13)


def test_pointwise_is_matmul_and_conv1d_is_correlate():
    x = RNG.standard_normal((2, 3, 3, 5))
    k = RNG.standard_normal((1, 1, 5, 7))
    assert np.allclose(ops.conv_fwd(x, k, None, 1, 0, 0).reshape(-1, 7), x.reshape(-1, 5) @ k[0, 0])
    sig, ker = RNG.standard_normal(17), RNG.standard_normal(5)
    y = ops.conv_fwd(sig.reshape(1, 1, 17, 1), ker.reshape(1, 5, 1, 1), None, 1, 0, 2)
    assert np.allclose(y.reshape(-1), np.correlate(sig, ker, mode="same"))


def test_delta_kernel_shifts_and_depthwise_centre_is_identity():
    x = RNG.standard_normal((1, 5, 6, 2))
    k = np.zeros((3, 3, 2, 2))
    k[0, 2] = np.eye(2)          # tap (r=0, s=2): y[i,j] = x[i-1, j+1]
    y = ops.conv_fwd(x, k, None, 1, 1, 1)
    ref = np.zeros_like(x)
    ref[:, 1:, :-1] = x[:, :-1, 1:]
    assert np.array_equal(y, ref)
    kd = np.zeros((3, 3, 2))
    kd[1, 1] = 1.0
    assert np.array_equal(ops.dwconv_fwd(x, kd, 1, 1), x)
    assert np.array_equal(ops.dwconv_fwd(x, kd, 2, 1), x[:, ::2, ::2])


def test_depthwise_equals_block_diagonal_dense_conv():
    x = RNG.standard_normal((2, 5, 5, 3))
    kd = RNG.standard_normal((3, 3, 3))
    dense = np.zeros((3, 3, 3, 3))
    for c in range(3):
        dense[:, :, c, c] = kd[:, :, c]
    for st in (1, 2):
        assert np.allclose(ops.dwconv_fwd(x, kd, st, 1), conv_loops(x, dense, None, st, 1, 1))


def test_conv_linearity():
    x1, x2 = RNG.standard_normal((2, 1, 4, 4, 3))
    k1, k2 = RNG.standard_normal((2, 3, 3, 3, 2))
    f = lambda x, k: ops.conv_fwd(x, k, None, 2, 1, 1)
    assert np.allclose(f(2 * x1 - x2, k1), 2 * f(x1, k1) - f(x2, k1))
    assert np.allclose(f(x1, k1 + 3 * k2), f(x1, k1) + 3 * f(x1, k2))


def test_maxpool_gap_brute_force_and_tie_rule():
    x = RNG.standard_normal((2, 4, 6, 3))
    y, arg = ops.maxpool_fwd(x)
    for b, i, j, c in itertools.product(range(2), range(2), range(3), range(3)):
        assert y[b, i, j, c] == max(x[b, 2 * i + p, 2 * j + q, c] for p in (0, 1) for q in (0, 1))
    t = np.ones((1, 2, 2, 1))
    _, arg = ops.maxpool_fwd(t)
    assert arg.item() == 0                       # all equal: first in row-major window order
    assert np.array_equal(ops.maxpool_bwd(np.full((1, 1, 1, 1), 5.0), arg, t.shape).reshape(-1), [5, 0, 0, 0])
    assert np.allclose(ops.gap_fwd(x)[1, 0, 0, 2], sum(x[1, :, :, 2].reshape(-1)) / 24)
    assert np.allclose(ops.gap_bwd(np.ones((2, 1, 1, 3)), x.shape), 1 / 24)


# ---- closed forms ---------------------------------------------------------------------------
def test_softmax_ce_closed_forms():
    n, k = 6, 5
    labels = np.arange(n) % k
    loss, p = ops.softmax_ce_fwd(np.full((n, 1, 1, k), 3.7), labels)
    assert abs(loss - np.log(k)) < 1e-14
    z = RNG.standard_normal((n, 1, 1, k)) * 4
    loss, p = ops.softmax_ce_fwd(z, labels)
    e = np.exp(z.reshape(n, k))
    soft = e / e.sum(1, keepdims=True)
    assert np.allclose(p, soft) and np.isclose(loss, -np.mean(np.log(soft[np.arange(n), labels])))
    d = ops.softmax_ce_bwd(p, labels, z.shape).reshape(n, k)
    onehot = np.eye(k)[labels]
    assert np.allclose(d, (soft - onehot) / n) and np.allclose(d.sum(1), 0)
    big, _ = ops.softmax_ce_fwd(z + 1e4, labels)       # shift invariance, no overflow
    assert np.isclose(big, loss)


def test_bn_invariants():
    y = RNG.standard_normal((4, 3, 5, 6)) * 3 + 2
    g, b = RNG.standard_normal(6), RNG.standard_normal(6)
    eps = 1e-5
    z, mu, var, xhat = ops.bn_fwd(y, g, b, eps)
    assert np.allclose(mu, y.reshape(-1, 6).mean(0)) and np.allclose(var, y.reshape(-1, 6).var(0))
    zz = ops.bn_fwd(y, np.ones(6), np.zeros(6), eps)[0].reshape(-1, 6)
    assert np.allclose(zz.mean(0), 0, atol=1e-13) and np.allclose(zz.var(0), var / (var + eps))
    dz = RNG.standard_normal(y.shape)
    dy, dg, db = ops.bn_bwd(dz, xhat, g, var, eps)
    assert np.allclose(dy.sum((0, 1, 2)), 0, atol=1e-12)
    # sum dy*xhat vanishes up to the eps term: sum xhat^2 = M*var/(var+eps), not M
    resid = g / np.sqrt(var + eps) * dg * eps / (var + eps)
    assert np.allclose((dy * xhat).sum((0, 1, 2)), resid, atol=1e-11) and np.all(np.abs(resid) < 1e-4)
    assert np.allclose(db, dz.sum((0, 1, 2))) and np.allclose(dg, (dz * xhat).sum((0, 1, 2)))


def test_activation_kinks():
    z = np.array([-1.0, 0.0, 0.5, 6.0, 7.0])
    assert np.array_equal(ops.act_fwd(z, 1), [0, 0, 0.5, 6, 7])
    assert np.array_equal(ops.act_fwd(z, 2), [0, 0, 0.5, 6, 6])
    assert np.array_equal(ops.act_bwd(z, np.ones(5), 1), [0, 0, 1, 1, 1])
    assert np.array_equal(ops.act_bwd(z, np.ones(5), 2), [0, 0, 1, 0, 0])
    assert np.array_equal(ops.act_bwd(z, np.ones(5), 0), np.ones(5))


# ---- backward: central finite differences and the adjoint identity ----------------------------
def fd(f, x, h=1e-6):
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        old = x[i]
        x[i] = old + h
        fp = f()
        x[i] = old - h
        fm = f()
        x[i] = old
        g[i] = (fp - fm) / (2 * h)
    return g


@pytest.mark.parametrize("kh,kw,st,ph,pw", [(3, 3, 1, 1, 1), (3, 3, 2, 1, 1), (1, 5, 1, 0, 2), (1, 1, 1, 0, 0)])
def test_conv_backward_fd(kh, kw, st, ph, pw):
    x = RNG.standard_normal((2, 1 if kh == 1 else 5, 6, 3))
    w = RNG.standard_normal((kh, kw, 3, 2))
    b = RNG.standard_normal(2)
    r = RNG.standard_normal(ops.conv_fwd(x, w, b, st, ph, pw).shape)
    loss = lambda: (ops.conv_fwd(x, w, b, st, ph, pw) * r).sum()
    dx, dw, db = ops.conv_bwd(x, w, r, st, ph, pw, True)
    assert np.allclose(dx, fd(loss, x), atol=1e-7)
    assert np.allclose(dw, fd(loss, w), atol=1e-7)
    assert np.allclose(db, fd(loss, b), atol=1e-7)


@pytest.mark.parametrize("st", [1, 2])
def test_dwconv_backward_fd_and_adjoint(st):
    x = RNG.standard_normal((2, 5, 6, 3))
    w = RNG.standard_normal((3, 3, 3))
    r = RNG.standard_normal(ops.dwconv_fwd(x, w, st, 1).shape)
    loss = lambda: (ops.dwconv_fwd(x, w, st, 1) * r).sum()
    dx, dw = ops.dwconv_bwd(x, w, r, st, 1)
    assert np.allclose(dx, fd(loss, x), atol=1e-7) and np.allclose(dw, fd(loss, w), atol=1e-7)
    v = RNG.standard_normal(x.shape)          # <dy, J v> == <J^T dy, v>
    assert np.isclose((r * ops.dwconv_fwd(v, w, st, 1)).sum(), (dx * v).sum())


def test_bn_backward_fd():
    y = RNG.standard_normal((3, 2, 3, 4)) * 2 + 1
    g, b = RNG.standard_normal(4) + 2, RNG.standard_normal(4)
    r = RNG.standard_normal(y.shape)
    eps = 1e-5
    loss = lambda: (ops.bn_fwd(y, g, b, eps)[0] * r).sum()
    _, mu, var, xhat = ops.bn_fwd(y, g, b, eps)
    dy, dg, db = ops.bn_bwd(r, xhat, g, var, eps)
    assert np.allclose(dy, fd(loss, y), atol=1e-6)
    assert np.allclose(dg, fd(loss, g), atol=1e-7) and np.allclose(db, fd(loss, b), atol=1e-7)


def test_pool_ce_backward_fd():
    x = RNG.standard_normal((2, 4, 4, 3))
    r = RNG.standard_normal((2, 2, 2, 3))
    y, arg = ops.maxpool_fwd(x)
    assert np.allclose(ops.maxpool_bwd(r, arg, x.shape), fd(lambda: (ops.maxpool_fwd(x)[0] * r).sum(), x), atol=1e-7)
    r1 = RNG.standard_normal((2, 1, 1, 3))
    assert np.allclose(ops.gap_bwd(r1, x.shape), fd(lambda: (ops.gap_fwd(x) * r1).sum(), x), atol=1e-7)
    z = RNG.standard_normal((4, 1, 1, 5))
    lab = np.array([0, 4, 2, 2])
    _, p = ops.softmax_ce_fwd(z, lab)
    assert np.allclose(ops.softmax_ce_bwd(p, lab, z.shape), fd(lambda: ops.softmax_ce_fwd(z, lab)[0], z), atol=1e-8)
