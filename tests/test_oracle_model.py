"""Pins for the oracle's model driver: whole-network finite differences, stage split equals the
unsplit run, SGD closed forms, an independent float64 autograd cross-check, snapshot layout."""
import numpy as np
import pytest

import oracle
import synth


def build(net, idx=9, **kw):
    ls, cfg = net(**kw)
    return ls, cfg, oracle.OracleModel(ls, cfg, synth.init_params(idx, ls), synth.init_state(ls))


def loss_of(m, x, y):
    keep = [[a.copy() for a in s] for s in m.s]
    v = m.forward(0, m.L, x, y)
    m.s = keep
    return float(v)


@pytest.mark.parametrize("net", [synth.tiny_mbv2, synth.tiny_vgg, lambda: synth.har_cnn(3, 2, 12, 4, 3)])
def test_whole_network_gradients_by_finite_differences(net):
    ls, cfg, m = build(net)
    rng = np.random.default_rng(3)
    for arrs in m.p:                       # move off the symmetric init (beta 0, bias 0)
        for a in arrs:
            a += 0.1 * rng.standard_normal(a.shape)
    x, y = synth.make_batch(9, cfg)
    x = x.astype(np.float64)
    m.forward(0, m.L, x, y)
    m.backward(0, m.L)
    h, checked = 1e-6, 0
    for i, arrs in enumerate(m.p):
        for k, a in enumerate(arrs):
            flat = a.reshape(-1)
            for j in rng.choice(flat.size, size=min(3, flat.size), replace=False):
                old = flat[j]
                flat[j] = old + h
                fp = loss_of(m, x, y)
                flat[j] = old - h
                fm = loss_of(m, x, y)
                flat[j] = old
                num = (fp - fm) / (2 * h)
                ana = m.g[i][k].reshape(-1)[j]
                assert abs(num - ana) <= 1e-6 + 1e-4 * abs(ana), (i, k, j, num, ana)
                checked += 1
    assert checked > 20


@pytest.mark.parametrize("net", [synth.tiny_mbv2, synth.tiny_vgg, synth.har_cnn])
def test_split_equals_unsplit_exactly(net):
    ls, cfg, ref = build(net)
    x, y = synth.make_batch(9, cfg)
    L = ref.L
    ref.step([0, L], x, y)
    ref.step([0, L], x, y)
    for pts in ([0, 1, L], [0, 2, L], [0, L - 1, L], [0, 1, 2, L], list(range(L + 1))):
        _, _, m = build(net)
        m.step(pts, x, y)
        m.step(pts, x, y)
        assert m.loss == ref.loss
        for u in range(L):
            assert np.array_equal(m.unit_params(u), ref.unit_params(u))
            assert np.array_equal(m.unit_grads(u), ref.unit_grads(u))
            assert np.array_equal(m.unit_state(u), ref.unit_state(u))


def test_boundary_tensors_of_a_split_run():
    ls, cfg, m = build(synth.tiny_mbv2)
    x, y = synth.make_batch(9, cfg)
    act = m.forward(0, 3, x)
    assert act.shape[0] == cfg["batch"] and act.ndim == 4
    m.forward(3, m.L, act, y)
    g = m.backward(3, m.L)
    assert g.shape == act.shape                 # boundary gradient is shaped like the boundary activation
    assert m.backward(0, 3, g).shape == x.shape


def test_sgd_closed_forms():
    ls, cfg = synth.har_cnn(2, 1, 4, 1, 2)
    cfg.update(lr=0.5, momentum=0.9, weight_decay=0.1)
    m = oracle.OracleModel(ls, cfg, synth.init_params(1, ls), synth.init_state(ls))
    w0 = m.p[0][0].copy()
    g = np.full_like(w0, 2.0)
    m.g[0][0] = g.copy()
    m.sgd(0, 1)                                  # first step: buffer = g + wd*w
    m1 = g + 0.1 * w0
    w1 = w0 - 0.5 * m1
    assert np.allclose(m.p[0][0], w1)
    m.g[0][0] = g.copy()
    m.sgd(0, 1)
    m2 = 0.9 * m1 + (g + 0.1 * w1)
    assert np.allclose(m.p[0][0], w1 - 0.5 * m2)
    cfg.update(momentum=0.0, weight_decay=0.0)   # reduces to w - lr*g
    m = oracle.OracleModel(ls, cfg, synth.init_params(1, ls), synth.init_state(ls))
    m.g[0][0] = g.copy()
    m.sgd(0, 1, lr=0.25)
    assert np.allclose(m.p[0][0], w0 - 0.25 * g)
    assert np.array_equal(m.p[1][0], synth.init_params(1, ls)[1][0])   # units outside [a,b) untouched


def _torch_reference(ls, cfg, params, x, y):
    """The same network through torch's float64 CPU autograd: a library cross-check."""
    import torch
    import torch.nn.functional as F
    K = synth.KIND
    ps = [[torch.tensor(np.asarray(a, np.float64), requires_grad=True) for a in arrs] for arrs in params]
    outs = {-1: torch.tensor(x.astype(np.float64)).permute(0, 3, 1, 2)}
    for i, l in enumerate(ls):
        t = outs[i - 1]
        if l.kind in (K["CONV1D"], K["CONV2D"], K["FC"]):
            w = ps[i][0].permute(3, 2, 0, 1)
            pad = (0, l.pad) if l.kind == K["CONV1D"] else (l.pad, l.pad)
            t = F.conv2d(t, w, ps[i][1] if l.has_bias else None, stride=l.stride, padding=pad)
        elif l.kind == K["DWCONV3x3"]:
            t = F.conv2d(t, ps[i][0].permute(2, 0, 1).unsqueeze(1), None, stride=l.stride, padding=1, groups=l.cin)
        elif l.kind == K["BN"]:
            t = F.batch_norm(t, None, None, ps[i][0], ps[i][1], training=True, eps=cfg["bn_eps"])
        elif l.kind == K["ADD_RESIDUAL"]:
            t = t + outs[l.residual_src]
        elif l.kind == K["MAXPOOL2"]:
            t = F.max_pool2d(t, 2)
        elif l.kind == K["GAP"]:
            t = t.mean((2, 3), keepdim=True)
        elif l.kind == K["SOFTMAX_CE"]:
            t = F.cross_entropy(t.flatten(1), torch.tensor(y, dtype=torch.long))
        if l.kind != K["SOFTMAX_CE"]:
            t = F.relu(t) if l.act == 1 else (F.relu6(t) if l.act == 2 else t)
        outs[i] = t
    outs[len(ls) - 1].backward()
    return float(outs[len(ls) - 1].detach()), [[p.grad.numpy() for p in arrs] for arrs in ps]


@pytest.mark.parametrize("net", [synth.tiny_mbv2, synth.tiny_vgg, synth.har_cnn])
def test_against_float64_autograd(net):
    ls, cfg, m = build(net)
    x, y = synth.make_batch(9, cfg)
    m.forward(0, m.L, x, y)
    m.backward(0, m.L)
    loss, grads = _torch_reference(ls, cfg, synth.init_params(9, ls), x, y)
    assert abs(loss - m.loss) < 1e-12
    for i, arrs in enumerate(grads):
        for k, g in enumerate(arrs):
            assert np.allclose(m.g[i][k], g, rtol=1e-9, atol=1e-12), (i, k)


def test_bn_running_statistics_use_unbiased_variance():
    ls, cfg, m = build(synth.tiny_vgg)
    x, y = synth.make_batch(9, cfg)
    m.forward(0, 1, x)
    conv = m.out[0].reshape(-1, 8)
    assert np.allclose(m.s[1][0], 0.1 * conv.mean(0))
    assert np.allclose(m.s[1][1], 0.9 + 0.1 * conv.var(0, ddof=1))


def test_snapshot_layout():
    ls, cfg, m = build(synth.tiny_vgg)
    snap = m.snapshot(0, m.L)
    n_par = sum(int(np.prod(s)) for l in ls for s in synth.param_shapes(l))
    n_st = sum(int(np.prod(s)) for l in ls for s in synth.state_shapes(l))
    assert snap.dtype == np.float32 and snap.size == n_par + n_st
    u0 = synth.flat_unit_params(ls, synth.init_params(9, ls), 0)
    assert np.array_equal(snap[:u0.size], u0)
    assert np.array_equal(np.concatenate([m.snapshot(0, 1), m.snapshot(1, m.L)]), snap)


# ---- the bf16 storage mode of the oracle (configs 3-5 fix bf16 activations and weights) ----------------
def test_bf16_rounding_matches_the_library_conversion():
    import torch
    from oracle.model import round_bf16
    rng = np.random.default_rng(0)
    x = rng.standard_normal(200000) * 10.0 ** rng.uniform(-6, 6, 200000)
    ref = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(round_bf16(x), ref)
    ties = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -1.0 - 2.0 ** -8])      # halfway cases go to even
    assert np.array_equal(round_bf16(ties), [1.0, 1.0 + 2.0 ** -6, -1.0])


@pytest.mark.parametrize("net", [synth.tiny_mbv2, synth.tiny_vgg])
def test_bf16_storage_mode(net):
    from oracle.model import round_bf16
    ls, cfg = net(precision=1)
    x, y = synth.make_batch(9, cfg)
    x = round_bf16(x)
    q = oracle.OracleModel(ls, cfg, synth.init_params(9, ls), synth.init_state(ls))
    f = oracle.OracleModel(ls, dict(cfg, precision=0), synth.init_params(9, ls), synth.init_state(ls))
    assert q.quantised and not f.quantised
    lq, lf = q.step([0, q.L], x, y), f.step([0, f.L], x, y)
    assert abs(lq - lf) < 2e-2 * abs(lf) and lq != lf              # close to, but not, the float64 run
    for i, l in enumerate(ls):                                     # what is stored is representable in bf16
        if l.kind not in (synth.KIND["FC"], synth.KIND["SOFTMAX_CE"]) and \
                not (i + 1 < len(ls) and ls[i + 1].kind == synth.KIND["ADD_RESIDUAL"]):
            assert np.array_equal(q.out[i], round_bf16(q.out[i])), i
    s = oracle.OracleModel(ls, cfg, synth.init_params(9, ls), synth.init_state(ls))   # split == unsplit still holds
    assert s.step([0, 1, q.L - 1, q.L], x, y) == lq
    for u in range(q.L):
        assert np.array_equal(s.unit_params(u), q.unit_params(u))


# ---- where the bf16 storage mode rounds: one constructed input per rounding point, expected values by hand ----
def _tail(unit, c, classes=2):
    L, K = synth.Layer, synth.KIND
    return [L(unit, K["GAP"], c, c, 0, 1, 0, 0, 0, -1), L(unit, K["FC"], c, classes, 1, 1, 0, 0, 1, -1),
            L(unit, K["SOFTMAX_CE"], classes, classes, 0, 1, 0, 0, 0, -1)]


def test_bf16_mode_rounds_a_convolution_output_to_nearest_even():
    """1 x 1 convolution, one channel: x = 1.5, w = 1 + 2^-7 (both bf16 numbers).  The exact product
    1.5 + 2^-7 + 2^-8 = 1.51171875 lies midway between the bf16 neighbours 1.5078125 (odd mantissa) and 1.515625 (even):
    stored 1.515625.  With w = 1 + 2^-7 + 2^-9 in the master copy the weight is first used as bf16 (rounds to
    1 + 2^-7): same stored output; the float64 mode keeps 1.5146484375."""
    L, K = synth.Layer, synth.KIND
    ls = [L(0, K["CONV2D"], 1, 1, 1, 1, 0, 0, 0, -1)] + _tail(1, 1)
    cfg = synth.config(1, 1, 1, 1, 2, precision=1)
    x = np.full((1, 1, 1, 1), 1.5)
    for w, exact in ((1 + 2.0 ** -7, 1.51171875), (1 + 2.0 ** -7 + 2.0 ** -9, 1.5146484375)):
        par = [[np.full((1, 1, 1, 1), w)], [], [np.zeros((1, 1, 1, 2)), np.zeros(2)], []]
        q = oracle.OracleModel(ls, cfg, par, synth.init_state(ls))
        assert q.forward(0, 1, x)[0, 0, 0, 0] == 1.515625
        f = oracle.OracleModel(ls, cfg, par, synth.init_state(ls), storage="none")
        assert f.forward(0, 1, x)[0, 0, 0, 0] == exact


def _bn_add_net():
    """[BN (no activation), residual add of the stage input] on a batch of four 1 x 1 x 1 samples x = (-a, a, -a, a),
    a = 2^-10, eps = 0: mean 0, variance a^2, xhat = (-1, 1, -1, 1) exactly, gamma / sigma = 256 for gamma = 0.25."""
    L, K = synth.Layer, synth.KIND
    ls = [L(0, K["BN"], 1, 1, 0, 1, 0, 0, 0, -1), L(0, K["ADD_RESIDUAL"], 1, 1, 0, 1, 0, 0, 0, -1)] + _tail(1, 1)
    cfg = synth.config(4, 1, 1, 1, 2, precision=1, bn_eps=0.0)
    a = 2.0 ** -10
    x = np.array([-a, a, -a, a]).reshape(4, 1, 1, 1)
    return ls, cfg, x


def test_bf16_mode_rounds_bn_plus_residual_once():
    """gamma = 0.25, beta = 1.25439453125: z_0 = beta - gamma = 1 + 2^-8 + 2^-11, just above the tie between 1 and
    1 + 2^-7.  Rounded once, after the add: z_0 + x_0 = 1 + 2^-8 - 2^-11 -> 1.0.  Rounding z first would give
    1.0078125 - 2^-10 -> 1.0078125."""
    ls, cfg, x = _bn_add_net()
    par = [[np.array([0.25]), np.array([1.25439453125])], [], [], [np.zeros((1, 1, 1, 2)), np.zeros(2)], []]
    q = oracle.OracleModel(ls, cfg, par, synth.init_state(ls))
    out = q.forward(0, 1, x).reshape(-1)
    assert out[0] == 1.0
    from oracle.model import round_bf16
    assert round_bf16(round_bf16(np.array([1.00439453125])) + x.reshape(-1)[:1])[0] == 1.0078125     # what "twice" would store
    assert out[1] == round_bf16(np.array([1.50439453125 + 2.0 ** -10]))[0]


def test_bf16_mode_rounds_a_gradient_with_two_contributions_after_the_sum():
    """Same net; incoming gradient d = (0.6875, 0, 9 * 2^-12, 0) (bf16 numbers).  The stage input receives d through
    the residual and 256 * (d - mean(d) - xhat * mean(d * xhat)) through the BN: for sample 0 that is
    128 * (d_0 - d_2) = 87.71875.  Stored once, after the sum: 0.6875 + 87.71875 = 88.40625 -> 88.5.  Rounding the
    BN contribution first (87.5) and then the sum (88.1875) would give 88.0."""
    ls, cfg, x = _bn_add_net()
    par = [[np.array([0.25]), np.array([1.0])], [], [], [np.zeros((1, 1, 1, 2)), np.zeros(2)], []]
    q = oracle.OracleModel(ls, cfg, par, synth.init_state(ls))
    q.forward(0, 1, x)
    d = np.array([0.6875, 0.0, 9 * 2.0 ** -12, 0.0]).reshape(4, 1, 1, 1)
    g = q.backward(0, 1, d).reshape(-1)
    assert g[0] == 88.5
    from oracle.model import round_bf16
    assert round_bf16(np.array([0.6875 + round_bf16(np.array([87.71875]))[0]]))[0] == 88.0
    # the BN's own parameter gradients are not stored in bf16: dgamma = sum d * xhat, dbeta = sum d, exactly
    assert q.g[0][0][0] == -(0.6875 + 9 * 2.0 ** -12) and q.g[0][1][0] == 0.6875 + 9 * 2.0 ** -12
