"""GPU parity of the bf16 path (bf16 activations and dense-convolution weights, float accumulation,
float master weights) against the oracle in its bf16 storage mode.  Tolerance: max-abs relative
error <= 2e-2 (helpers.TOL_BF16).

Both sides round to bf16 at the same points, so they differ only where float32 accumulation lands on
the other side of a bf16 rounding boundary than exact accumulation does (about 5e-4 of all stored
values, by one bf16 step).  Those single steps are far inside the tolerance for every continuous
quantity, but a few of them push a pre-activation across a ReLU kink, where the gradient jumps.
With K inputs per output about K * 5e-4 of the pre-activations move by ~1e-4 relative, so ~1e-4 of all
ReLU decisions (and more max-pool choices, where bf16 values tie within one step) differ, each changing
its gradient entry by 100 %: about 1 % L2 error per layer, inherent to bf16 storage.  Whole-network
tests therefore hold the continuous quantities (loss, logits, activations, running statistics) to the
max-abs tolerance and the gradients to GRAD_L2 in the L2 norm (a dropped term or a wrong sign gives
O(1)); the per-layer tests below zero the incoming gradient wherever the oracle sees an output within
reach of a kink and hold every gradient to the max-abs tolerance of 2e-2."""
import numpy as np
import pytest

import oracle
import synth
from helpers import TOL_BF16, perturb, rel_err

pytestmark = pytest.mark.gpu
GRAD_L2 = 0.1       # whole-network gradients, L2 norm (see the module docstring)
F = pytest.importorskip("paper_2110_02781_b200")


def dev_bf16(x):
    import torch
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda().to(torch.bfloat16)


def host(t):
    return t.float().cpu().numpy()


def l2_err(got, ref):
    got, ref = np.asarray(got, np.float64).reshape(-1), np.asarray(ref, np.float64).reshape(-1)
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)) if ref.size else 0.0


def step_case(net, idx, points, params="perturbed", max_stages=8):
    import torch
    from oracle.model import round_bf16
    ls, cfg = net
    assert cfg["precision"] == 1
    par = perturb(ls, idx) if params == "perturbed" else synth.init_params(idx, ls)
    om = oracle.OracleModel(ls, cfg, par, synth.init_state(ls))
    x, y = synth.make_batch(idx, cfg)
    x = round_bf16(x)                      # the device reads a bf16 batch
    gm = F.Model(ls, dict(cfg, max_stages=max_stages))
    gm.load_params(par, synth.init_state(ls))
    acts = [x]
    for a, b in zip(points[:-1], points[1:]):
        acts.append(om.forward(a, b, acts[-1], y if b == om.L else None))
    og = [None]
    for a, b in reversed(list(zip(points[:-1], points[1:]))):
        og.append(om.backward(a, b, og[-1]))
    og = og[::-1]
    xd, yd = dev_bf16(x), torch.from_numpy(y).cuda()
    L = gm.L
    gacts, ggrads = [xd], []
    loss = torch.zeros(1, device="cuda")
    for a, b in zip(points[:-1], points[1:]):
        if b == L:
            gm.ftp_run_stage_forward(a, b, gacts[-1], None, yd, loss)
        else:
            shp, _ = gm.ftp_unit_output_shape(b - 1)
            out = torch.empty(shp, dtype=torch.bfloat16, device="cuda")
            gm.ftp_run_stage_forward(a, b, gacts[-1], out)
            gacts.append(out)
    g = None
    for i in range(len(points) - 2, -1, -1):
        a, b = points[i], points[i + 1]
        gin = torch.empty_like(gacts[i]) if a > 0 else None
        gm.ftp_run_stage_backward(a, b, g, gin)
        ggrads.append(gin)
        g = gin
    ggrads = ggrads[::-1]
    torch.cuda.synchronize()
    assert abs(loss.item() - om.loss) <= TOL_BF16 * max(abs(om.loss), 1.0)
    assert rel_err(gm.ftp_get_logits(), om.logits) <= TOL_BF16
    for k in range(1, len(points) - 1):
        assert rel_err(host(gacts[k]), acts[k]) <= TOL_BF16, f"boundary activation {k}"
        assert l2_err(host(ggrads[k]), og[k]) <= GRAD_L2, f"boundary gradient {k}"
    for u in range(L):
        got, ref = gm.ftp_get_tensor(F.T_GRADS, u), om.unit_grads(u)
        assert l2_err(got, ref) <= GRAD_L2, f"weight gradient of unit {u}: {l2_err(got, ref):.3e} / {rel_err(got, ref):.3e}"
        assert rel_err(gm.ftp_get_tensor(F.T_STATE, u), om.unit_state(u)) <= TOL_BF16
    for a, b in zip(points[:-1], points[1:]):
        om.sgd(a, b, 0.01)
        gm.ftp_sgd_step(a, b, 0.01)
    for u in range(L):
        assert rel_err(gm.ftp_get_tensor(F.T_WEIGHTS, u), om.unit_params(u)) <= 1e-3      # master weights stay float
    gm.close()


def test_tiny_mobilenet_bf16_every_unit_a_stage():
    ls, cfg = synth.tiny_mbv2(precision=1)
    step_case((ls, cfg), 61, list(range(synth.num_units(ls) + 1)))


def test_stride_two_depthwise_rows_on_odd_maps_bf16():
    """The stride-2 depthwise kernels (with the batch norm in front of them folded in, the bf16 default) on 9 x 9 and 5 x 5 maps."""
    net = synth.mobilenetv2(3, 9, 7, 1, True, table=[(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 1, 2)], stem_c=32, last_c=64)
    step_case(net, 29, [0, 2, 4, 7])


def test_tiny_vgg_bf16_dense_3x3_and_maxpool():
    step_case(synth.tiny_vgg(batch=6, hw=4, precision=1), 62, [0, 1, 3])


def test_small_vgg_bf16_channels_of_the_real_net():
    """The first VGG groups at their real widths (64, 64, pool, 128, 128, pool, 128, pool) on 8x8 inputs, batch 32
    (the last BN still averages over 32 values)."""
    net = synth.vgg16(32, 8, 10, 1, plan=[64, 64, "M", 128, 128, "M", 128, "M"])
    step_case(net, 63, [0, 2, 4, 6], params="init")


def test_mobilenet_bf16_split_equals_unsplit_bitwise():
    import torch
    ls, cfg = synth.mobilenetv2(4, 16, 10, 1, True)
    a, b = F.Model(ls, cfg), F.Model(ls, cfg)
    for m in (a, b):
        m.load_params(synth.init_params(64, ls), synth.init_state(ls))
    b.ftp_set_partition([0, 6, 13, 20])
    x, y = synth.make_batch(64, cfg)
    xd, yd = dev_bf16(x), torch.from_numpy(y).cuda()
    for _ in range(2):
        assert a.ftp_train_step(xd, yd, 0.01) == b.ftp_train_step(xd, yd, 0.01)
    for u in range(a.L):
        for which in (F.T_WEIGHTS, F.T_GRADS, F.T_STATE, F.T_MOMENTUM):
            assert np.array_equal(a.ftp_get_tensor(which, u), b.ftp_get_tensor(which, u))


def full_size_case(net, idx, pts):
    """A benchmark network at (or near) its full size in the launch configuration the benchmark times.
    (i) Every unit on its own, fed the oracle's input of that unit: output against the oracle at the bf16 tolerance,
    element by element (what differs is single bf16 steps where float32 and exact accumulation round apart).
    (ii) The chained network: loss and BN running statistics at the tolerance; the logits only loosely, because a
    randomly initialised deep ReLU + BN network amplifies those single steps by about 1.7x per layer (measured on the
    VGG: 1e-5 after the first unit, 2e-2 after the thirteenth, with every unit correct to 2e-4 in isolation).
    (iii) The backward pass and update by what is unique at this size: the staged run equals the single-stage run
    bit for bit."""
    import torch
    from oracle.model import round_bf16
    ls, cfg = net
    om = oracle.OracleModel(ls, cfg, synth.init_params(idx, ls), synth.init_state(ls))
    x, y = synth.make_batch(idx, cfg)
    x = round_bf16(x)
    om.forward(0, om.L, x, y)
    probe, ref, alt = F.Model(ls, cfg), F.Model(ls, cfg), F.Model(ls, cfg)
    for m in (probe, ref, alt):
        m.load_params(synth.init_params(idx, ls), synth.init_state(ls))
    for u in range(probe.L - 1):
        ops = [i for i, l in enumerate(ls) if l.unit == u]
        unit_in = x if u == 0 else om.out[ops[0] - 1]
        shp, _ = probe.ftp_unit_output_shape(u)
        out = torch.empty(shp, dtype=torch.bfloat16, device="cuda")
        probe.ftp_run_stage_forward(u, u + 1, dev_bf16(unit_in), out)
        torch.cuda.synchronize()
        assert rel_err(host(out), om.out[ops[-1]]) <= TOL_BF16, f"unit {u} on the oracle's input"
        assert l2_err(host(out), om.out[ops[-1]]) <= 1e-3, f"unit {u} on the oracle's input (L2)"
    probe.close()
    alt.ftp_set_partition(pts)
    xd, yd = dev_bf16(x), torch.from_numpy(y).cuda()
    l0, l1 = ref.ftp_train_step(xd, yd, 0.01), alt.ftp_train_step(xd, yd, 0.01)
    assert l0 == l1 and abs(l0 - om.loss) <= TOL_BF16 * max(abs(om.loss), 1.0)
    assert l2_err(ref.ftp_get_logits(), om.logits) <= 5e-2
    for u in range(ref.L):
        assert rel_err(ref.ftp_get_tensor(F.T_STATE, u), om.unit_state(u)) <= TOL_BF16, f"running statistics of unit {u}"
        for which in (F.T_WEIGHTS, F.T_GRADS, F.T_MOMENTUM):
            assert np.array_equal(ref.ftp_get_tensor(which, u), alt.ftp_get_tensor(which, u)), f"unit {u}: the split changed a bit"
    ref.close(); alt.close()


def test_full_size_vgg16_batch_256():
    """Config 4 as benchmarked: VGG-16-style, 32 x 32 x 3, batch 256, 3 stages."""
    full_size_case(synth.vgg16(256, 32, 10, 1), 3, [0, 3, 8, 14])


def test_mobilenet_224_full_resolution():
    """Config 3's network at its full 224 x 224 resolution and 4 stages (every tile count and ragged edge of the
    benchmark's launches per image), at batch 8 of 64 to keep the float64 oracle's memory in bounds."""
    ls, cfg = synth.mobilenetv2(8, 224, 1000, 1, False)
    full_size_case((ls, dict(cfg, max_stages=5)), 2, [0, 1, 3, 7, 20])


# ---- one layer at a time: every gradient at the max-abs tolerance ------------------------------------------
LAYER_CASES = [  # kind, hw, cin, cout, k, stride, act, batch
    ("CONV2D", 16, 3, 32, 3, 2, 2, 8),        # MobileNetV2 stem (3 input channels, stride 2)
    ("CONV2D", 15, 3, 32, 3, 2, 2, 3),        # the same on an odd map (15 -> 8), pixel count not a multiple of 32
    ("CONV2D", 9, 3, 64, 3, 1, 1, 5),         # VGG stem (3 -> 64, stride 1), 405 pixels
    ("CONV2D", 16, 32, 96, 1, 1, 2, 16),      # pointwise expand
    ("CONV2D", 16, 96, 24, 1, 1, 0, 16),      # pointwise project (no activation)
    ("CONV2D", 7, 160, 960, 1, 1, 2, 8),      # late expand, odd map size
    ("DWCONV3x3", 16, 96, 96, 3, 1, 2, 8),
    ("DWCONV3x3", 16, 144, 144, 3, 2, 2, 8),
    ("CONV2D", 16, 64, 64, 3, 1, 1, 8),       # VGG dense 3x3
    ("CONV2D", 8, 128, 256, 3, 1, 1, 8),
    ("CONV2D", 4, 512, 512, 3, 1, 1, 16),
    # enough tiles for the persistent product (two or more per SM), a ragged last row tile and a last column tile of 16 columns
    ("CONV2D", 56, 24, 144, 1, 1, 2, 7),
    ("CONV2D", 28, 64, 96, 1, 1, 0, 50),
    ("CONV2D", 28, 96, 64, 1, 1, 0, 50),      # 64-wide tiles, two reduction blocks
]


@pytest.mark.parametrize("case", LAYER_CASES, ids=lambda c: "%s_hw%d_%dto%d_k%ds%d_act%d_b%d" % c)
def test_each_layer_kind_bf16(case):
    import torch
    from oracle.model import round_bf16
    kind, hw, cin, cout, k, stride, act, batch = case
    L, K = synth.Layer, synth.KIND
    pad = 1 if k == 3 else 0
    ho = (hw + 2 * pad - k) // stride + 1
    ls = [L(0, K[kind], cin, cout, k, stride, pad, 0, 0, -1), L(0, K["BN"], cout, cout, 0, 1, 0, act, 0, -1),
          L(1, K["GAP"], cout, cout, 0, 1, 0, 0, 0, -1), L(1, K["FC"], cout, 4, 1, 1, 0, 0, 1, -1),
          L(1, K["SOFTMAX_CE"], 4, 4, 0, 1, 0, 0, 0, -1)]
    cfg = synth.config(batch, cin, hw, hw, 4, precision=1, momentum=0.9, weight_decay=4e-5)
    g = synth.rng_stream(70, "misc")
    params = perturb(ls, 70)
    x = g.standard_normal((batch, hw, hw, cin)).astype(np.float32)
    if cin > 3:
        x = np.clip(x + 0.3, 0.0, 6.0)
    x = round_bf16(x)
    gout = round_bf16(g.standard_normal((batch, ho, ho, cout)) / (batch * ho * ho))
    om = oracle.OracleModel(ls, cfg, params, synth.init_state(ls))
    yref = om.forward(0, 1, x)
    gout[om.ambiguous_outputs(1, 2e-2)] = 0.0          # within two bf16 steps of a kink: the decision is not unique
    dxref = om.backward(0, 1, gout)
    gm = F.Model(ls, cfg)
    gm.load_params(params, synth.init_state(ls))
    y = torch.empty(yref.shape, dtype=torch.bfloat16, device="cuda")
    dx = torch.empty(x.shape, dtype=torch.bfloat16, device="cuda")
    xd, gd = dev_bf16(x), dev_bf16(gout)
    gm.ftp_run_stage_forward(0, 1, xd, y)
    gm.ftp_run_stage_backward(0, 1, gd, dx)
    torch.cuda.synchronize()
    assert rel_err(host(y), yref) <= TOL_BF16
    assert rel_err(host(dx), dxref) <= TOL_BF16
    got, ref = gm.ftp_get_tensor(F.T_GRADS, 0), om.unit_grads(0)
    nW = int(np.prod(synth.param_shapes(ls[0])[0]))
    for name, sl in (("dW", slice(0, nW)), ("dgamma", slice(nW, nW + cout)), ("dbeta", slice(nW + cout, nW + 2 * cout))):
        e = rel_err(got[sl], ref[sl])
        assert e <= TOL_BF16, f"{name}: {e:.3e}"
    assert rel_err(gm.ftp_get_tensor(F.T_STATE, 0), om.unit_state(0)) <= TOL_BF16
    gm.close()


# ---- the bf16 path against the plain float64 definition (no rounding anywhere in the oracle) ------------------
F64_NETS = {"tiny_mbv2": (lambda: synth.tiny_mbv2(precision=1), 66, "perturbed"),
            "tiny_mbv2_b16_hw16": (lambda: synth.tiny_mbv2(batch=16, hw=16, precision=1), 67, "init"),
            "tiny_vgg": (lambda: synth.tiny_vgg(batch=6, hw=4, precision=1), 68, "perturbed"),
            "vgg_real_widths": (lambda: synth.vgg16(32, 8, 10, 1, plan=[64, 64, "M", 128, 128, "M", 128, "M"]), 69, "init")}


@pytest.mark.parametrize("name", list(F64_NETS))
def test_bf16_path_against_the_float64_oracle(name, record_property):
    """One step of the bf16 device path from float32 master weights against the oracle with storage switched off:
    every tensor float64, nothing rounded anywhere.  The stated bar (2e-2, max-abs relative) is asserted on what is
    continuous in the stored values: the loss, the logits, the BN running statistics, the updated master weights.
    Weight gradients are measured in the same norm and printed, not asserted at 2e-2: storing activations and
    gradients with an 8-bit mantissa moves some pre-activations across a ReLU kink, and on these nets that alone puts
    15-20 % between ANY bf16-storage run and the float64 one (the oracle's own bf16 mode, run beside it here, shows
    the same figures).  What is asserted for them: the device is no further from float64 than bf16 storage itself is
    (the oracle's bf16 mode against its float64 mode, plus the 2e-2 bar)."""
    import torch
    from oracle.model import round_bf16
    net, idx, params = F64_NETS[name]
    ls, cfg = net()
    par = perturb(ls, idx) if params == "perturbed" else synth.init_params(idx, ls)
    om = oracle.OracleModel(ls, cfg, par, synth.init_state(ls), storage="none")
    oq = oracle.OracleModel(ls, cfg, par, synth.init_state(ls))
    assert not om.quantised and oq.quantised
    x, y = synth.make_batch(idx, cfg)
    x = round_bf16(x)                                  # all three read the same (bf16-representable) batch
    ref_loss = om.step([0, om.L], x, y, lr=0.01)
    oq.step([0, oq.L], x, y, lr=0.01)
    gm = F.Model(ls, cfg)
    gm.load_params(par, synth.init_state(ls))
    xd, yd = dev_bf16(x), torch.from_numpy(y).cuda()
    loss = torch.zeros(1, device="cuda")
    gm.ftp_run_stage_forward(0, gm.L, xd, None, yd, loss)
    gm.ftp_run_stage_backward(0, gm.L)
    torch.cuda.synchronize()
    e_loss = abs(loss.item() - ref_loss) / max(abs(ref_loss), 1e-30)
    e_logits = rel_err(gm.ftp_get_logits(), om.logits)
    units = [u for u in range(gm.L) if om.unit_grads(u).size]
    got = {u: gm.ftp_get_tensor(F.T_GRADS, u) for u in units}
    e_dev = {u: (rel_err(got[u], om.unit_grads(u)), l2_err(got[u], om.unit_grads(u))) for u in units}
    e_fmt = {u: (rel_err(oq.unit_grads(u), om.unit_grads(u)), l2_err(oq.unit_grads(u), om.unit_grads(u))) for u in units}
    e_state = max(rel_err(gm.ftp_get_tensor(F.T_STATE, u), om.unit_state(u)) for u in range(gm.L))
    gm.ftp_sgd_step(0, gm.L, 0.01)
    e_w = max(rel_err(gm.ftp_get_tensor(F.T_WEIGHTS, u), om.unit_params(u)) for u in range(gm.L))
    report = dict(loss=float(e_loss), logits=e_logits, state=e_state, weights=e_w,
                  grad_maxabs_device={u: round(v[0], 4) for u, v in e_dev.items()}, grad_maxabs_bf16_storage={u: round(v[0], 4) for u, v in e_fmt.items()},
                  grad_l2_device={u: round(v[1], 4) for u, v in e_dev.items()}, grad_l2_bf16_storage={u: round(v[1], 4) for u, v in e_fmt.items()})
    print(f"\nbf16 device path vs float64 oracle, {name}: {report}")
    record_property("bf16_vs_float64", str(report))
    assert e_loss <= TOL_BF16 and e_logits <= TOL_BF16 and e_state <= TOL_BF16 and e_w <= TOL_BF16, report
    for u in units:
        assert e_dev[u][0] <= e_fmt[u][0] + TOL_BF16 and e_dev[u][1] <= e_fmt[u][1] + TOL_BF16, (u, report)
    gm.close()


# ---- config 4 at its full size, one unit at a time, backward included: every gradient at the max-abs tolerance ------
def _vgg_units():
    ls, cfg = synth.vgg16(256, 32, 10, 1)
    return list(range(synth.num_units(ls) - 1))


@pytest.mark.parametrize("u", _vgg_units())
def test_full_size_vgg16_unit_forward_and_backward(u):
    """Unit u of the VGG-16-style network at batch 256 ([3x3 convolution, BN + ReLU] and, where the group closes, the
    2x2 max-pool), fed the input that unit has in the chained oracle run with the real initialisation, and a seeded
    incoming gradient that is zero wherever the oracle's decision is within bf16 reach of flipping (a pre-activation
    within 2e-2 of the ReLU kink, a pool window whose two largest values lie within 2e-2, a pool window that holds such
    a pre-activation).  What is compared is then unique: output, input gradient, dW, dgamma, dbeta, running statistics,
    each at 2e-2 max-abs."""
    import torch
    from oracle.model import round_bf16
    ls, cfg = synth.vgg16(256, 32, 10, 1)
    K = synth.KIND
    ops = [i for i, l in enumerate(ls) if l.unit == u]
    om = oracle.OracleModel(ls, cfg, synth.init_params(3, ls), synth.init_state(ls))
    x, y = synth.make_batch(3, cfg)
    act = round_bf16(x)
    for v in range(u):                                        # the chained run up to this unit (forward only)
        act = om.forward(v, v + 1, act)
    out = om.forward(u, u + 1, act)
    bn = next(i for i in ops if ls[i].kind == K["BN"])
    amb = om.ambiguous_outputs(bn, 2e-2)
    if ls[ops[-1]].kind == K["MAXPOOL2"]:
        n, h, w, c = amb.shape
        amb = amb.reshape(n, h // 2, 2, w // 2, 2, c).any(axis=(2, 4)) | om.ambiguous_outputs(ops[-1], 2e-2)
    g = synth.rng_stream(71 + u, "misc")
    gout = round_bf16(g.standard_normal(out.shape) / out[0].size)
    gout[amb] = 0.0
    dxref = om.backward(u, u + 1, gout)
    gm = F.Model(ls, cfg)
    gm.load_params(synth.init_params(3, ls), synth.init_state(ls))
    xd, gd = dev_bf16(act), dev_bf16(gout)
    yd = torch.empty(out.shape, dtype=torch.bfloat16, device="cuda")
    dxd = torch.empty(act.shape, dtype=torch.bfloat16, device="cuda")
    gm.ftp_run_stage_forward(u, u + 1, xd, yd)
    gm.ftp_run_stage_backward(u, u + 1, gd, dxd)
    torch.cuda.synchronize()
    assert rel_err(host(yd), out) <= TOL_BF16
    assert rel_err(host(dxd), dxref) <= TOL_BF16, f"input gradient: {rel_err(host(dxd), dxref):.3e}"
    got, ref = gm.ftp_get_tensor(F.T_GRADS, u), om.unit_grads(u)
    cout = ls[ops[0]].cout
    nW = ref.size - 2 * cout
    for name, sl in (("dW", slice(0, nW)), ("dgamma", slice(nW, nW + cout)), ("dbeta", slice(nW + cout, nW + 2 * cout))):
        e = rel_err(got[sl], ref[sl])
        assert e <= TOL_BF16, f"{name}: {e:.3e}"
    assert rel_err(gm.ftp_get_tensor(F.T_STATE, u), om.unit_state(u)) <= TOL_BF16
    gm.close()


def test_mobilenet_224_batch_64_first_units():
    """Config 3 at its full batch of 64: the first three units (first convolution, the expand-1 block, the first
    stride-2 block at 112 x 112), one at a time to keep the float64 oracle's memory in bounds, each fed the oracle's
    input of that unit: output and BN running statistics at the bf16 tolerance (max-abs) and 1e-3 in L2."""
    import gc
    import torch
    from oracle.model import round_bf16
    ls, cfg = synth.mobilenetv2(64, 224, 1000, 1, False)
    om = oracle.OracleModel(ls, cfg, synth.init_params(2, ls), synth.init_state(ls))
    gm = F.Model(ls, dict(cfg, max_stages=5))
    gm.load_params(synth.init_params(2, ls), synth.init_state(ls))
    x, _ = synth.make_batch(2, cfg)
    act = round_bf16(x)
    for u in range(3):
        ref = om.forward(u, u + 1, act)
        shp, _ = gm.ftp_unit_output_shape(u)
        out = torch.empty(shp, dtype=torch.bfloat16, device="cuda")
        xd = dev_bf16(act)
        gm.ftp_run_stage_forward(u, u + 1, xd, out)
        torch.cuda.synchronize()
        got = host(out)
        assert rel_err(got, ref) <= TOL_BF16, f"unit {u}"
        assert l2_err(got, ref) <= 1e-3, f"unit {u} (L2)"
        assert rel_err(gm.ftp_get_tensor(F.T_STATE, u), om.unit_state(u)) <= TOL_BF16, f"running statistics of unit {u}"
        act = ref
        om.out.clear(); om.saved.clear()
        del got, out, xd
        gc.collect()
    gm.close()
