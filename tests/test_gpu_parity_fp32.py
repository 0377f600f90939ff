"""GPU parity of the fp32 path against the float64 oracle, through the C ABI.
Tolerance: max-abs relative error <= 1e-4 per tensor (helpers.TOL_FP32); integer / byte results exact."""
import numpy as np
import pytest

import synth
from helpers import (TOL_FP32, gpu_step_split, make_gpu, make_oracle, perturb, rel_err, to_dev)

pytestmark = pytest.mark.gpu
F = pytest.importorskip("paper_2110_02781_b200")


def unit_arrays(m, which):
    return [m.ftp_get_tensor(which, u) for u in range(m.L)]


def compare_units(gm, om, what, tol=TOL_FP32):
    worst = 0.0
    for u in range(gm.L):
        if what == "grads":
            got, ref = gm.ftp_get_tensor(F.T_GRADS, u), om.unit_grads(u)
        elif what == "weights":
            got, ref = gm.ftp_get_tensor(F.T_WEIGHTS, u), om.unit_params(u)
        else:
            got, ref = gm.ftp_get_tensor(F.T_STATE, u), om.unit_state(u)
        e = rel_err(got, ref)
        assert e <= tol, f"{what} of unit {u}: relative error {e:.3e} > {tol}"
        worst = max(worst, e)
    return worst


def one_step_case(net, idx, points, lr=0.01, perturbed=True, max_stages=5):
    ls, cfg = net
    params = perturb(ls, idx) if perturbed else synth.init_params(idx, ls)
    import oracle
    om = oracle.OracleModel(ls, cfg, params, synth.init_state(ls))
    gm = F.Model(ls, dict(cfg, max_stages=max_stages))
    gm.load_params(params, synth.init_state(ls))
    x, y = synth.make_batch(idx, cfg)
    xd, yd = to_dev(x), to_dev(y)
    # forward + backward only first: gradients
    acts = [x]
    for a, b in zip(points[:-1], points[1:]):
        acts.append(om.forward(a, b, acts[-1], y if b == om.L else None))
    ograds = [None]
    for a, b in reversed(list(zip(points[:-1], points[1:]))):
        ograds.append(om.backward(a, b, ograds[-1]))
    for a, b in zip(points[:-1], points[1:]):
        om.sgd(a, b, lr)
    loss, gacts, ggrads = gpu_step_split(gm, points, xd, yd, lr)
    assert abs(loss - om.loss) <= TOL_FP32 * max(abs(om.loss), 1.0)
    assert rel_err(gm.ftp_get_logits(), om.logits) <= TOL_FP32
    for k in range(1, len(points) - 1):                           # boundary activations and gradients
        assert rel_err(gacts[k].cpu().numpy(), acts[k]) <= TOL_FP32
        assert rel_err(ggrads[k].cpu().numpy(), ograds[len(points) - 1 - k]) <= TOL_FP32
    compare_units(gm, om, "grads")
    compare_units(gm, om, "weights")
    compare_units(gm, om, "state")
    gm.close()


def test_tiny_mobilenet_one_step_every_unit_is_a_stage():
    ls, cfg = synth.tiny_mbv2()
    one_step_case((ls, cfg), 21, list(range(synth.num_units(ls) + 1)), max_stages=8)


def test_tiny_vgg_with_maxpool():
    net = synth.tiny_vgg(batch=6, hw=8)
    one_step_case(net, 22, [0, 1, 3])


def test_har_cnn_ten_iterations_split_after_layer_two():
    """Config 1: batch 32 x 9 x 128, three conv1d(k5, 64)+ReLU, pool, FC, plain SGD lr 0.01, 10 iterations."""
    ls, cfg = synth.har_cnn()
    om = make_oracle(ls, cfg, 0)
    gm = make_gpu(ls, cfg, 0)
    pts = [0, 2, 5]
    gm.ftp_set_partition(pts)
    for it in range(10):
        x, y = synth.make_batch(0, cfg, it)
        ref = om.step(pts, x, y)
        got = gm.ftp_train_step(to_dev(x), to_dev(y), cfg["lr"])
        assert abs(got - ref) <= TOL_FP32 * abs(ref), (it, got, ref)
        assert rel_err(gm.ftp_get_logits(), om.logits) <= TOL_FP32
        compare_units(gm, om, "grads")
    compare_units(gm, om, "weights")
    gm.close()


@pytest.mark.parametrize("pts", [[0, 5], [0, 3, 5], [0, 1, 2, 3, 4, 5]])
def test_split_equals_unsplit_bitwise_on_the_gpu(pts):
    """Every reduction has a fixed order, so grouping units into stages changes no bit."""
    ls, cfg = synth.har_cnn()
    ref, alt = make_gpu(ls, cfg, 0), make_gpu(ls, cfg, 0)
    alt.ftp_set_partition(pts)
    for it in range(3):
        x, y = synth.make_batch(0, cfg, it)
        xd, yd = to_dev(x), to_dev(y)
        l0 = ref.ftp_train_step(xd, yd, 0.01)
        l1, _, _ = gpu_step_split(alt, pts, xd, yd, 0.01)
        assert l0 == l1
    for u in range(ref.L):
        assert np.array_equal(ref.ftp_get_tensor(F.T_WEIGHTS, u), alt.ftp_get_tensor(F.T_WEIGHTS, u))
        assert np.array_equal(ref.ftp_get_tensor(F.T_GRADS, u), alt.ftp_get_tensor(F.T_GRADS, u))


def test_mobilenet_split_equals_unsplit_bitwise_with_momentum():
    ls, cfg = synth.mobilenetv2(8, 16, 10, 0, True)
    ref, alt = make_gpu(ls, cfg, 3), make_gpu(ls, cfg, 3)
    pts = [0, 4, 11, 20]
    alt.ftp_set_partition(pts)
    x, y = synth.make_batch(3, cfg)
    xd, yd = to_dev(x), to_dev(y)
    for it in range(2):
        assert ref.ftp_train_step(xd, yd, 0.01) == gpu_step_split(alt, pts, xd, yd, 0.01)[0]
    for u in range(ref.L):
        for which in (F.T_WEIGHTS, F.T_GRADS, F.T_STATE, F.T_MOMENTUM):
            assert np.array_equal(ref.ftp_get_tensor(which, u), alt.ftp_get_tensor(which, u))


def test_mobilenet_cifar_several_tiles_and_ragged_tail():
    """MobileNetV2 32x32 at batch 6: M = 6144 rows spans 48 GEMM tiles; late layers (M = 96) are one ragged tile."""
    net = synth.mobilenetv2(6, 32, 10, 0, True)
    one_step_case(net, 23, [0, 7, 14, 20], perturbed=True)


def test_momentum_and_weight_decay_over_three_steps():
    ls, cfg = synth.tiny_mbv2(batch=5, hw=6)
    om, gm = make_oracle(ls, cfg, 24), make_gpu(ls, cfg, 24)
    pts = [0, 3, gm.L]
    gm.ftp_set_partition(pts)
    for it in range(3):
        x, y = synth.make_batch(24, cfg, it)
        ref = om.step(pts, x, y)
        got = gm.ftp_train_step(to_dev(x), to_dev(y), cfg["lr"])
        assert abs(got - ref) <= TOL_FP32 * abs(ref)
        for u in range(gm.L):          # re-synchronise: tolerance is per step from identical state
            gm.ftp_set_tensor(F.T_WEIGHTS, u, om.unit_params(u).astype(np.float32))
    # momentum buffers were re-marked by set_tensor; a fresh pair checks the buffer itself
    om, gm = make_oracle(ls, cfg, 24), make_gpu(ls, cfg, 24)
    for it in range(3):
        x, y = synth.make_batch(24, cfg, it)
        om.step([0, gm.L], x, y)
        gm.ftp_train_step(to_dev(x), to_dev(y), cfg["lr"])
    compare_units(gm, om, "weights", tol=5e-4)     # three steps of drift, not one
    compare_units(gm, om, "state", tol=5e-4)


def test_edge_shapes_batch_one_odd_channels():
    """Batch 1, channel counts that are not multiples of 4 (scalar paths), 1x1 spatial maps, odd widths."""
    L = synth.Layer
    K, A = synth.KIND, synth.ACT
    ls = [L(0, K["CONV2D"], 3, 6, 3, 1, 1, 0, 0, -1), L(0, K["BN"], 6, 6, 0, 1, 0, A["RELU6"], 0, -1),
          L(1, K["DWCONV3x3"], 6, 6, 3, 2, 1, 0, 0, -1), L(1, K["BN"], 6, 6, 0, 1, 0, A["RELU"], 0, -1),
          L(1, K["CONV2D"], 6, 10, 1, 1, 0, A["RELU"], 1, -1), L(2, K["MAXPOOL2"], 10, 10, 2, 2, 0, 0, 0, -1),
          L(2, K["GAP"], 10, 10, 0, 1, 0, 0, 0, -1), L(2, K["FC"], 10, 7, 1, 1, 0, 0, 1, -1),
          L(2, K["SOFTMAX_CE"], 7, 7, 0, 1, 0, 0, 0, -1)]
    for batch, hw in ((1, 7), (3, 5), (2, 4)):
        cfg = synth.config(batch, 3, hw, hw, 7, momentum=0.9, weight_decay=1e-4)
        one_step_case((ls, cfg), 25, [0, 1, 2, 3])


def test_conv1d_ragged_lengths():
    for batch, t, width in ((3, 50, 12), (1, 5, 4), (5, 131, 20)):
        one_step_case(synth.har_cnn(batch, 9, t, width, 6), 26, [0, 2, 5])
