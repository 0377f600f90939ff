"""GPU tests of the fused routes: a batch norm that is applied by the op that reads it (never stored) against the
same network with every batch norm stored by its own kernel.  The reader evaluates (y - mean) * scale + offset with
offset = beta - mean_lo * scale formed in double (mean_lo: the part of the mean that a float does not hold), the
stand-alone kernel ((y - mean) - mean_lo) * scale + beta: the two agree to float rounding, so losses, gradients, updated weights and running statistics must agree to a few 1e-6 in
float models; in bf16 models a value that rounds to the neighbouring bf16 number can flip an activation decision
further on, so gradients are compared in the L2 norm there.  The oracle comparisons of the other files run on the
default (fused) route."""
import os

import numpy as np
import pytest

import synth
from helpers import make_gpu, to_dev

pytestmark = pytest.mark.gpu
F = pytest.importorskip("paper_2110_02781_b200")


def _run(ls, cfg, idx, env, steps=2):
    import torch
    old = {k: os.environ.get(k) for k in env}
    os.environ.update(env)
    try:
        gm = make_gpu(ls, cfg, idx)
    finally:
        for k, v in old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v
    x, y = synth.make_batch(idx, cfg)
    xd = to_dev(x, torch.bfloat16 if cfg["precision"] == 1 else None)
    yd = to_dev(y)
    gm.ftp_set_partition([0, gm.L // 2, gm.L])
    out = []
    for _ in range(steps):
        loss = gm.ftp_train_step(xd, yd, cfg["lr"])
        out.append((loss, [gm.ftp_get_tensor(F.T_GRADS, u) for u in range(gm.L)],
                    [gm.ftp_get_tensor(F.T_WEIGHTS, u) for u in range(gm.L)],
                    [gm.ftp_get_tensor(F.T_STATE, u) for u in range(gm.L)]))
    gm.close()
    return out


# ragged on purpose: 3 x 10 x 10 = 300 rows (not a multiple of 128), 24 / 144 channels (reductions that end inside a
# 32-wide block), a stride-2 block, a residual block
RAGGED = dict(table=[(1, 16, 1, 1), (6, 24, 2, 1), (6, 40, 1, 2)], stem_c=32, last_c=64)


def test_default_route_defers_batch_norms_in_float_models():
    """The float default really takes the fused route: fewer launches per step than with every batch norm stored."""
    ls, cfg = synth.tiny_mbv2()
    counts = []
    for env in ({}, {"FTP_FUSE_BN": "0"}):
        old = os.environ.pop("FTP_FUSE_BN", None)
        os.environ.update(env)
        try:
            gm = make_gpu(ls, cfg, 41)
        finally:
            os.environ.pop("FTP_FUSE_BN", None)
            if old is not None:
                os.environ["FTP_FUSE_BN"] = old
        x, y = synth.make_batch(41, cfg)
        xd, yd = to_dev(x), to_dev(y)
        gm.ftp_train_step(xd, yd, 0.01)
        n0 = gm.ftp_launch_count()
        gm.ftp_train_step(xd, yd, 0.01)
        counts.append(gm.ftp_launch_count() - n0)
        gm.close()
    assert counts[0] < counts[1], counts


@pytest.mark.parametrize("precision", [0, 1])
@pytest.mark.parametrize("shape", ["tiny", "ragged", "wide"])
def test_bn_applied_on_load_matches_bn_stored(precision, shape):
    if shape == "tiny":
        ls, cfg = synth.tiny_mbv2(precision=precision)
    elif shape == "ragged":
        ls, cfg = synth.mobilenetv2(3, 10, 7, precision, True, **RAGGED)
    else:       # several 128-row tiles and reductions cut into slices (late-layer shapes)
        ls, cfg = synth.mobilenetv2(8, 16, 10, precision, True, table=[(6, 64, 1, 2), (6, 96, 2, 1), (6, 160, 1, 2)], stem_c=32, last_c=256)
    a = _run(ls, cfg, 41, {"FTP_FUSE_BN": "3"})          # into depthwise and 1x1 readers
    b = _run(ls, cfg, 41, {"FTP_FUSE_BN": "0"})
    tol = 2e-5 if precision == 0 else 5e-2

    def l2(p, q):
        p, q = np.asarray(p, np.float64), np.asarray(q, np.float64)
        return float(np.linalg.norm(p - q) / max(np.linalg.norm(q), 1e-30)) if q.size else 0.0

    for step, ((la, ga, wa, sa), (lb, gb, wb, sb)) in enumerate(zip(a, b)):
        assert abs(la - lb) <= tol * abs(lb)
        if precision == 1 and step > 0:
            # The second bf16 step starts from weights that differ in a few last bits (a depthwise backward kernel that
            # also leaves the batch-norm sums adds them in another order than the separate reduction pass), and that is
            # enough to flip activation decisions all through the network: only the loss is comparable there.
            continue
        for u in range(len(ga)):
            assert l2(ga[u], gb[u]) <= tol, f"gradients of unit {u}: {l2(ga[u], gb[u]):.3e}"
            assert l2(wa[u], wb[u]) <= tol and l2(sa[u], sb[u]) <= tol, f"weights / running statistics of unit {u}"
