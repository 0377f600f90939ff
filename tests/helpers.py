"""Shared test plumbing: build the oracle and the CUDA model from the same seeded arrays and
compare tensors.  No arithmetic of the method lives here."""
import numpy as np

import oracle
import synth

TOL_FP32 = 1e-4      # relative, max-abs norm: the tolerance the fp32 path is held to
TOL_BF16 = 2e-2      # relative, max-abs norm on logits and gradients: the bf16 tensor-core path


MARGIN = 4e-7        # per contraction of depth: least relative distance from a kink / pool tie (see clear_batch)


def _depths(layers):
    d, out = 0, []
    for l in layers:
        if l.kind in (synth.KIND["CONV1D"], synth.KIND["CONV2D"], synth.KIND["DWCONV3x3"], synth.KIND["FC"]):
            d += 1
        out.append(d)
    return out


def clear_batch(om, idx, cfg, first_try=0, margin=MARGIN, tries=3000, transform=None):
    """Seeded rejection: the first batch (by draw index) whose oracle forward keeps every value of
    op i at least margin * depth_i (relative) away from an activation kink or a max-pool tie,
    depth_i being the number of contractions before it: float32 rounding noise grows about linearly
    with depth (measured ~1e-7 per contraction).  Float32 and float64 then take the same discrete
    decisions and gradients are comparable to 1e-4.  The oracle's BN running statistics are
    restored after each probe."""
    depth = _depths(om.layers)
    for t in range(first_try, first_try + tries):
        x, y = synth.make_batch(idx, cfg, t)
        if transform is not None:
            x = transform(x)            # e.g. rounding to the storage type the device path reads
        keep = [[v.copy() for v in s] for s in om.s]
        om.forward(0, om.L, x, y)
        om.s = keep
        if all(m >= margin * max(depth[i], 1) for i, m in om.decision_margin(per_op=True)):
            return x, y, t
    raise RuntimeError("no kink-free batch found; lower the size or the margin")


def rel_err(got, ref):
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if ref.size == 0:
        return 0.0
    assert np.all(np.isfinite(got)), "non-finite values from the CUDA path"
    return float(np.max(np.abs(got - ref)) / max(np.max(np.abs(ref)), 1e-30))


def make_oracle(layers, cfg, idx):
    return oracle.OracleModel(layers, cfg, synth.init_params(idx, layers), synth.init_state(layers))


def make_gpu(layers, cfg, idx, max_stages=None):
    import paper_2110_02781_b200 as F
    cfg = dict(cfg)
    if max_stages:
        cfg["max_stages"] = max_stages
    m = F.Model(layers, cfg)
    m.load_params(synth.init_params(idx, layers), synth.init_state(layers))
    return m


def perturb(layers, idx, scale=0.1):
    """Initial parameters moved off the symmetric start (beta 0, bias 0) with seeded noise."""
    g = synth.rng_stream(idx, "misc")
    return [[(a + scale * g.standard_normal(a.shape)).astype(np.float32) for a in arrs]
            for arrs in synth.init_params(idx, layers)]


def safe_params(layers, idx, scale=0.1):
    """Perturbed parameters whose BN outputs stay inside the linear range of ReLU / ReLU6
    (beta near 3, gamma near 0.25: a kink is 12 standard deviations away), so large cases have no
    ambiguous activation decision at all; contraction, depthwise and BN arithmetic is unchanged."""
    out = perturb(layers, idx, scale)
    for l, arrs in zip(layers, out):
        if l.kind == synth.KIND["BN"]:
            arrs[0] = (0.25 * arrs[0]).astype(np.float32)
            arrs[1] = (3.0 + arrs[1]).astype(np.float32)
        if l.kind == synth.KIND["FC"]:          # features now carry a large offset: keep the softmax unsaturated
            arrs[0] = (0.05 * arrs[0]).astype(np.float32)
    return out


def to_dev(x, dtype=None):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    return t.to(dtype) if dtype is not None else t


def gpu_step_split(m, points, x_dev, y_dev, lr, bufs=None):
    """One synchronous step through the public stage calls, with caller-owned boundary buffers."""
    import torch
    L = m.L
    acts, grads = [x_dev], []
    for a, b in zip(points[:-1], points[1:]):
        if b == L:
            loss = torch.zeros(1, device="cuda")
            m.ftp_run_stage_forward(a, b, acts[-1], None, y_dev, loss)
        else:
            shp, _ = m.ftp_unit_output_shape(b - 1)
            out = torch.empty(shp, dtype=m.act_dtype, device="cuda")
            m.ftp_run_stage_forward(a, b, acts[-1], out)
            acts.append(out)
    g = None
    for i in range(len(points) - 2, -1, -1):
        a, b = points[i], points[i + 1]
        gin = torch.empty_like(acts[i]) if a > 0 else None
        m.ftp_run_stage_backward(a, b, g, gin)
        grads.append(gin)
        g = gin
    for a, b in zip(points[:-1], points[1:]):
        m.ftp_sgd_step(a, b, lr)
    torch.cuda.synchronize()
    return float(loss.item()), acts, grads[::-1]
