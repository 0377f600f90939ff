"""Seeded inputs, labels and initial weights (float32 arrays handed to both implementations)."""
import numpy as np
from .nets import KIND, param_shapes, state_shapes

BASE_SEED = 211002781
STREAMS = dict(inputs=0, labels=1, weights=2, capacity=3, misc=4)


def rng_stream(config_index, stream):
    """Counter-based generator (Philox-4x64, key = (seed, stream)): one independent stream per
    purpose, so that drawing more inputs never changes the weights."""
    key = np.array([BASE_SEED + int(config_index), STREAMS[stream]], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def make_batch(config_index, cfg, it=0):
    """Inputs i.i.d. N(0,1) as float32 (N, H, W, C); labels uniform over the classes as int32."""
    g = rng_stream(config_index, "inputs")
    g.bit_generator.advance(int(it) << 40)
    x = g.standard_normal((cfg["batch"], cfg["in_h"], cfg["in_w"], cfg["in_c"])).astype(np.float32)
    h = rng_stream(config_index, "labels")
    h.bit_generator.advance(int(it) << 40)
    y = h.integers(0, cfg["n_classes"], size=cfg["batch"]).astype(np.int32)
    return x, y


def init_params(config_index, layers):
    """Per op a list of float32 arrays in canonical order.  Contraction weights are drawn
    N(0, 2/fan_in) in float64 and rounded once to float32; biases 0; BN gamma 1, beta 0."""
    g = rng_stream(config_index, "weights")
    out = []
    for l in layers:
        arrs = []
        shapes = param_shapes(l)
        if l.kind in (KIND["CONV1D"], KIND["CONV2D"], KIND["FC"], KIND["DWCONV3x3"]):
            s = shapes[0]
            fan_in = s[0] * s[1] * (1 if l.kind == KIND["DWCONV3x3"] else s[2])
            arrs.append((g.standard_normal(s) * np.sqrt(2.0 / fan_in)).astype(np.float32))
            for b in shapes[1:]:
                arrs.append(np.zeros(b, np.float32))
        elif l.kind == KIND["BN"]:
            arrs = [np.ones(shapes[0], np.float32), np.zeros(shapes[1], np.float32)]
        out.append(arrs)
    return out


def init_state(layers):
    """BN running mean 0 and running variance 1."""
    return [[np.zeros(s, np.float32) if i == 0 else np.ones(s, np.float32)
             for i, s in enumerate(state_shapes(l))] for l in layers]


def flat_unit_params(layers, per_op, unit):
    """Concatenate the arrays of one unit's ops in canonical order (pure data movement)."""
    parts = [a.reshape(-1) for l, arrs in zip(layers, per_op) if l.unit == unit for a in arrs]
    return np.concatenate(parts) if parts else np.zeros(0, np.float32)
