"""Float64 model driver: stage forward / backward over a unit range, SGD, snapshot
(test infrastructure only; shares no code with the CUDA library).

Follows Sec. III-B (a worker builds the sub-model [start_i, end_i] from the partition
points), Sec. III-C restricted to one batch in flight (forward through all stages, then
backward, then the update), Sec. IV-B (SGD with momentum and weight decay) and
Sec. III-E (a replica is a copy of a stage's weights).
"""
import numpy as np
from . import ops

CONV1D, CONV2D, DW, BN, ACT, ADD, MAXPOOL, GAP, FC, CE = range(10)


def round_bf16(x):
    """Round to the nearest bfloat16 (ties to even), returned as float64."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


class OracleModel:
    def __init__(self, layers, cfg, params, state, storage=None):
        """`params` / `state`: per op a list of arrays in canonical order (copied to float64).

        storage: None -> everything float64.  "bf16" -> the precision the bf16 configurations fix:
        activations and the gradients handed from op to op are stored as bfloat16, dense-convolution
        weights are used as bfloat16, accumulation is exact (float64 here, float32 on the device);
        master weights, depthwise / BN / classifier parameters, statistics, logits and the loss are
        not rounded.  A value is rounded where it is stored: a BN whose result goes straight into a
        residual add is rounded once, after the add; a gradient with two contributions is rounded
        once, after they are summed.  Activation decisions are taken on the stored values for
        convolutions with a fused activation and on the unrounded normalised value for BN."""
        self.q = round_bf16 if (storage if storage is not None else ("bf16" if cfg.get("precision") == 1 else None)) == "bf16" \
            else (lambda v: v)
        self.quantised = self.q is round_bf16
        self.layers = list(layers)
        self.cfg = dict(cfg)
        self.L = self.layers[-1].unit + 1
        self.p = [[np.array(a, dtype=np.float64) for a in arrs] for arrs in params]
        self.s = [[np.array(a, dtype=np.float64) for a in arrs] for arrs in state]
        self.g = [[np.zeros_like(a) for a in arrs] for arrs in self.p]
        self.m = [[None for _ in arrs] for arrs in self.p]         # momentum buffers
        self.out = {}            # op index -> forward output (index first_op-1 = stage input)
        self.saved = {}          # op index -> extra values kept for backward
        self.labels = None
        self.loss = None
        self.logits = None

    # ---- helpers -------------------------------------------------------------------------
    def ops_of(self, a, b):
        return [i for i, l in enumerate(self.layers) if a <= l.unit < b]

    def _pads(self, l):
        return (0, l.pad) if l.kind == CONV1D else (l.pad, l.pad)

    # ---- forward of units [a, b) ---------------------------------------------------------
    def forward(self, a, b, act_in, labels=None):
        idx = self.ops_of(a, b)
        self.out[idx[0] - 1] = np.asarray(act_in, dtype=np.float64)
        for i in idx:
            l = self.layers[i]
            x = self.out[i - 1]
            if l.kind in (CONV1D, CONV2D, FC):
                ph, pw = self._pads(l)
                bias = self.p[i][1] if l.has_bias else None
                w = self.q(self.p[i][0]) if l.kind != FC else self.p[i][0]
                pre = ops.conv_fwd(x, w, bias, l.stride, ph, pw)
                if l.kind != FC:
                    pre = self.q(pre)
                self.saved[i] = pre
                y = ops.act_fwd(pre, l.act)
            elif l.kind == DW:
                y = self.q(ops.dwconv_fwd(x, self.p[i][0], l.stride, l.pad))
            elif l.kind == BN:
                z, mu, var, xhat = ops.bn_fwd(x, self.p[i][0], self.p[i][1], self.cfg["bn_eps"])
                self.saved[i] = (z, var, xhat)
                m = x.shape[0] * x.shape[1] * x.shape[2]
                mom = self.cfg["bn_momentum"]
                unbiased = var * m / (m - 1) if m > 1 else var
                self.s[i][0] = (1 - mom) * self.s[i][0] + mom * mu
                self.s[i][1] = (1 - mom) * self.s[i][1] + mom * unbiased
                y = ops.act_fwd(z, l.act)
                if not (i + 1 < len(self.layers) and self.layers[i + 1].kind == ADD):
                    y = self.q(y)
            elif l.kind == ACT:
                y = ops.act_fwd(x, l.act)
            elif l.kind == ADD:
                y = self.q(x + self.out[l.residual_src])
            elif l.kind == MAXPOOL:
                y, arg = ops.maxpool_fwd(x)
                self.saved[i] = arg
            elif l.kind == GAP:
                y = self.q(ops.gap_fwd(x))
            elif l.kind == CE:
                self.labels = np.asarray(labels)
                self.logits = x.reshape(x.shape[0], -1).copy()
                self.loss, prob = ops.softmax_ce_fwd(x, self.labels)
                self.saved[i] = prob
                y = np.array(self.loss)
            else:
                raise ValueError(l.kind)
            self.out[i] = y
        return self.out[idx[-1]]

    # ---- backward of units [a, b) --------------------------------------------------------
    def backward(self, a, b, grad_out=None):
        idx = self.ops_of(a, b)
        grad = {}
        if grad_out is not None:
            grad[idx[-1]] = np.asarray(grad_out, dtype=np.float64)

        def acc(j, v):
            grad[j] = grad[j] + v if j in grad else v

        for i in reversed(idx):
            l = self.layers[i]
            x = self.out[i - 1]
            if l.kind == CE:
                acc(i - 1, ops.softmax_ce_bwd(self.saved[i], self.labels, x.shape))
                continue
            d = grad.pop(i)
            if l.kind != FC:
                d = self.q(d)                    # the gradient as it was stored for this op to read
            if l.kind in (CONV1D, CONV2D, FC):
                ph, pw = self._pads(l)
                d = ops.act_bwd(self.saved[i], d, l.act)
                w = self.q(self.p[i][0]) if l.kind != FC else self.p[i][0]
                dx, dw, db = ops.conv_bwd(x, w, d, l.stride, ph, pw, l.has_bias)
                self.g[i][0] = dw
                if l.has_bias:
                    self.g[i][1] = db
                acc(i - 1, dx)
            elif l.kind == DW:
                dx, dw = ops.dwconv_bwd(x, self.p[i][0], d, l.stride, l.pad)
                self.g[i][0] = dw
                acc(i - 1, dx)
            elif l.kind == BN:
                z, var, xhat = self.saved[i]
                d = ops.act_bwd(z, d, l.act)
                dy, dgam, dbet = ops.bn_bwd(d, xhat, self.p[i][0], var, self.cfg["bn_eps"])
                self.g[i][0], self.g[i][1] = dgam, dbet
                acc(i - 1, dy)
            elif l.kind == ACT:
                acc(i - 1, ops.act_bwd(x, d, l.act))
            elif l.kind == ADD:
                acc(i - 1, d)
                acc(l.residual_src, d)
            elif l.kind == MAXPOOL:
                acc(i - 1, ops.maxpool_bwd(d, self.saved[i], x.shape))
            elif l.kind == GAP:
                acc(i - 1, ops.gap_bwd(d, x.shape))
        g = grad.get(idx[0] - 1)
        return None if g is None else self.q(g)

    # ---- how close the last forward came to a discrete decision ---------------------------------
    def decision_margin(self, a=0, b=None, per_op=False):
        """Smallest gap, over units [a, b) of the last forward, between a value and a point where
        the path takes a discrete decision: an activation kink (0, and 6 for ReLU6) or a tie
        between the two largest entries of a max-pool window.  Each gap is relative to the
        largest magnitude in its tensor.  At such a point float32 and float64 arithmetic may
        decide differently and the gradient jumps, so parity inputs are drawn with this margin
        above the float32 rounding noise; what is compared is then unique."""
        worst = np.inf
        each = []
        for i in self.ops_of(a, self.L if b is None else b):
            l = self.layers[i]
            if l.kind == MAXPOOL:
                x = self.out[i - 1]
                n, h, w, c = x.shape
                ho, wo = h // 2, w // 2
                win = np.sort(np.stack([x[:, p:2 * ho:2, q:2 * wo:2] for p in (0, 1) for q in (0, 1)]), axis=0)
                gap = win[3] - win[2]
                # a tie between values clamped by the preceding activation routes no gradient either way
                prev = self.layers[i - 1].act if i > 0 else 0
                harmless = (gap == 0) & ((win[3] == 0.0) if prev else False)
                if prev == 2:
                    harmless |= (gap == 0) & (win[3] == 6.0)
                gap = np.where(harmless, np.inf, gap)
                each.append((i, float(gap.min() / max(np.abs(x).max(), 1e-300))))
                worst = min(worst, each[-1][1])
                continue
            if l.act == 0 or l.kind == CE:
                continue
            if l.kind in (CONV1D, CONV2D, FC):
                z = self.saved[i]
            elif l.kind == BN:
                z = self.saved[i][0]
            else:
                z = self.out[i - 1]
            gap = np.abs(z).min()
            if l.act == 2:
                gap = min(gap, np.abs(z - 6.0).min())
            each.append((i, float(gap / max(np.abs(z).max(), 1e-300))))
            worst = min(worst, each[-1][1])
        return each if per_op else worst

    def ambiguous_outputs(self, i, margin):
        """Boolean mask over op i's output: True where its own discrete decision (activation kink,
        max-pool tie) lies within `margin` (relative to the tensor's largest magnitude)."""
        l = self.layers[i]
        if l.kind == MAXPOOL:
            x = self.out[i - 1]
            ho, wo = x.shape[1] // 2, x.shape[2] // 2
            win = np.sort(np.stack([x[:, p:2 * ho:2, q:2 * wo:2] for p in (0, 1) for q in (0, 1)]), axis=0)
            return (win[3] - win[2]) <= margin * np.abs(x).max()
        z = self.saved[i] if l.kind in (CONV1D, CONV2D, FC) else (self.saved[i][0] if l.kind == BN else self.out[i - 1])
        if l.act == 0:
            return np.zeros(z.shape, bool)
        near = np.abs(z) <= margin * np.abs(z).max()
        if l.act == 2:
            near |= np.abs(z - 6.0) <= margin * np.abs(z).max()
        return near

    # ---- SGD on units [a, b) (Sec. IV-B: momentum 0.9, weight decay 4e-5) --------------------
    def sgd(self, a, b, lr=None):
        """g <- g + wd*w ; m <- g on the first update, else mu*m + g ; w <- w - lr*m."""
        lr = self.cfg["lr"] if lr is None else lr
        mu, wd = self.cfg["momentum"], self.cfg["weight_decay"]
        for i in self.ops_of(a, b):
            for k, w in enumerate(self.p[i]):
                g = self.g[i][k] + wd * w
                if mu != 0.0:
                    self.m[i][k] = g.copy() if self.m[i][k] is None else mu * self.m[i][k] + g
                    g = self.m[i][k]
                self.p[i][k] = w - lr * g

    def step(self, points, x, labels, lr=None):
        """One synchronous step over the stages given by partition points p_0=0 < ... < p_N=L."""
        act = x
        for a, b in zip(points[:-1], points[1:]):
            act = self.forward(a, b, act, labels if b == self.L else None)
        grad = None
        for a, b in reversed(list(zip(points[:-1], points[1:]))):
            grad = self.backward(a, b, grad)
        for a, b in zip(points[:-1], points[1:]):
            self.sgd(a, b, lr)
        return self.loss

    # ---- flat views in canonical unit order -------------------------------------------------
    def _flat(self, store, unit):
        parts = [v.reshape(-1) for i, l in enumerate(self.layers) if l.unit == unit
                 for v in store[i]]
        return np.concatenate(parts) if parts else np.zeros(0)

    def unit_params(self, unit):
        return self._flat(self.p, unit)

    def unit_grads(self, unit):
        return self._flat(self.g, unit)

    def unit_state(self, unit):
        return self._flat(self.s, unit)

    def set_unit(self, unit, params_flat, state_flat, reset_momentum=True):
        """Load a unit from a replica (Sec. III-F): trainable weights and BN running statistics in
        canonical order; the momentum of the unit starts afresh, as on a worker that just received
        the weights (the replica of Sec. III-E holds weights only)."""
        def scatter(store, flat):
            off = 0
            for i, l in enumerate(self.layers):
                if l.unit != unit:
                    continue
                for k, v in enumerate(store[i]):
                    store[i][k] = np.asarray(flat[off:off + v.size], np.float64).reshape(v.shape).copy()
                    off += v.size
            assert off == len(flat), "replica size does not match the unit"
        scatter(self.p, params_flat)
        scatter(self.s, state_flat)
        if reset_momentum:
            for i, l in enumerate(self.layers):
                if l.unit == unit:
                    self.m[i] = [None] * len(self.m[i])

    def unit_param_count(self, unit):
        return self.unit_params(unit).size

    def snapshot(self, a, b):
        """A replica of a stage (Sec. III-E): its trainable weights then its BN running
        statistics, unit by unit in canonical order, as float32 bytes."""
        parts = []
        for u in range(a, b):
            parts += [self.unit_params(u), self.unit_state(u)]
        return np.concatenate(parts).astype(np.float32)
