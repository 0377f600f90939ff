"""Float64 forward and backward of every op on the path (test infrastructure only).

Each function is the textbook definition written out with numpy; a matrix product is the
only library primitive used as a step.  The paper trains MobileNetV2 with PyTorch autograd
(Sec. IV-A, IV-B) and fixes none of these formulas itself, so the definitions are the
standard ones of that setting: cross-correlation with zero padding, batch normalisation in
training mode with biased batch variance, ReLU6 = min(max(z, 0), 6), mean-reduced softmax
cross-entropy.  Activations are (N, H, W, C).
"""
import numpy as np

__all__ = ["conv_fwd", "conv_bwd", "dwconv_fwd", "dwconv_bwd", "bn_fwd", "bn_bwd", "act_fwd",
           "act_bwd", "maxpool_fwd", "maxpool_bwd", "gap_fwd", "gap_bwd", "softmax_ce_fwd",
           "softmax_ce_bwd", "out_size"]


def out_size(n_in, k, stride, pad):
    return (n_in + 2 * pad - k) // stride + 1


def _pad(x, ph, pw):
    return np.pad(x, ((0, 0), (ph, ph), (pw, pw), (0, 0)))


def conv_fwd(x, w, bias, stride, ph, pw):
    """y[n,ho,wo,co] = sum_{r,s,ci} x[n, ho*st-ph+r, wo*st-pw+s, ci] * w[r,s,ci,co] (+ bias[co])."""
    kh, kw, cin, cout = w.shape
    n, h, wd, _ = x.shape
    ho, wo = out_size(h, kh, stride, ph), out_size(wd, kw, stride, pw)
    xp = _pad(x, ph, pw)
    y = np.zeros((n, ho, wo, cout))
    for r in range(kh):
        for s in range(kw):
            xs = xp[:, r:r + stride * (ho - 1) + 1:stride, s:s + stride * (wo - 1) + 1:stride, :]
            y += xs @ w[r, s]
    if bias is not None:
        y += bias
    return y


def conv_bwd(x, w, dy, stride, ph, pw, has_bias):
    """dw[r,s] = sum_{n,ho,wo} x_shift^T dy ; dx = scatter of dy w[r,s]^T ; dbias = sum dy."""
    kh, kw, cin, cout = w.shape
    n, ho, wo, _ = dy.shape
    xp = _pad(x, ph, pw)
    dxp = np.zeros_like(xp)
    dw = np.zeros_like(w)
    for r in range(kh):
        for s in range(kw):
            sl = (slice(None), slice(r, r + stride * (ho - 1) + 1, stride),
                  slice(s, s + stride * (wo - 1) + 1, stride), slice(None))
            dw[r, s] = xp[sl].reshape(-1, cin).T @ dy.reshape(-1, cout)
            dxp[sl] += dy @ w[r, s].T
    dx = dxp[:, ph:ph + x.shape[1], pw:pw + x.shape[2], :]
    db = dy.sum(axis=(0, 1, 2)) if has_bias else None
    return dx, dw, db


def dwconv_fwd(x, w, stride, pad):
    """Per-channel 3x3: y[n,ho,wo,c] = sum_{r,s} x[n, ho*st-p+r, wo*st-p+s, c] * w[r,s,c]."""
    kh, kw, c = w.shape
    n, h, wd, _ = x.shape
    ho, wo = out_size(h, kh, stride, pad), out_size(wd, kw, stride, pad)
    xp = _pad(x, pad, pad)
    y = np.zeros((n, ho, wo, c))
    for r in range(kh):
        for s in range(kw):
            y += xp[:, r:r + stride * (ho - 1) + 1:stride, s:s + stride * (wo - 1) + 1:stride, :] * w[r, s]
    return y


def dwconv_bwd(x, w, dy, stride, pad):
    kh, kw, c = w.shape
    n, ho, wo, _ = dy.shape
    xp = _pad(x, pad, pad)
    dxp = np.zeros_like(xp)
    dw = np.zeros_like(w)
    for r in range(kh):
        for s in range(kw):
            sl = (slice(None), slice(r, r + stride * (ho - 1) + 1, stride),
                  slice(s, s + stride * (wo - 1) + 1, stride), slice(None))
            dw[r, s] = (xp[sl] * dy).sum(axis=(0, 1, 2))
            dxp[sl] += dy * w[r, s]
    return dxp[:, pad:pad + x.shape[1], pad:pad + x.shape[2], :], dw


def bn_fwd(y, gamma, beta, eps):
    """Training-mode batch norm over (N,H,W): returns z, and (mean, biased var, xhat) for backward."""
    mu = y.mean(axis=(0, 1, 2))
    var = ((y - mu) ** 2).mean(axis=(0, 1, 2))
    xhat = (y - mu) / np.sqrt(var + eps)
    return gamma * xhat + beta, mu, var, xhat


def bn_bwd(dz, xhat, gamma, var, eps):
    """dbeta = sum dz; dgamma = sum dz*xhat; dy = gamma/sqrt(var+eps) * (dz - dbeta/M - xhat*dgamma/M)."""
    m = dz.shape[0] * dz.shape[1] * dz.shape[2]
    dbeta = dz.sum(axis=(0, 1, 2))
    dgamma = (dz * xhat).sum(axis=(0, 1, 2))
    dy = gamma / np.sqrt(var + eps) * (dz - dbeta / m - xhat * dgamma / m)
    return dy, dgamma, dbeta


def act_fwd(z, act):
    if act == 1:
        return np.maximum(z, 0.0)
    if act == 2:
        return np.minimum(np.maximum(z, 0.0), 6.0)
    return z


def act_bwd(z_pre, dout, act):
    """Gradient passes where the unit is strictly inside its linear range (0 at the kinks)."""
    if act == 1:
        return dout * (z_pre > 0.0)
    if act == 2:
        return dout * ((z_pre > 0.0) & (z_pre < 6.0))
    return dout


def maxpool_fwd(x):
    """2x2 window, stride 2; ties go to the first element in row-major window order."""
    n, h, w, c = x.shape
    ho, wo = h // 2, w // 2
    win = np.stack([x[:, 0:2 * ho:2, 0:2 * wo:2], x[:, 0:2 * ho:2, 1:2 * wo:2],
                    x[:, 1:2 * ho:2, 0:2 * wo:2], x[:, 1:2 * ho:2, 1:2 * wo:2]], axis=0)
    arg = win.argmax(axis=0)            # argmax returns the first maximum
    return win.max(axis=0), arg


def maxpool_bwd(dy, arg, in_shape):
    n, h, w, c = in_shape
    ho, wo = h // 2, w // 2
    dx = np.zeros(in_shape)
    for q, (a, b) in enumerate([(0, 0), (0, 1), (1, 0), (1, 1)]):
        dx[:, a:2 * ho:2, b:2 * wo:2, :] = dy * (arg == q)
    return dx


def gap_fwd(x):
    return x.mean(axis=(1, 2), keepdims=True)


def gap_bwd(dy, in_shape):
    return np.broadcast_to(dy / (in_shape[1] * in_shape[2]), in_shape).copy()


def softmax_ce_fwd(logits, labels):
    """loss = -(1/N) sum_n log softmax(logits_n)[label_n], with the row maximum subtracted."""
    z = logits.reshape(logits.shape[0], -1)
    zs = z - z.max(axis=1, keepdims=True)
    logp = zs - np.log(np.exp(zs).sum(axis=1, keepdims=True))
    return -logp[np.arange(z.shape[0]), labels].mean(), np.exp(logp)


def softmax_ce_bwd(prob, labels, shape):
    d = prob.copy()
    d[np.arange(d.shape[0]), labels] -= 1.0
    return (d / d.shape[0]).reshape(shape)
