"""Layer definitions in float64, NHWC activations, KRSC convolution weights.

Each function is the textbook definition written with numpy slices; the only
library primitive used as a step is a matrix product over the channel axis.
Test infrastructure only.
"""
import numpy as np

__all__ = ["conv2d_forward", "conv2d_backward", "dwconv2d_forward", "dwconv2d_backward",
           "bn_forward", "bn_backward", "act_forward", "act_backward", "gap_forward",
           "gap_backward", "linear_forward", "linear_backward", "mse_loss",
           "softmax_xent_loss", "sgd_momentum_step", "warmup_forwards", "stage_memory", "sigmoid", "se_forward", "se_backward"]


def _out_size(n, k, stride, pad):
    return (n + 2 * pad - k) // stride + 1


def _padded(x, pad):
    return np.pad(x, ((0, 0), (pad, pad), (pad, pad), (0, 0))) if pad else x


def conv2d_forward(x, w, stride, pad):
    """z[n,ho,wo,k] = sum_{r,s,c} x[n, ho*stride-pad+r, wo*stride-pad+s, c] * w[k,r,s,c]
    (cross-correlation, zero padding, no bias).  One FP layer of a stage model (Section 3.2)."""
    n, h, wd, c = x.shape
    k, kr, ks, c2 = w.shape
    assert c == c2
    ho, wo = _out_size(h, kr, stride, pad), _out_size(wd, ks, stride, pad)
    xp = _padded(x, pad)
    z = np.zeros((n, ho, wo, k))
    for r in range(kr):
        for s in range(ks):
            xs = xp[:, r:r + stride * (ho - 1) + 1:stride, s:s + stride * (wo - 1) + 1:stride, :]
            z += xs @ w[:, r, s, :].T
    return z


def conv2d_backward(x, w, dz, stride, pad):
    """Adjoints of conv2d_forward: dx (w.r.t. the input) and dw (w.r.t. the weights)."""
    n, h, wd, c = x.shape
    k, kr, ks, _ = w.shape
    _, ho, wo, _ = dz.shape
    xp = _padded(x, pad)
    dxp = np.zeros_like(xp)
    dw = np.zeros_like(w)
    for r in range(kr):
        for s in range(ks):
            sl = (slice(None), slice(r, r + stride * (ho - 1) + 1, stride),
                  slice(s, s + stride * (wo - 1) + 1, stride), slice(None))
            dxp[sl] += dz @ w[:, r, s, :]
            dw[:, r, s, :] = dz.reshape(-1, k).T @ xp[sl].reshape(-1, c)
    dx = dxp[:, pad:pad + h, pad:pad + wd, :] if pad else dxp
    return dx, dw


def dwconv2d_forward(x, w, stride, pad):
    """Depthwise: z[n,ho,wo,c] = sum_{r,s} x[n, ho*stride-pad+r, wo*stride-pad+s, c] * w[c,r,s]."""
    n, h, wd, c = x.shape
    c2, kr, ks = w.shape
    assert c == c2
    ho, wo = _out_size(h, kr, stride, pad), _out_size(wd, ks, stride, pad)
    xp = _padded(x, pad)
    z = np.zeros((n, ho, wo, c))
    for r in range(kr):
        for s in range(ks):
            z += xp[:, r:r + stride * (ho - 1) + 1:stride, s:s + stride * (wo - 1) + 1:stride, :] * w[:, r, s]
    return z


def dwconv2d_backward(x, w, dz, stride, pad):
    n, h, wd, c = x.shape
    _, kr, ks = w.shape
    _, ho, wo, _ = dz.shape
    xp = _padded(x, pad)
    dxp = np.zeros_like(xp)
    dw = np.zeros_like(w)
    for r in range(kr):
        for s in range(ks):
            sl = (slice(None), slice(r, r + stride * (ho - 1) + 1, stride),
                  slice(s, s + stride * (wo - 1) + 1, stride), slice(None))
            dxp[sl] += dz * w[:, r, s]
            dw[:, r, s] = (dz * xp[sl]).sum(axis=(0, 1, 2))
    dx = dxp[:, pad:pad + h, pad:pad + wd, :] if pad else dxp
    return dx, dw


def bn_forward(z, gamma, beta, eps):
    """Training-mode BatchNorm over the micro-batch: per channel, over all N*H*W positions,
    mu = mean(z), var = mean((z-mu)^2) (biased), xhat = (z-mu)/sqrt(var+eps), y = gamma*xhat+beta."""
    ax = tuple(range(z.ndim - 1))
    mu = z.mean(axis=ax)
    var = ((z - mu) ** 2).mean(axis=ax)
    xhat = (z - mu) / np.sqrt(var + eps)
    return gamma * xhat + beta, (mu, var, xhat)


def bn_backward(dy, cache, gamma, eps):
    """dbeta = sum dy; dgamma = sum dy*xhat; dz = gamma/sqrt(var+eps) * (dy - dbeta/N - xhat*dgamma/N)."""
    mu, var, xhat = cache
    ax = tuple(range(dy.ndim - 1))
    cnt = dy.size // dy.shape[-1]
    dbeta = dy.sum(axis=ax)
    dgamma = (dy * xhat).sum(axis=ax)
    dz = gamma / np.sqrt(var + eps) * (dy - dbeta / cnt - xhat * dgamma / cnt)
    return dz, dgamma, dbeta


def act_forward(kind, pre):
    if kind == "relu6":
        return np.minimum(np.maximum(pre, 0.0), 6.0)
    if kind == "relu":
        return np.maximum(pre, 0.0)
    if kind == "silu":
        return pre * sigmoid(pre)
    raise ValueError(kind)


def sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def act_backward(kind, dy, pre):
    """ReLU / ReLU6: gradient passes only strictly inside the linear region (0 at the kinks).
    SiLU x*sigmoid(x): derivative sigmoid(x) * (1 + x * (1 - sigmoid(x)))."""
    if kind == "relu6":
        return dy * ((pre > 0.0) & (pre < 6.0))
    if kind == "relu":
        return dy * (pre > 0.0)
    if kind == "silu":
        sg = sigmoid(pre)
        return dy * sg * (1.0 + pre * (1.0 - sg))
    raise ValueError(kind)


def se_forward(x, w1, b1, w2, b2):
    """Squeeze-and-excitation of the EfficientNet block (one of the paper's vision workloads, Section 5.1): per sample
    s[n,c] = mean_{h,w} x;  h = silu(s w1^T + b1);  g = sigmoid(h w2^T + b2);  out[n,h,w,c] = x[n,h,w,c] * g[n,c].
    Returns (out, cache)."""
    s = x.mean(axis=(1, 2))
    p1 = s @ w1.T + b1
    h = p1 * sigmoid(p1)
    p2 = h @ w2.T + b2
    g = sigmoid(p2)
    return x * g[:, None, None, :], (s, p1, h, g)


def se_backward(x, w1, w2, cache, dout):
    """Adjoint of se_forward: returns (dx, dw1, db1, dw2, db2)."""
    s, p1, h, g = cache
    hw = x.shape[1] * x.shape[2]
    dg = (dout * x).sum(axis=(1, 2))
    dp2 = dg * g * (1.0 - g)
    dw2 = dp2.T @ h
    db2 = dp2.sum(axis=0)
    dh = dp2 @ w2
    sg = sigmoid(p1)
    dp1 = dh * sg * (1.0 + p1 * (1.0 - sg))
    dw1 = dp1.T @ s
    db1 = dp1.sum(axis=0)
    ds = dp1 @ w1
    dx = dout * g[:, None, None, :] + (ds / hw)[:, None, None, :]
    return dx, dw1, db1, dw2, db2


def gap_forward(x):
    return x.mean(axis=(1, 2), keepdims=True)


def gap_backward(da, h, w):
    return np.broadcast_to(da / (h * w), (da.shape[0], h, w, da.shape[3])).copy()


def linear_forward(a, w, b):
    """logits[n,j] = sum_i a[n,i] * w[j,i] + b[j]."""
    return a @ w.T + b


def linear_backward(a, w, dlogits):
    return dlogits @ w, dlogits.T @ a, dlogits.sum(axis=0)


def mse_loss(y, t):
    """L = mean over all elements of (y-t)^2; dL/dy = 2 (y-t) / numel."""
    d = y - t
    return float((d * d).mean()), 2.0 * d / d.size


def softmax_xent_loss(logits, labels):
    """L = mean_n( -log softmax(logits_n)[label_n] ); dL/dlogits = (softmax - onehot)/rows."""
    rows = logits.shape[0]
    s = logits - logits.max(axis=1, keepdims=True)
    lse = np.log(np.exp(s).sum(axis=1, keepdims=True))
    logp = s - lse
    loss = float(-logp[np.arange(rows), labels].mean())
    d = np.exp(logp)
    d[np.arange(rows), labels] -= 1.0
    return loss, d / rows


def sgd_momentum_step(w, v, grad_sum, n_micro, lr, momentum):
    """End-of-round update (Section 3.2: accumulated gradients are applied once per round):
    g = grad_sum / M;  v <- momentum * v + g;  w <- w - lr * v."""
    g = grad_sum / n_micro
    v_new = momentum * v + g
    return w - lr * v_new, v_new


def warmup_forwards(n_stages, p):
    """K_p = 2 (P - p) - 1 forward passes of stage p before strict 1F1B (Section 3.2)."""
    return 2 * (n_stages - p) - 1


def stage_memory(mem_mod, mem_opt, mem_act, k_p):
    """Eq. (3): Mem_p = Mem_MOD + Mem_OPT + K_p * Mem_ACT(beta)."""
    return mem_mod + mem_opt + k_p * mem_act
