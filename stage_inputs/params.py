"""Initial parameter values and the flat parameter order.

Flat order: layers in list order; per layer (weight, [bias], gamma, beta):
  conv    weight [c_out][k][k][c_in]      (KRSC, no bias)
  dwconv  weight [c][k][k]
  bn      gamma [c], beta [c]
  linear  weight [c_out][c_in], bias [c_out]
  se      w1 [k][c], b1 [k], w2 [c][k], b2 [c]      (k = squeeze width)
Conv, linear and squeeze-excite weights ~ U(-b, b), b = sqrt(6 / fan_in), fan_in = k*k*c_in/groups;
gamma = 1, beta = 0, biases = 0.  The stream of a layer's weight is keyed by its index
in the whole network, so a stage cut out of a network sees the same values.
"""
import numpy as np
from .rng import uniform

_PARAM_TID = 1000


def param_layout(net, first, last):
    """[(layer_index, name, shape)] in flat order."""
    out = []
    for i in range(first, last + 1):
        L = net[i]
        if L.op == "conv":
            out.append((i, "weight", (L.c_out, L.k, L.k, L.c_in)))
        elif L.op == "dwconv":
            out.append((i, "weight", (L.c_out, L.k, L.k)))
        elif L.op == "bn":
            out.append((i, "gamma", (L.c_out,)))
            out.append((i, "beta", (L.c_out,)))
        elif L.op == "linear":
            out.append((i, "weight", (L.c_out, L.c_in)))
            out.append((i, "bias", (L.c_out,)))
        elif L.op == "se":
            out.append((i, "w1", (L.k, L.c_out)))
            out.append((i, "b1", (L.k,)))
            out.append((i, "w2", (L.c_out, L.k)))
            out.append((i, "b2", (L.c_out,)))
    return out


def param_count(net, first, last):
    return sum(int(np.prod(s)) for _, _, s in param_layout(net, first, last))


def init_params(net, first, last, seed=0):
    """Flat float32 parameter vector of stage [first, last]."""
    parts = []
    for i, name, shape in param_layout(net, first, last):
        n = int(np.prod(shape))
        L = net[i]
        if name == "weight":
            fan_in = {"conv": L.k * L.k * L.c_in, "dwconv": L.k * L.k, "linear": L.c_in}[L.op]
            b = np.sqrt(6.0 / fan_in)
            parts.append(((2.0 * uniform(seed, _PARAM_TID + i, n) - 1.0) * b).astype(np.float32))
        elif name in ("w1", "w2"):
            b = np.sqrt(6.0 / shape[1])
            parts.append(((2.0 * uniform(seed, (4 if name == "w1" else 5) * _PARAM_TID + i, n) - 1.0) * b).astype(np.float32))
        elif name == "gamma":
            parts.append(np.ones(n, np.float32))
        else:
            parts.append(np.zeros(n, np.float32))
    return np.concatenate(parts) if parts else np.zeros(0, np.float32)


def randomize_bn(params, net, first, last, seed=0):
    """Copy of a flat parameter vector with every BatchNorm's gamma drawn from U(0.5, 1.5) and beta from U(-0.5, 0.5):
    with the initial gamma = 1, beta = 0 a mistake in how scale and shift are used would not show."""
    out = np.array(params, np.float32, copy=True)
    off = 0
    for i, name, shape in param_layout(net, first, last):
        n = int(np.prod(shape))
        if name == "gamma":
            out[off:off + n] = (0.5 + uniform(seed, 2 * _PARAM_TID + i, n)).astype(np.float32)
        elif name == "beta":
            out[off:off + n] = (uniform(seed, 3 * _PARAM_TID + i, n) - 0.5).astype(np.float32)
        off += n
    return out
