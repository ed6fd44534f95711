"""One stage of the pipeline and its HPP-Round, in float64.  Test infrastructure only.

A stage holds the consecutive layers [first, last] of a network (Section 3.2).  Per round it
runs FP for micro-batches 0..M-1, BP for the same micro-batches, accumulates the parameter
gradients of all of them, and applies them once.  Everything is evaluated layer by layer
from the definitions in `layers.py`; nothing is fused, blocked or reordered.

Flat parameter order (the interchange format with any other implementation): layers in list
order; conv weight [c_out][k][k][c_in]; depthwise weight [c][k][k]; bn gamma, beta; linear
weight [c_out][c_in], bias; squeeze-excite w1 [k][c], b1 [k], w2 [c][k], b2 [c].
"""
import numpy as np
from . import layers as L

__all__ = ["Stage", "layer_profile", "group_step"]


def _layer_param_shapes(layer):
    op = layer.op
    if op == "conv":
        return [("weight", (layer.c_out, layer.k, layer.k, layer.c_in))]
    if op == "dwconv":
        return [("weight", (layer.c_out, layer.k, layer.k))]
    if op == "bn":
        return [("gamma", (layer.c_out,)), ("beta", (layer.c_out,))]
    if op == "linear":
        return [("weight", (layer.c_out, layer.c_in)), ("bias", (layer.c_out,))]
    if op == "se":                # squeeze width in the layer's k field
        return [("w1", (layer.k, layer.c_out)), ("b1", (layer.k,)), ("w2", (layer.c_out, layer.k)), ("b2", (layer.c_out,))]
    return []


_CONVLIKE = ("conv", "dwconv", "linear")
_ACTS = ("relu6", "relu")


class Stage:
    """`store`: optional rounding function applied wherever a reduced-precision implementation
    keeps a tensor in memory (all arithmetic stays float64).  With bfloat16 activations the
    ReLU/ReLU6 masks are decisions taken on stored values; a comparison against such an
    implementation is only meaningful if both sides decide on the same stored numbers.  The
    storage points are: the output of every conv / depthwise conv / linear layer (before its
    BatchNorm), the output of a residual add (after the ReLU that directly follows it, if any),
    the pooled features, the stage output, and the gradient with respect to each of those
    stored-or-recomputed unit outputs and to the stage input (rounded after every term added
    to it).  BatchNorm and ReLU/ReLU6 outputs inside a conv->BN->activation chain are never
    stored; a SiLU is not part of a chain: its output and the output of a squeeze-excite layer are
    stored tensors (the squeeze-excite layer's per-sample vectors are not rounded).
    store=None is the plain float64 definition.

    `operand`: optional rounding applied to both operands of every dense contraction (conv and
    linear layers, in FP, in the input-gradient product and in the weight-gradient product; not the
    depthwise conv), modelling tensor-core inputs of reduced precision with exact products and wide
    accumulation.  operand=None keeps float64 operands."""

    def __init__(self, net, first, last, micro_batch, n_micro, params, eps=1e-5, bn_momentum=0.1, store=None, operand=None):
        if not (0 <= first <= last < len(net)):
            raise ValueError("bad layer range")
        self.net, self.first, self.last = net, first, last
        self.B, self.M = micro_batch, n_micro
        self.eps, self.bn_momentum = eps, bn_momentum
        self.p, self.v, self.G, self.g = {}, {}, {}, {}
        self.running = {}
        flat = np.asarray(params, dtype=np.float64)
        off = 0
        for i in range(first, last + 1):
            for name, shape in _layer_param_shapes(net[i]):
                n = int(np.prod(shape))
                self.p[(i, name)] = flat[off:off + n].reshape(shape).copy()
                self.v[(i, name)] = np.zeros(shape)
                self.G[(i, name)] = np.zeros(shape)
                off += n
            if net[i].op == "bn":
                self.running[i] = [np.zeros(net[i].c_out), np.ones(net[i].c_out)]
        if off != flat.size:
            raise ValueError("parameter vector has %d values, stage needs %d" % (flat.size, off))
        self.saved = {}          # micro-batch -> {layer index: output}, caches
        self.n_accumulated = 0
        self.store = store
        self.operand = operand if operand is not None else (lambda t: t)

    def _chains_into_next(self, i):
        """True if layer i+1 continues layer i's chain (conv->BN, conv/BN->activation, add->ReLU),
        i.e. the output of layer i is an unstored intermediate."""
        if i < self.first or i >= self.last:
            return False
        a, b = self.net[i], self.net[i + 1]
        if b.src != i:
            return False
        if a.op in _CONVLIKE:
            return b.op == "bn" or b.op in _ACTS      # _ACTS holds the chain-fused activations only (not silu)
        if a.op == "bn":
            return b.op in _ACTS and i - 1 >= self.first and self.net[i - 1].op in _CONVLIKE and a.src == i - 1
        if a.op == "add":
            return b.op == "relu"
        return False

    def _stored_forward(self, i):
        op = self.net[i].op
        if i == self.last or op in _CONVLIKE or op == "gap":
            return True
        if op == "add":
            return not self._chains_into_next(i)
        if op == "relu":
            return i - 1 >= self.first and self.net[i - 1].op == "add" and self.net[i].src == i - 1
        if op in ("silu", "se"):
            return True
        return False

    # ---- flat views -------------------------------------------------------------------
    def _flat(self, d):
        keys = [(i, name) for i in range(self.first, self.last + 1)
                for name, _ in _layer_param_shapes(self.net[i])]
        return np.concatenate([d[k].ravel() for k in keys]) if keys else np.zeros(0)

    def flat_params(self):
        return self._flat(self.p)

    def flat_momentum(self):
        return self._flat(self.v)

    def flat_grad_accum(self):
        return self._flat(self.G)

    def flat_micro_grad(self):
        return self._flat(self.g)

    # ---- FP of one micro-batch --------------------------------------------------------
    def forward(self, mb, x):
        net = self.net
        val = {self.first - 1: np.asarray(x, dtype=np.float64)}
        cache = {}
        for i in range(self.first, self.last + 1):
            ly = net[i]
            a = val[ly.src]
            if ly.op == "conv":
                val[i] = L.conv2d_forward(self.operand(a), self.operand(self.p[(i, "weight")]), ly.stride, ly.pad)
            elif ly.op == "dwconv":
                val[i] = L.dwconv2d_forward(a, self.p[(i, "weight")], ly.stride, ly.pad)
            elif ly.op == "bn":
                val[i], cache[i] = L.bn_forward(a, self.p[(i, "gamma")], self.p[(i, "beta")], self.eps)
                mu, var, _ = cache[i]
                cnt = a.size // a.shape[-1]
                rm, rv = self.running[i]
                self.running[i] = [(1 - self.bn_momentum) * rm + self.bn_momentum * mu,
                                   (1 - self.bn_momentum) * rv + self.bn_momentum * var * cnt / max(cnt - 1, 1)]
            elif ly.op in ("relu6", "relu", "silu"):
                val[i] = L.act_forward(ly.op, a)
            elif ly.op == "se":
                val[i], cache[i] = L.se_forward(a, self.p[(i, "w1")], self.p[(i, "b1")], self.p[(i, "w2")], self.p[(i, "b2")])
            elif ly.op == "add":
                val[i] = a + val[ly.add_from]
            elif ly.op == "gap":
                val[i] = L.gap_forward(a)
            elif ly.op == "linear":
                val[i] = L.linear_forward(self.operand(a.reshape(a.shape[0], -1)), self.operand(self.p[(i, "weight")]),
                                          self.p[(i, "bias")]).reshape(a.shape[0], 1, 1, -1)
            else:
                raise ValueError(ly.op)
            if self.store is not None and self._stored_forward(i):
                val[i] = self.store(val[i])
        self.saved[mb] = (val, cache)
        return val[self.last]

    # ---- BP of one micro-batch --------------------------------------------------------
    def backward(self, mb, dy):
        net = self.net
        val, cache = self.saved.pop(mb)
        grad = {self.last: np.asarray(dy, dtype=np.float64).reshape(val[self.last].shape)}
        g = {}

        def give(idx, d):
            grad[idx] = grad[idx] + d if idx in grad else d
            if self.store is not None and not self._chains_into_next(idx):
                grad[idx] = self.store(grad[idx])

        for i in range(self.last, self.first - 1, -1):
            ly = net[i]
            d = grad.pop(i)
            a = val[ly.src]
            if ly.op == "conv":
                dx, g[(i, "weight")] = L.conv2d_backward(self.operand(a), self.operand(self.p[(i, "weight")]), self.operand(d),
                                                         ly.stride, ly.pad)
                give(ly.src, dx)
            elif ly.op == "dwconv":
                dx, g[(i, "weight")] = L.dwconv2d_backward(a, self.p[(i, "weight")], d, ly.stride, ly.pad)
                give(ly.src, dx)
            elif ly.op == "bn":
                dz, g[(i, "gamma")], g[(i, "beta")] = L.bn_backward(d, cache[i], self.p[(i, "gamma")], self.eps)
                give(ly.src, dz)
            elif ly.op in ("relu6", "relu", "silu"):
                give(ly.src, L.act_backward(ly.op, d, a))
            elif ly.op == "se":
                dx, g[(i, "w1")], g[(i, "b1")], g[(i, "w2")], g[(i, "b2")] = L.se_backward(a, self.p[(i, "w1")], self.p[(i, "w2")], cache[i], d)
                give(ly.src, dx)
            elif ly.op == "add":
                give(ly.src, d)
                give(ly.add_from, d)
            elif ly.op == "gap":
                give(ly.src, L.gap_backward(d, a.shape[1], a.shape[2]))
            elif ly.op == "linear":
                a2 = a.reshape(a.shape[0], -1)
                d2 = d.reshape(a.shape[0], -1)
                da, g[(i, "weight")], _ = L.linear_backward(self.operand(a2), self.operand(self.p[(i, "weight")]), self.operand(d2))
                g[(i, "bias")] = d2.sum(axis=0)
                give(ly.src, da.reshape(a.shape))
        self.g = g
        return grad[self.first - 1]

    # ---- accumulation and update ------------------------------------------------------
    def accumulate(self, mb):
        """G += g_mb: gradients of all micro-batches of the mini-batch are accumulated."""
        for k in self.G:
            self.G[k] = self.G[k] + self.g[k]
        self.n_accumulated += 1

    def step(self, lr, momentum):
        """Apply the accumulated gradients once at the end of the round, then clear them."""
        if self.n_accumulated != self.M:
            raise RuntimeError("step before all micro-batches were accumulated")
        for k in self.p:
            self.p[k], self.v[k] = L.sgd_momentum_step(self.p[k], self.v[k], self.G[k], self.M, lr, momentum)
            self.G[k] = np.zeros_like(self.G[k])
        self.n_accumulated = 0

    def layer_outputs(self, mb):
        return self.saved[mb][0]


def group_step(stages, shares, lr, momentum):
    """Update of a device group that runs one stage data-parallel (Section 3.2: every device of the group holds the
    stage model and processes its share y_d of each micro-batch; the gradients are synchronised with AllReduce, Eq. (5),
    before they are applied).  Each device's micro-batch loss is a mean over its own samples, so the gradient of the
    whole micro-batch's mean loss is sum_d (y_d / B) G_d with B = sum_d y_d; every device then applies the same
    SGD-momentum step to its copy of the parameters.  reading: the paper does not say how shares of unequal size are
    weighted; y_d / B is the weighting under which a BatchNorm-free group reproduces the single-device round."""
    B = float(sum(shares))
    if any(st.n_accumulated != st.M for st in stages):
        raise RuntimeError("step before all micro-batches were accumulated")
    keys = list(stages[0].p)
    total = {k: sum((y / B) * st.G[k] for st, y in zip(stages, shares)) for k in keys}
    for st in stages:
        for k in keys:
            st.p[k], st.v[k] = L.sgd_momentum_step(st.p[k], st.v[k], total[k], st.M, lr, momentum)
            st.G[k] = np.zeros_like(st.G[k])
        st.n_accumulated = 0


def layer_profile(net, first, last, in_h, in_w, layer, batch, elem_bytes):
    """Closed-form part of the planner's per-layer record (Section 3.3): output bytes a_l,
    weight bytes w_l (float32 parameters), forward FLOPs (2 per multiply-accumulate of the
    conv / linear layers; 0 for the others)."""
    shp = {first - 1: (in_h, in_w)}
    for i in range(first, layer + 1):
        ly = net[i]
        h, w = shp[ly.src]
        if ly.op in ("conv", "dwconv"):
            shp[i] = ((h + 2 * ly.pad - ly.k) // ly.stride + 1, (w + 2 * ly.pad - ly.k) // ly.stride + 1)
        elif ly.op in ("gap", "linear"):
            shp[i] = (1, 1)
        else:
            shp[i] = (h, w)
    ly = net[layer]
    h, w = shp[layer]
    a_l = batch * h * w * ly.c_out * elem_bytes
    w_l = 4 * sum(int(np.prod(s)) for _, s in _layer_param_shapes(ly))
    macs = {"conv": h * w * ly.c_out * ly.c_in * ly.k * ly.k, "dwconv": h * w * ly.c_out * ly.k * ly.k,
            "linear": ly.c_in * ly.c_out}.get(ly.op, 0)
    return {"a_l": a_l, "w_l": w_l, "flops": 2 * macs * batch}
