"""Pins of the oracle's whole-stage round: torch.autograd (float64, CPU) as an independent
library implementation, finite differences, and the invariants of micro-batched training."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle as O
import stage_inputs as si


def torch_stage(net, first, last, params, x_nhwc, eps=1e-5):
    """Forward of layers [first,last] with torch.nn.functional in NCHW float64.
    Returns (output NHWC tensor, list of parameter leaves in flat order, input leaf)."""
    leaves, off = [], 0
    per_layer = {}
    for i, name, shape in si.param_layout(net, first, last):
        n = int(np.prod(shape))
        t = torch.tensor(np.asarray(params[off:off + n], dtype=np.float64).reshape(shape), requires_grad=True)
        off += n
        leaves.append(t)
        per_layer[(i, name)] = t
    x = torch.tensor(np.asarray(x_nhwc, dtype=np.float64), requires_grad=True)
    val = {first - 1: x.permute(0, 3, 1, 2)}
    for i in range(first, last + 1):
        ly = net[i]
        a = val[ly.src]
        if ly.op == "conv":
            val[i] = F.conv2d(a, per_layer[(i, "weight")].permute(0, 3, 1, 2), None, ly.stride, ly.pad)
        elif ly.op == "dwconv":
            val[i] = F.conv2d(a, per_layer[(i, "weight")].unsqueeze(1), None, ly.stride, ly.pad, 1, ly.c_in)
        elif ly.op == "bn":
            val[i] = F.batch_norm(a, None, None, per_layer[(i, "gamma")], per_layer[(i, "beta")], True, 0.1, eps)
        elif ly.op == "relu6":
            val[i] = F.relu6(a)
        elif ly.op == "relu":
            val[i] = F.relu(a)
        elif ly.op == "silu":
            val[i] = F.silu(a)
        elif ly.op == "se":
            sq = a.mean(dim=(2, 3))
            hid = F.silu(F.linear(sq, per_layer[(i, "w1")], per_layer[(i, "b1")]))
            val[i] = a * torch.sigmoid(F.linear(hid, per_layer[(i, "w2")], per_layer[(i, "b2")]))[:, :, None, None]
        elif ly.op == "add":
            val[i] = a + val[ly.add_from]
        elif ly.op == "gap":
            val[i] = F.adaptive_avg_pool2d(a, 1)
        elif ly.op == "linear":
            val[i] = F.linear(a.flatten(1), per_layer[(i, "weight")], per_layer[(i, "bias")])[:, :, None, None]
    return val[last].permute(0, 2, 3, 1), leaves, x


def rel(a, b):
    return np.abs(np.asarray(a) - np.asarray(b)).max() / max(np.abs(np.asarray(b)).max(), 1e-300)


CASES = {
    "mbv2_block": (si.block_net(4, 3), 6, 6, "mse"),
    "mbv2_4blocks": (si.stage_net_mbv2_4blocks(), 8, 8, "mse"),
    "bottlenecks": (si.bottleneck_net(4, [(2, 8, 2, 1), (4, 16, 2, 2)]), 8, 8, "mse"),
    "small_mobilenet": (si.small_mobilenet(10)[0], 16, 16, "xent"),
    "mbconv_k5_se": (si.mbconv_net(4, [(4, 1, 3, 5), (8, 2, 2, 3)]), 9, 9, "mse"),
}


def run_round(net, first, last, h, w, B, M, loss, seed, lr=0.01, mu=0.9, order=None, params=None):
    """One HPP-Round on the oracle.  Returns stage, per-micro-batch (y, dx, loss)."""
    if params is None:
        params = si.init_params(net, first, last, seed) + 0.05 * si.normal(seed, 7, (si.param_count(net, first, last),)).astype(np.float32)
    st = O.Stage(net, first, last, B, M, params)
    c_in = net[first].c_in
    shp = si.out_shape(net, first, last, h, w)[last]
    xs = [si.normal(seed, 100000 + m, (B, h, w, c_in)) for m in range(M)]
    if loss == "mse":
        tg = [si.normal(seed, 200000 + m, (B,) + shp) for m in range(M)]
    else:
        tg = [si.labels(seed, 300000 + m, B, shp[2]) for m in range(M)]
    out = {}
    order = order or [("F", m) for m in range(M)] + [("B", m) for m in range(M)]
    ys = {}
    for kind, m in order:
        if kind == "F":
            ys[m] = st.forward(m, xs[m])
        else:
            if loss == "mse":
                Lm, dy = O.mse_loss(ys[m], tg[m])
            else:
                Lm, dy = O.softmax_xent_loss(ys[m].reshape(B, -1), tg[m])
            dx = st.backward(m, dy)
            st.accumulate(m)
            out[m] = (ys[m], dx, Lm)
    return st, out, xs, tg, params


@pytest.mark.parametrize("name", list(CASES))
def test_round_matches_torch_autograd(name):
    net, h, w, loss = CASES[name]
    first, last = 0, len(net) - 1
    B, M = 3, 2
    st, out, xs, tg, params = run_round(net, first, last, h, w, B, M, loss, seed=11)
    G_ref = None
    for m in range(M):
        y, leaves, x = torch_stage(net, first, last, params, xs[m])
        if loss == "mse":
            Lt = F.mse_loss(y, torch.tensor(tg[m]))
        else:
            Lt = F.cross_entropy(y.reshape(B, -1), torch.tensor(tg[m], dtype=torch.long))
        Lt.backward()
        assert rel(out[m][0], y.detach().numpy()) < 1e-11
        assert abs(out[m][2] - Lt.item()) < 1e-11 * max(1, abs(Lt.item()))
        assert rel(out[m][1], x.grad.numpy()) < 1e-9
        g = np.concatenate([t.grad.numpy().ravel() for t in leaves])
        G_ref = g if G_ref is None else G_ref + g
    assert rel(st.flat_grad_accum(), G_ref) < 1e-9
    w0 = st.flat_params().copy()
    st.step(0.01, 0.9)
    np.testing.assert_allclose(st.flat_params(), w0 - 0.01 * G_ref / M, rtol=0, atol=1e-12)
    np.testing.assert_allclose(st.flat_momentum(), G_ref / M, rtol=0, atol=1e-12)
    assert not st.flat_grad_accum().any()
    # second round: momentum carries over exactly as torch.optim.SGD(momentum) defines it
    opt_w = torch.tensor(w0 - 0.01 * G_ref / M)
    buf = torch.tensor(G_ref / M)
    for m in range(M):
        y = st.forward(m, xs[m])
        Lm, dy = (O.mse_loss(y, tg[m]) if loss == "mse" else O.softmax_xent_loss(y.reshape(B, -1), tg[m]))
        st.backward(m, dy); st.accumulate(m)
    G2 = st.flat_grad_accum().copy()
    st.step(0.01, 0.9)
    buf = 0.9 * buf + torch.tensor(G2 / M)
    np.testing.assert_allclose(st.flat_params(), (opt_w - 0.01 * buf).numpy(), rtol=0, atol=1e-12)


def test_stage_finite_differences():
    net = si.block_net(2, 2)
    first, last, h, w, B = 0, len(net) - 1, 4, 4, 2
    params = (si.init_params(net, first, last, 3) + 0.1 * si.normal(3, 9, (si.param_count(net, first, last),))).astype(np.float64)
    # gamma scaled down so that pre-activations stay away from the ReLU6 kinks
    x = si.normal(3, 1, (B, h, w, 2))
    t = si.normal(3, 2, (B, h, w, 2))

    def loss_of(p, xx):
        st = O.Stage(net, first, last, B, 1, p)
        return O.mse_loss(st.forward(0, xx), t)[0]

    st = O.Stage(net, first, last, B, 1, params)
    y = st.forward(0, x)
    pre_vals = [v for i, v in st.layer_outputs(0).items() if i >= 0 and net[i].op == "bn"]
    margin = min(min(np.abs(v).min(), np.abs(v - 6).min()) for v in pre_vals)
    assert margin > 1e-4
    dx = st.backward(0, O.mse_loss(y, t)[1])
    g = st.flat_micro_grad()
    hstep = 1e-6
    gfd = np.zeros_like(params)
    for i in range(params.size):
        pp, pm = params.copy(), params.copy()
        pp[i] += hstep; pm[i] -= hstep
        gfd[i] = (loss_of(pp, x) - loss_of(pm, x)) / (2 * hstep)
    assert rel(g, gfd) < 1e-6
    dxfd = np.zeros_like(x)
    for i in np.ndindex(*x.shape):
        xp, xm = x.copy(), x.copy()
        xp[i] += hstep; xm[i] -= hstep
        dxfd[i] = (loss_of(params, xp) - loss_of(params, xm)) / (2 * hstep)
    assert rel(dx, dxfd) < 1e-6


@pytest.mark.parametrize("act", ["relu6", "relu"])
def test_accumulated_gradient_equals_full_batch_gradient_without_bn(act):
    net = si.bnfree_net(4, 2, act)
    first, last, h, w, B, M = 0, len(net) - 1, 5, 5, 2, 4
    st, out, xs, tg, params = run_round(net, first, last, h, w, B, M, "mse", seed=5)
    full = O.Stage(net, first, last, B * M, 1, params)
    y = full.forward(0, np.concatenate(xs))
    Lf, dy = O.mse_loss(y, np.concatenate(tg))
    full.backward(0, dy); full.accumulate(0)
    assert rel(st.flat_grad_accum() / M, full.flat_grad_accum()) < 1e-13
    assert abs(np.mean([out[m][2] for m in range(M)]) - Lf) < 1e-13
    st.step(0.01, 0.9); full.step(0.01, 0.9)
    assert rel(st.flat_params(), full.flat_params()) < 1e-14


@pytest.mark.parametrize("shares", [(2, 2), (3, 1), (1, 2, 1)])
def test_group_of_devices_without_bn_reproduces_the_single_device_round(shares):
    """Section 3.2: a group runs the stage data-parallel on shares y_d of every micro-batch and synchronises the gradients
    before the update.  Without BatchNorm the group's update must be the single device's, for equal and unequal shares."""
    net = si.bnfree_net(4, 2, "relu6")
    first, last, h, w, M = 0, len(net) - 1, 5, 5, 3
    B = sum(shares)
    one, out, xs, tg, params = run_round(net, first, last, h, w, B, M, "mse", seed=8)
    one.step(0.05, 0.9)
    group = [O.Stage(net, first, last, y, M, params) for y in shares]
    lo = 0
    for st, y in zip(group, shares):
        for m in range(M):
            ym = st.forward(m, xs[m][lo:lo + y])
            _, dy = O.mse_loss(ym, tg[m][lo:lo + y])
            st.backward(m, dy)
            st.accumulate(m)
        lo += y
    O.group_step(group, shares, 0.05, 0.9)
    for st in group:
        assert rel(st.flat_params(), one.flat_params()) < 1e-13
        assert rel(st.flat_momentum(), one.flat_momentum()) < 1e-13
        assert not st.flat_grad_accum().any()
    # a wrong weighting (plain mean over devices) differs as soon as the shares are unequal
    if len(set(shares)) > 1:
        wrong = [O.Stage(net, first, last, y, M, params) for y in shares]
        lo = 0
        for st, y in zip(wrong, shares):
            for m in range(M):
                _, dy = O.mse_loss(st.forward(m, xs[m][lo:lo + y]), tg[m][lo:lo + y])
                st.backward(m, dy); st.accumulate(m)
            lo += y
        O.group_step(wrong, [1] * len(shares), 0.05, 0.9)
        assert rel(wrong[0].flat_params(), one.flat_params()) > 1e-6


def test_with_bn_single_microbatch_round_is_the_plain_minibatch_step():
    net = si.block_net(4, 2)
    st, out, xs, tg, params = run_round(net, 0, len(net) - 1, 5, 5, 4, 1, "mse", seed=2)
    y, leaves, x = torch_stage(net, 0, len(net) - 1, params, xs[0])
    F.mse_loss(y, torch.tensor(tg[0])).backward()
    assert rel(st.flat_grad_accum(), np.concatenate([t.grad.numpy().ravel() for t in leaves])) < 1e-10


def test_any_legal_interleaving_gives_the_same_update():
    net = si.block_net(4, 2)
    M = 4
    gpipe = [("F", m) for m in range(M)] + [("B", m) for m in range(M)]
    k = O.warmup_forwards(2, 0)        # 3 warm-up forwards, then strict one-forward-one-backward
    f1b = [("F", 0), ("F", 1), ("F", 2), ("B", 0), ("F", 3), ("B", 1), ("B", 2), ("B", 3)]
    assert k == 3
    a = run_round(net, 0, len(net) - 1, 5, 5, 2, M, "mse", seed=4, order=gpipe)[0]
    b = run_round(net, 0, len(net) - 1, 5, 5, 2, M, "mse", seed=4, order=f1b)[0]
    np.testing.assert_array_equal(a.flat_grad_accum(), b.flat_grad_accum())


def test_substage_composition_equals_whole_network():
    """Cutting the layer list into two stages and chaining them (activations forward, input
    gradients backward) reproduces the single-stage result: what a pipeline relies on."""
    net, _ = si.small_mobilenet(10)
    n = len(net)
    cut = si.small_mobilenet(10)[1][2]       # after the second block
    h = w = 16; B = 2
    p_all = si.init_params(net, 0, n - 1, 1)
    x = si.normal(1, 1, (B, h, w, 3)); lab = si.labels(1, 2, B, 10)
    whole = O.Stage(net, 0, n - 1, B, 1, p_all)
    Lw, dl = O.softmax_xent_loss(whole.forward(0, x).reshape(B, -1), lab)
    dxw = whole.backward(0, dl)
    n0 = si.param_count(net, 0, cut)
    s0 = O.Stage(net, 0, cut, B, 1, p_all[:n0])
    s1 = O.Stage(net, cut + 1, n - 1, B, 1, p_all[n0:])
    y0 = s0.forward(0, x)
    L1, dl1 = O.softmax_xent_loss(s1.forward(0, y0).reshape(B, -1), lab)
    dx0 = s0.backward(0, s1.backward(0, dl1))
    assert abs(Lw - L1) < 1e-13
    assert rel(dx0, dxw) < 1e-12
    assert rel(np.concatenate([s0.flat_micro_grad(), s1.flat_micro_grad()]), whole.flat_micro_grad()) < 1e-12


def test_order_errors_and_layout():
    net = si.block_net(4, 2)
    n = si.param_count(net, 0, len(net) - 1)
    with pytest.raises(ValueError):
        O.Stage(net, 0, len(net) - 1, 2, 2, np.zeros(n + 1))
    st = O.Stage(net, 0, len(net) - 1, 2, 2, si.init_params(net, 0, len(net) - 1, 0))
    with pytest.raises(RuntimeError):
        st.step(0.1, 0.9)
    np.testing.assert_array_equal(st.flat_params(), si.init_params(net, 0, len(net) - 1, 0).astype(np.float64))


def test_layer_profile_closed_forms():
    net = si.stage_net_mbv2_4blocks()
    # first expand conv: 56x56x24 -> 56x56x144 at batch 32, bf16
    r = O.layer_profile(net, 0, len(net) - 1, 56, 56, 0, 32, 2)
    assert r == {"a_l": 32 * 56 * 56 * 144 * 2, "w_l": 4 * 144 * 24, "flops": 2 * 32 * 56 * 56 * 144 * 24}
    dw = [i for i, l in enumerate(net) if l.op == "dwconv" and l.stride == 2][0]
    r = O.layer_profile(net, 0, len(net) - 1, 56, 56, dw, 4, 2)
    assert r == {"a_l": 4 * 28 * 28 * 144 * 2, "w_l": 4 * 144 * 9, "flops": 2 * 4 * 28 * 28 * 144 * 9}
