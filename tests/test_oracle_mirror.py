"""Pins of the oracle's storage-mirroring mode (`Stage(store=, operand=)`), the diagnostic mode that
rounds where a bfloat16 implementation keeps tensors in memory and at the inputs of dense contractions.

The mode changes no formula; it only inserts a rounding function at a fixed set of places.  The pins fix
that set: the identity function gives the plain result bit for bit; a recording function sees exactly the
hand-written list of tensors, in order; with a rounding function whose range is a coarse grid, the tensors
on the list lie on the grid and the tensors inside a conv-BN-activation chain do not; and the operand rounding
reaches a brute-force convolution of the rounded operands."""
import numpy as np

import oracle as O
import stage_inputs as si
from test_oracle_layers import brute_conv, brute_conv_grads


def _round(net, first, last, h, w, B, M, loss, seed, **kw):
    c_in = net[first].c_in
    shp = si.out_shape(net, first, last, h, w)[last]
    params = si.init_params(net, first, last, seed)
    st = O.Stage(net, first, last, B, M, params, **kw)
    out = []
    for m in range(M):
        x = si.normal(seed, 100000 + m, (B, h, w, c_in))
        y = st.forward(m, x)
        if loss == "mse":
            _, dy = O.mse_loss(y, si.normal(seed, 200000 + m, (B,) + shp))
        else:
            _, dy = O.softmax_xent_loss(y.reshape(B, -1), si.labels(seed, 300000 + m, B, shp[2]))
        out.append((y, st.backward(m, dy)))
        st.accumulate(m)
    G = st.flat_grad_accum().copy()
    st.step(0.01, 0.9)
    return st, out, G


def test_identity_rounding_is_the_plain_oracle_bit_for_bit():
    ident = lambda t: t
    for net, h, w, loss in ((si.stage_net_mbv2_4blocks(), 8, 8, "mse"), (si.bottleneck_net(4, [(2, 8, 2, 1), (4, 16, 2, 2)]), 8, 8, "mse"),
                            (si.small_mobilenet(10)[0], 16, 16, "xent")):
        a, oa, Ga = _round(net, 0, len(net) - 1, h, w, 2, 2, loss, 3)
        b, ob, Gb = _round(net, 0, len(net) - 1, h, w, 2, 2, loss, 3, store=ident, operand=ident)
        assert np.array_equal(Ga, Gb) and np.array_equal(a.flat_params(), b.flat_params())
        for (ya, dxa), (yb, dxb) in zip(oa, ob):
            assert np.array_equal(ya, yb) and np.array_equal(dxa, dxb)


def test_stored_forward_layers_equal_the_hand_written_lists():
    # config 2: blocks of conv,bn,relu6, dw,bn,relu6, conv,bn,[add]; layers 0-8, 9-17, 18-25 (stride 2, no add), 26-34.
    # Stored: every conv / depthwise output (raw, before its BatchNorm), every residual sum, the stage output.
    net = si.stage_net_mbv2_4blocks()
    st = O.Stage(net, 0, len(net) - 1, 1, 1, si.init_params(net, 0, len(net) - 1, 0), store=lambda t: t)
    assert [i for i in range(len(net)) if st._stored_forward(i)] == [0, 3, 6, 8, 9, 12, 15, 17, 18, 21, 24, 26, 29, 32, 34]
    # the same network cut after block 2: its last layer (a BatchNorm) is the stage output and therefore stored
    st = O.Stage(net, 0, 25, 1, 1, si.init_params(net, 0, 25, 0), store=lambda t: t)
    assert [i for i in range(26) if st._stored_forward(i)] == [0, 3, 6, 8, 9, 12, 15, 17, 18, 21, 24, 25]
    # config 4: first bottleneck of a group = conv,bn,relu, conv,bn,relu, conv,bn, conv(shortcut),bn, add,relu (12 layers),
    # the others = conv,bn,relu, conv,bn,relu, conv,bn, add,relu (10 layers).  Stored: conv outputs and the ReLU after each add.
    net = si.resnet50_c2c3_net()
    st = O.Stage(net, 0, len(net) - 1, 1, 1, si.init_params(net, 0, len(net) - 1, 0), store=lambda t: t)
    expect, base = [], 0
    for first_of_group in (True, False, False, True, False, False, False):
        expect += [base + 0, base + 3, base + 6] + ([base + 8, base + 11] if first_of_group else [base + 9])
        base += 12 if first_of_group else 10
    assert base == len(net)
    assert [i for i in range(len(net)) if st._stored_forward(i)] == expect
    # classifier head: conv, bn, relu6, gap, linear -> conv output, pooled features, logits
    net = si.head_net(8, 5, bn_conv=16)
    st = O.Stage(net, 0, len(net) - 1, 1, 1, si.init_params(net, 0, len(net) - 1, 0), store=lambda t: t)
    assert [i for i in range(len(net)) if st._stored_forward(i)] == [0, 2, 3]


def test_recording_store_sees_the_hand_written_sequence_of_tensors():
    """One inverted-residual block 4 -> 12 -> 4 with residual (layers: 0 conv, 1 bn, 2 relu6, 3 dw, 4 bn, 5 relu6,
    6 conv, 7 bn, 8 add) at 5x5, micro-batch 2."""
    net = si.block_net(4, 3)
    calls = []

    def rec(t):
        calls.append(np.asarray(t).shape)
        return t

    st = O.Stage(net, 0, 8, 2, 1, si.init_params(net, 0, 8, 0), store=rec)
    y = st.forward(0, si.normal(0, 1, (2, 5, 5, 4)))
    # forward: z of the expand conv, z of the depthwise conv, z of the project conv, the residual sum (stage output)
    assert calls == [(2, 5, 5, 12), (2, 5, 5, 12), (2, 5, 5, 4), (2, 5, 5, 4)]
    del calls[:]
    st.backward(0, np.ones_like(y))
    # backward, in reverse layer order; a gradient is stored where it is the gradient of a unit's output value:
    #   add      -> gradient of the project unit's output (layer 7) and first term of the block input's gradient
    #   bn 7     -> dz of the project conv: consumed while loading, not stored
    #   conv 6   -> gradient of the depthwise unit's output (layer 5, after BN + ReLU6)
    #   relu6 5, bn 4 -> inside the chain: not stored
    #   dw 3     -> gradient of the expand unit's output (layer 2)
    #   relu6 2, bn 1 -> not stored
    #   conv 0   -> second term added to the block input's gradient, rounded again after the addition
    assert calls == [(2, 5, 5, 4), (2, 5, 5, 4), (2, 5, 5, 12), (2, 5, 5, 12), (2, 5, 5, 4)]


def test_grid_rounding_puts_exactly_the_stored_tensors_on_the_grid():
    q = 2.0 ** -5
    grid = lambda t: np.round(np.asarray(t, np.float64) / q) * q
    on_grid = lambda t: bool(np.all(t == grid(t)))
    net = si.bottleneck_net(4, [(2, 8, 2, 1)])
    first, last = 0, len(net) - 1
    st = O.Stage(net, first, last, 2, 1, si.init_params(net, first, last, 1), store=grid)
    st.forward(0, si.normal(1, 7, (2, 6, 6, 4)))
    val = st.layer_outputs(0)
    for i in range(first, last + 1):
        assert on_grid(val[i]) == st._stored_forward(i), (i, net[i].op)
    # stored values feed the next layer as stored: the second conv's output is a function of the rounded first conv output
    z0 = val[0]
    y1, _ = O.bn_forward(z0, st.p[(1, "gamma")], st.p[(1, "beta")], 1e-5)
    assert np.array_equal(val[3], grid(O.conv2d_forward(O.act_forward("relu", y1), st.p[(3, "weight")], 1, 1)))
    # the input gradient is stored, hence on the grid
    dx = st.backward(0, si.normal(1, 8, val[last].shape))
    assert on_grid(dx)


def test_operand_rounding_reaches_a_brute_force_conv_of_the_rounded_operands():
    q = 2.0 ** -4
    grid = lambda t: np.round(np.asarray(t, np.float64) / q) * q
    net = si.single_unit_net("conv", 3, 5, k=3, stride=2)
    params = si.init_params(net, 0, 0, 2).astype(np.float64) * 4.0
    st = O.Stage(net, 0, 0, 2, 1, params, operand=grid)
    x = si.normal(2, 1, (2, 7, 6, 3))
    y = st.forward(0, x)
    w = params.reshape(5, 3, 3, 3)
    assert np.allclose(y, brute_conv(grid(x), grid(w), 2, 1), rtol=0, atol=1e-12)
    assert not np.allclose(y, brute_conv(x, w, 2, 1), rtol=0, atol=1e-3)      # the rounding is really there
    dy = si.normal(2, 2, y.shape)
    dx = st.backward(0, dy)
    bdx, bdw = brute_conv_grads(grid(x), grid(w), grid(dy), 2, 1)
    assert np.allclose(dx, bdx, rtol=0, atol=1e-12) and np.allclose(st.flat_micro_grad(), bdw.ravel(), rtol=0, atol=1e-12)
    # the depthwise conv is not a dense contraction: its operands stay unrounded
    net = si.single_unit_net("dwconv", 4, 4)
    a = O.Stage(net, 0, 0, 1, 1, si.init_params(net, 0, 0, 2), operand=grid)
    b = O.Stage(net, 0, 0, 1, 1, si.init_params(net, 0, 0, 2))
    x = si.normal(2, 3, (1, 5, 5, 4))
    assert np.array_equal(a.forward(0, x), b.forward(0, x))
