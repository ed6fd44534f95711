"""Host side of the intra-group data parallelism (Section 3.2, Eq. 5) on CPU: the share split, and two gloo ranks whose
weighted AllReduce of the accumulated gradients gives the single-device gradient of a BatchNorm-free stage."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2408_08015_b200 import dp  # noqa: E402


@pytest.mark.parametrize("batch,weights", [(32, [1, 1]), (32, [3, 1]), (7, [1, 1, 1]), (5, [10, 1, 1]), (2, [1, 5, 1]), (0, [1, 2]),
                                           (33, [1.0 / 12.5, 1.0 / 31.0, 1.0 / 31.0, 1.0 / 97.0])])
def test_group_shares_are_a_proportional_integer_split(batch, weights):
    y = dp.group_shares(batch, weights)
    assert sum(y) == batch and len(y) == len(weights)
    assert all(isinstance(v, int) and v >= 0 for v in y)
    if batch >= len(weights):
        assert min(y) >= 1
        # a share differs from the exact proportion by less than one sample per device that was lifted to the minimum
        tot = float(sum(weights))
        for v, w in zip(y, weights):
            assert abs(v - batch * w / tot) < 1 + len(weights)
    # a faster device never gets fewer samples than a slower one
    for i in range(len(weights)):
        for j in range(len(weights)):
            if weights[i] > weights[j]:
                assert y[i] >= y[j]


def test_group_shares_reject_bad_weights():
    with pytest.raises(ValueError):
        dp.group_shares(8, [1, 0])
    with pytest.raises(ValueError):
        dp.group_shares(8, [])


def _round_on_share(net, params, xs, tg, lo, y, M):
    import oracle as O
    st = O.Stage(net, 0, len(net) - 1, y, M, params)
    for m in range(M):
        out = st.forward(m, xs[m][lo:lo + y])
        _, dy = O.mse_loss(out, tg[m][lo:lo + y])
        st.backward(m, dy)
        st.accumulate(m)
    return st


def _case(shares):
    import stage_inputs as si
    net = si.bnfree_net(4, 2, "relu6")
    B, M, h, w, seed = sum(shares), 3, 5, 5, 8
    n = si.param_count(net, 0, len(net) - 1)
    params = si.init_params(net, 0, len(net) - 1, seed) + 0.05 * si.normal(seed, 7, (n,)).astype(np.float32)
    shp = si.out_shape(net, 0, len(net) - 1, h, w)[len(net) - 1]
    xs = [si.normal(seed, 100000 + m, (B, h, w, net[0].c_in)) for m in range(M)]
    tg = [si.normal(seed, 200000 + m, (B,) + shp) for m in range(M)]
    return net, params, xs, tg, B, M


def _worker(rank, world, port, shares, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    net, params, xs, tg, B, M = _case(shares)
    st = _round_on_share(net, params, xs, tg, sum(shares[:rank]), shares[rank], M)
    t = torch.from_numpy(st.flat_grad_accum().copy())
    dp.allreduce_weighted(t, shares[rank], B)
    q.put((rank, t.numpy().copy()))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("shares", [(4, 4), (6, 2)])
def test_two_ranks_synchronise_to_the_single_device_gradient(shares):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000 + shares[0]
    procs = [ctx.Process(target=_worker, args=(r, 2, port, shares, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    net, params, xs, tg, B, M = _case(shares)
    one = _round_on_share(net, params, xs, tg, 0, B, M).flat_grad_accum()
    np.testing.assert_array_equal(res[0], res[1])                     # every replica holds the same synchronised gradient
    assert np.abs(res[0] - one).max() <= 1e-12 * np.abs(one).max()
