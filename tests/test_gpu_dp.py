"""Intra-group data parallelism (Section 3.2, Eq. 5) on one GPU: the gradient arena as a torch view, the weighted
AllReduce through a one-rank NCCL group, and a two-replica group run one replica after the other whose synchronised update
is the oracle's `group_step`."""
import os

import numpy as np
import pytest
import torch

import stage_inputs as si
import harness as H

pytestmark = pytest.mark.gpu


def _replica(P, net, h, w, y, M, params, xs, tg, lo):
    """Forward, loss, backward and accumulation of M micro-batch shares on a fresh replica; returns its handle."""
    dev = torch.device("cuda:0")
    last = len(net) - 1
    hdl = P.asteroid_stage_create(net, 0, last, h, w, y, M, dtype=P.AST_F32, slots=0, need_input_grad=1)
    P.asteroid_stage_import_state(hdl, np.ascontiguousarray(params, np.float32), None)
    n_out, shp = P.asteroid_stage_output_elems(hdl)
    keep = []
    for m in range(M):
        x = torch.from_numpy(np.ascontiguousarray(xs[m][lo:lo + y], np.float32)).to(dev)
        t = torch.from_numpy(np.ascontiguousarray(tg[m][lo:lo + y], np.float32)).to(dev)
        yv, dy, dx = torch.empty((y,) + shp, device=dev), torch.empty((y,) + shp, device=dev), torch.empty_like(x)
        ls = torch.zeros(1, device=dev)
        P.asteroid_stage_forward(hdl, m, x.data_ptr(), yv.data_ptr(), 0)
        P.asteroid_loss_mse(yv.data_ptr(), t.data_ptr(), n_out, P.AST_F32, dy.data_ptr(), ls.data_ptr(), 0)
        P.asteroid_stage_backward(hdl, m, dy.data_ptr(), dx.data_ptr(), 0)
        P.asteroid_stage_accumulate(hdl, m, 0)
        keep += [x, t, yv, dy, dx, ls]
    torch.cuda.synchronize()
    return hdl


def _case(shares):
    net = si.bnfree_net(8, 2, "relu6")
    last = len(net) - 1
    B, M, h, w, seed = sum(shares), 2, 6, 6, 11
    n = si.param_count(net, 0, last)
    params = (si.init_params(net, 0, last, seed) + 0.05 * si.normal(seed, 7, (n,)).astype(np.float32)).astype(np.float32)
    shp = si.out_shape(net, 0, last, h, w)[last]
    xs = [si.normal(seed, 100000 + m, (B, h, w, net[0].c_in)).astype(np.float32) for m in range(M)]
    tg = [si.normal(seed, 200000 + m, (B,) + shp).astype(np.float32) for m in range(M)]
    return net, params, xs, tg, B, M, h, w, n


def test_gradient_arena_view_is_the_exported_gradient():
    import paper_2408_08015_b200 as P
    from paper_2408_08015_b200 import dp
    net, params, xs, tg, B, M, h, w, n = _case((3, 2))
    hdl = _replica(P, net, h, w, B, M, params, xs, tg, 0)
    try:
        G = np.empty(n, np.float32)
        P.asteroid_stage_export_state(hdl, grad_accum=G)
        t = dp.grad_tensor(hdl)
        assert t.is_cuda and t.dtype == torch.float32 and t.numel() >= n
        # the arena holds every exported value (its order and padding are the library's own)
        a = np.sort(t.cpu().numpy()[t.cpu().numpy() != 0])
        b = np.sort(G[G != 0])
        np.testing.assert_array_equal(a, b)
        # a change through the view is a change of the stage's accumulated gradient
        t.mul_(0.5)
        torch.cuda.synchronize()
        G2 = np.empty(n, np.float32)
        P.asteroid_stage_export_state(hdl, grad_accum=G2)
        np.testing.assert_array_equal(G2, 0.5 * G)
    finally:
        P.asteroid_stage_destroy(hdl)


def test_one_rank_nccl_group_scales_by_the_share():
    import torch.distributed as dist
    import paper_2408_08015_b200 as P
    from paper_2408_08015_b200 import dp
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(30500 + os.getpid() % 2000), RANK="0", WORLD_SIZE="1")
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1)
    net, params, xs, tg, B, M, h, w, n = _case((4, 4))
    hdl = _replica(P, net, h, w, B, M, params, xs, tg, 0)
    try:
        G = np.empty(n, np.float32)
        P.asteroid_stage_export_state(hdl, grad_accum=G)
        dp.allreduce_gradients(hdl, B, B)            # the whole micro-batch on the only rank: unchanged
        torch.cuda.synchronize()
        G1 = np.empty(n, np.float32)
        P.asteroid_stage_export_state(hdl, grad_accum=G1)
        np.testing.assert_array_equal(G1, G)
        dp.allreduce_gradients(hdl, B // 4, B)       # a quarter share: scaled by 1/4 (exact in binary)
        torch.cuda.synchronize()
        P.asteroid_stage_export_state(hdl, grad_accum=G1)
        np.testing.assert_array_equal(G1, 0.25 * G)
        P.asteroid_stage_step(hdl, 0.05, 0.9, 0)                 # the update accepts the synchronised arena
        torch.cuda.synchronize()
    finally:
        P.asteroid_stage_destroy(hdl)
        dist.destroy_process_group()


@pytest.mark.parametrize("shares", [(4, 4), (5, 3)])
def test_two_replicas_synchronised_update_is_the_oracle_group_step(shares):
    import oracle as O
    import paper_2408_08015_b200 as P
    from paper_2408_08015_b200 import dp
    net, params, xs, tg, B, M, h, w, n = _case(shares)
    last = len(net) - 1
    lr, mu = 0.05, 0.9
    # oracle: the group, and the single device it must reproduce
    group, lo = [], 0
    for y in shares:
        st = O.Stage(net, 0, last, y, M, params)
        for m in range(M):
            _, dy = O.mse_loss(st.forward(m, xs[m][lo:lo + y]), tg[m][lo:lo + y])
            st.backward(m, dy)
            st.accumulate(m)
        group.append(st)
        lo += y
    O.group_step(group, shares, lr, mu)
    # library: the two replicas run one after the other; the group sum is taken over their arena views
    hs, lo = [], 0
    for y in shares:
        hs.append(_replica(P, net, h, w, y, M, params, xs, tg, lo))
        lo += y
    try:
        ts = [dp.grad_tensor(hd) for hd in hs]
        total = sum(t * (float(y) / B) for t, y in zip(ts, shares))
        for t in ts:
            t.copy_(total)
        for hd in hs:
            P.asteroid_stage_step(hd, lr, mu, 0)
        torch.cuda.synchronize()
        got = []
        for hd in hs:
            wv, vv = np.empty(n, np.float32), np.empty(n, np.float32)
            P.asteroid_stage_export_state(hd, params=wv, momentum=vv)
            got.append((wv, vv))
        np.testing.assert_array_equal(got[0][0], got[1][0])           # replicas stay identical
        np.testing.assert_array_equal(got[0][1], got[1][1])
        assert H.rel_err(got[0][0], group[0].flat_params()) < 1e-4    # float32 storage tolerance of the parity tests
        assert H.rel_err(got[0][1], group[0].flat_momentum()) < 1e-4
    finally:
        for hd in hs:
            P.asteroid_stage_destroy(hd)
