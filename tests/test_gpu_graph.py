"""A whole HPP-Round (Section 3.2: forward x M, backward x M, accumulate, update) captured into a CUDA graph: the stage calls
only enqueue work on the caller's stream (and on the stage's weight-gradient stream, which forks from and joins it), so a
round can be captured once and replayed; replays must leave the same state, bit for bit, as the same rounds issued call by call."""
import numpy as np
import pytest
import torch

import stage_inputs as si

pytestmark = pytest.mark.gpu


def _setup(P, net, h, w, B, M, bf16, seed):
    dev = torch.device("cuda:0")
    last = len(net) - 1
    tdt = torch.bfloat16 if bf16 else torch.float32
    dt = P.AST_BF16 if bf16 else P.AST_F32
    hdl = P.asteroid_stage_create(net, 0, last, h, w, B, M, dtype=dt, slots=0, need_input_grad=1)
    P.asteroid_stage_import_state(hdl, np.ascontiguousarray(si.init_params(net, 0, last, seed), np.float32), None)
    n_out, shp = P.asteroid_stage_output_elems(hdl)
    x = [torch.from_numpy(si.normal(seed, 100000 + m, (B, h, w, net[0].c_in)).astype(np.float32)).to(dev, tdt) for m in range(M)]
    t = [torch.from_numpy(si.normal(seed, 200000 + m, (B,) + shp).astype(np.float32)).to(dev, tdt) for m in range(M)]
    buf = {"y": [torch.empty((B,) + shp, device=dev, dtype=tdt) for _ in range(M)],
           "dy": [torch.empty((B,) + shp, device=dev, dtype=tdt) for _ in range(M)],
           "dx": [torch.empty_like(x[0]) for _ in range(M)],
           "loss": torch.zeros(M, device=dev, dtype=torch.float32)}
    return hdl, dt, n_out, x, t, buf


def _round(P, hdl, dt, n_out, x, t, buf, M, sp):
    for m in range(M):
        P.asteroid_stage_forward(hdl, m, x[m].data_ptr(), buf["y"][m].data_ptr(), sp)
        P.asteroid_loss_mse(buf["y"][m].data_ptr(), t[m].data_ptr(), n_out, dt, buf["dy"][m].data_ptr(), buf["loss"].data_ptr() + 4 * m, sp)
    for m in range(M):
        P.asteroid_stage_backward(hdl, m, buf["dy"][m].data_ptr(), buf["dx"][m].data_ptr(), sp)
        P.asteroid_stage_accumulate(hdl, m, sp)
    P.asteroid_stage_step(hdl, 0.05, 0.9, sp)


def _state(P, hdl):
    n = P.asteroid_stage_param_count(hdl)
    wv, vv = np.empty(n, np.float32), np.empty(n, np.float32)
    P.asteroid_stage_export_state(hdl, params=wv, momentum=vv)
    return wv, vv


@pytest.mark.parametrize("case", ["block_f32", "block_bf16", "bottlenecks_bf16"])
def test_captured_round_replays_to_the_same_state(case):
    import paper_2408_08015_b200 as P
    bf16 = case.endswith("bf16")
    if case.startswith("block"):
        net, h, w, B, M, replays = si.block_net(16, 6), 12, 10, 4, 3, 2
    else:
        # bottleneck blocks with a strided projection shortcut: tensor-core 3x3 kernels, the weight-gradient stream, a
        # device-to-device copy inside the round
        net, h, w, B, M, replays = si.resnet50_c2c3_net(), 16, 16, 2, 2, 2
    # call by call: one round, then `replays` more
    hdl, dt, n_out, x, t, buf = _setup(P, net, h, w, B, M, bf16, seed=5)
    try:
        for _ in range(1 + replays):
            _round(P, hdl, dt, n_out, x, t, buf, M, 0)
        torch.cuda.synchronize()
        ref_w, ref_v = _state(P, hdl)
        ref_y = [v.float().cpu().numpy() for v in buf["y"]]
        ref_loss = buf["loss"].cpu().numpy()
    finally:
        P.asteroid_stage_destroy(hdl)
    # one plain round (first-use set-up happens here), then one captured round replayed `replays` times
    hdl, dt, n_out, x, t, buf = _setup(P, net, h, w, B, M, bf16, seed=5)
    try:
        _round(P, hdl, dt, n_out, x, t, buf, M, 0)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            _round(P, hdl, dt, n_out, x, t, buf, M, torch.cuda.current_stream().cuda_stream)
        for _ in range(replays):
            g.replay()
        torch.cuda.synchronize()
        got_w, got_v = _state(P, hdl)
        np.testing.assert_array_equal(got_w, ref_w)
        np.testing.assert_array_equal(got_v, ref_v)
        for a, b in zip(ref_y, buf["y"]):
            np.testing.assert_array_equal(a, b.float().cpu().numpy())
        np.testing.assert_array_equal(ref_loss, buf["loss"].cpu().numpy())
    finally:
        P.asteroid_stage_destroy(hdl)
