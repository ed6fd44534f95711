"""The allocation-free MSE head against the regular one, through the C ABI.

Some hosts cannot let a library allocate device memory while a round runs: they pre-plan every
byte for a fixed budget, use a pool that forbids cudaMalloc after start-up, or call from a region
where allocation is illegal.  For them the library keeps the loss reduction's scratch in a static
device array.  The variant must produce exactly what the allocating entry point produces, also
when called twice in a row (the shared scratch keeps the previous call's contents)."""
import numpy as np
import pytest

import stage_inputs as si

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bf16", [False, True], ids=["f32", "bf16"])
def test_noalloc_mse_matches_allocating_entry_point_twice(bf16):
    import torch
    import paper_2408_08015_b200 as P
    dev = torch.device("cuda:0")
    tdt = torch.bfloat16 if bf16 else torch.float32
    dt = P.AST_BF16 if bf16 else P.AST_F32
    tol = 2e-2 if bf16 else 1e-4
    for call, n in enumerate((3 * 1000 * 1000 + 17, 777)):          # a many-block case, then a one-block case
        y = torch.from_numpy(si.normal(5, 10 + call, (n,)).astype(np.float32)).to(dev, tdt)
        t = torch.from_numpy(si.normal(5, 20 + call, (n,)).astype(np.float32)).to(dev, tdt)
        dy_a, dy_b = torch.empty_like(y), torch.empty_like(y)
        loss = torch.zeros(2, device=dev, dtype=torch.float32)
        P.asteroid_loss_mse(y.data_ptr(), t.data_ptr(), n, dt, dy_a.data_ptr(), loss.data_ptr())
        P.asteroid_loss_mse_noalloc(y.data_ptr(), t.data_ptr(), n, dt, dy_b.data_ptr(), loss.data_ptr() + 4)
        torch.cuda.synchronize()
        la, lb = loss.cpu().numpy().tolist()
        assert np.isfinite(lb) and abs(la - lb) <= tol * abs(la)
        a, b = dy_a.float().cpu().numpy(), dy_b.float().cpu().numpy()
        assert np.abs(a - b).max() <= tol * np.abs(a).max()
        ref = ((y.double() - t.double()) ** 2).mean().item()        # and both are the mean squared error
        assert abs(lb - ref) <= tol * ref


def test_noalloc_calls_leave_the_free_device_memory_unchanged_and_work_on_a_second_stream():
    import torch
    import paper_2408_08015_b200 as P
    dev = torch.device("cuda:0")
    n = 1 << 20
    y = torch.from_numpy(si.normal(6, 1, (n,)).astype(np.float32)).to(dev)
    t = torch.from_numpy(si.normal(6, 2, (n,)).astype(np.float32)).to(dev)
    dy, loss = torch.empty_like(y), torch.zeros(2, device=dev)
    side = torch.cuda.Stream(device=dev)
    P.asteroid_loss_mse_noalloc(y.data_ptr(), t.data_ptr(), n, P.AST_F32, dy.data_ptr(), loss.data_ptr())     # warm-up: address look-up
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for _ in range(20):
        P.asteroid_loss_mse_noalloc(y.data_ptr(), t.data_ptr(), n, P.AST_F32, dy.data_ptr(), loss.data_ptr())
    torch.cuda.synchronize()
    # a call on another stream once the first stream's calls have finished (the shared ticket word is cleared per call)
    P.asteroid_loss_mse_noalloc(y.data_ptr(), t.data_ptr(), n, P.AST_F32, dy.data_ptr(), loss.data_ptr() + 4, side.cuda_stream)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0            # no allocation by the entry point (torch allocated nothing in between)
    la, lb = loss.cpu().numpy().tolist()
    ref = ((y.double() - t.double()) ** 2).mean().item()
    assert abs(la - ref) <= 1e-5 * ref and la == lb


def test_noalloc_rejects_sizes_beyond_its_limit():
    import torch
    import paper_2408_08015_b200 as P
    buf = torch.zeros(16, device="cuda:0")
    with pytest.raises(P.binding.AsteroidError) as e:
        P.asteroid_loss_mse_noalloc(buf.data_ptr(), buf.data_ptr(), (1 << 26) + 1, P.AST_F32, buf.data_ptr(), buf.data_ptr())
    assert e.value.code == P.AST_ERR_ARG and "limit" in str(e.value)
