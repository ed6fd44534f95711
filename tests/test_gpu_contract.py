"""The C ABI's contract surface on a GPU: every documented error code, the exported BatchNorm running statistics, the
one-forward-one-backward order against the oracle, the activation-memory saving of fewer slots (Eq. (3)), the bounded
device-side wait, and the arena guard bands.  Nothing here faults or hangs the device: errors are refusals taken on
the host before any launch, and the bounded-wait case gives up after 1024 polls and returns."""
import os
import subprocess
import sys

import numpy as np
import pytest

import oracle as O
import stage_inputs as si
from harness import ALL, CONTRACT, MIRROR, bf16_store, compare, gpu_round, make_inputs, oracle_round, summary

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _code(fn, *a, **k):
    import paper_2408_08015_b200 as P
    with pytest.raises(P.binding.AsteroidError) as e:
        fn(*a, **k)
    assert str(e.value).split(":", 1)[1].strip(), "an error must carry a message"
    return e.value.code


def test_order_errors_through_the_abi():
    import torch
    import paper_2408_08015_b200 as P
    net = si.block_net(16, 6)
    B, M, K = 2, 3, 2
    hdl = P.asteroid_stage_create(net, 0, len(net) - 1, 8, 8, B, M, dtype=P.AST_F32, slots=K)
    try:
        P.asteroid_stage_import_state(hdl, si.init_params(net, 0, len(net) - 1, 0))
        x = torch.randn(B, 8, 8, 16, device="cuda:0")
        y, dy, dx = torch.empty_like(x), torch.randn_like(x), torch.empty_like(x)
        fwd = lambda m: P.asteroid_stage_forward(hdl, m, x.data_ptr(), y.data_ptr())
        bwd = lambda m: P.asteroid_stage_backward(hdl, m, dy.data_ptr(), dx.data_ptr())
        assert _code(bwd, 0) == P.AST_ERR_ORDER                          # backward without a resident forward
        assert _code(P.asteroid_stage_step, hdl, 0.01, 0.9) == P.AST_ERR_ORDER     # step before any accumulation
        fwd(0)
        assert _code(fwd, 0) == P.AST_ERR_ORDER                          # forward twice without backward
        fwd(1)
        assert _code(fwd, 2) == P.AST_ERR_ORDER                          # more than `slots` micro-batches resident
        bwd(0)
        assert _code(bwd, 1) == P.AST_ERR_ORDER                          # previous gradients not yet accumulated
        assert _code(P.asteroid_stage_accumulate, hdl, 1) == P.AST_ERR_ORDER       # accumulate of another micro-batch
        P.asteroid_stage_accumulate(hdl, 0)
        assert _code(P.asteroid_stage_accumulate, hdl, 0) == P.AST_ERR_ORDER       # nothing pending
        assert _code(P.asteroid_stage_step, hdl, 0.01, 0.9) == P.AST_ERR_ORDER     # 1 of 3 accumulated
        fwd(2)
        bwd(1); P.asteroid_stage_accumulate(hdl, 1)
        bwd(2); P.asteroid_stage_accumulate(hdl, 2)
        P.asteroid_stage_step(hdl, 0.01, 0.9)                            # the legal sequence still completes
        w = np.empty(P.asteroid_stage_param_count(hdl), np.float32)
        P.asteroid_stage_export_state(hdl, params=w)
        assert np.isfinite(w).all()
    finally:
        P.asteroid_stage_destroy(hdl)


def test_argument_errors_through_the_abi():
    import torch
    import paper_2408_08015_b200 as P
    net = si.block_net(16, 6)
    n = len(net)
    assert _code(P.asteroid_stage_create, net, 3, 2, 8, 8, 2, 2) == P.AST_ERR_ARG            # last < first
    assert _code(P.asteroid_stage_create, net, 0, n, 8, 8, 2, 2) == P.AST_ERR_ARG            # last outside the network
    assert _code(P.asteroid_stage_create, net, 0, n - 1, 0, 8, 2, 2) == P.AST_ERR_ARG        # empty input
    assert _code(P.asteroid_stage_create, net, 0, n - 1, 8, 8, 2, 0) == P.AST_ERR_ARG        # M = 0
    assert _code(P.asteroid_stage_create, net, 0, n - 1, 8, 8, 2, 2, dtype=7) == P.AST_ERR_ARG
    # the residual add of the block reads the block input: a stage that starts after it cannot resolve the reference
    assert _code(P.asteroid_stage_create, net, 3, n - 1, 8, 8, 2, 2) == P.AST_ERR_ARG
    hdl = P.asteroid_stage_create(net, 0, n - 1, 8, 8, 2, 2)
    try:
        params = si.init_params(net, 0, n - 1, 0)
        assert _code(P.asteroid_stage_import_state, hdl, params[:-1].copy()) == P.AST_ERR_ARG
        P.asteroid_stage_import_state(hdl, params)
        x = torch.randn(2, 8, 8, 16, device="cuda:0")
        y = torch.empty_like(x)
        assert _code(P.asteroid_stage_forward, hdl, 2, x.data_ptr(), y.data_ptr()) == P.AST_ERR_ARG      # mb outside [0, M)
        assert _code(P.asteroid_stage_forward, hdl, -1, x.data_ptr(), y.data_ptr()) == P.AST_ERR_ARG
        assert _code(P.asteroid_stage_forward, hdl, 0, None, y.data_ptr()) == P.AST_ERR_ARG
        P.asteroid_stage_forward(hdl, 0, x.data_ptr(), y.data_ptr())
        assert _code(P.asteroid_stage_backward, hdl, 0, y.data_ptr(), None) == P.AST_ERR_ARG             # dx required
        assert _code(P.asteroid_stage_profile, hdl, n, 2) == P.AST_ERR_ARG
        assert _code(P.asteroid_stage_profile, hdl, 0, 0) == P.AST_ERR_ARG
        mean = np.empty(3, np.float32)
        assert _code(P.asteroid_stage_export_bn_running, hdl, mean, mean.copy()) == P.AST_ERR_ARG        # wrong channel count
        buf = torch.zeros(8, device="cuda:0")
        assert _code(P.asteroid_loss_mse, buf.data_ptr(), buf.data_ptr(), 0, P.AST_F32, buf.data_ptr(), buf.data_ptr()) == P.AST_ERR_ARG
        assert _code(P.asteroid_loss_softmax_xent, buf.data_ptr(), buf.data_ptr(), 0, 4, P.AST_F32, buf.data_ptr(), buf.data_ptr()) == P.AST_ERR_ARG
    finally:
        P.asteroid_stage_destroy(hdl)


def test_unsupported_patterns_are_refused():
    import paper_2408_08015_b200 as P
    L = si.Layer
    bn_first = [L("bn", 8, 8, 0, 1, 0, -1, -1), L("conv", 8, 8, 1, 1, 0, 0, -1)]
    assert _code(P.asteroid_stage_create, bn_first, 0, 1, 4, 4, 2, 1) == P.AST_ERR_UNSUPPORTED          # BN with no conv to belong to
    dw9 = [L("dwconv", 8, 8, 9, 1, 4, -1, -1)]
    assert _code(P.asteroid_stage_create, dw9, 0, 0, 8, 8, 2, 1) == P.AST_ERR_UNSUPPORTED                # depthwise is 3x3, 5x5 or 7x7
    dw5_pad = [L("dwconv", 8, 8, 5, 1, 1, -1, -1)]
    assert _code(P.asteroid_stage_create, dw5_pad, 0, 0, 8, 8, 2, 1) == P.AST_ERR_UNSUPPORTED            # ... with "same" padding
    se_wide = [L("conv", 8, 8, 1, 1, 0, -1, -1), L("se", 8, 8, 2000, 1, 0, 0, -1)]
    assert _code(P.asteroid_stage_create, se_wide, 0, 1, 4, 4, 2, 1) == P.AST_ERR_ARG                    # squeeze width out of range
    dw_odd = [L("dwconv", 12, 12, 3, 1, 1, -1, -1)]
    assert _code(P.asteroid_stage_create, dw_odd, 0, 0, 8, 8, 2, 1, dtype=P.AST_BF16) == P.AST_ERR_UNSUPPORTED   # 12 % 8 != 0 in bfloat16
    # a layer that reads the un-normalised conv output from inside a conv-BN-activation chain
    tap = [L("conv", 8, 8, 1, 1, 0, -1, -1), L("bn", 8, 8, 0, 1, 0, 0, -1), L("relu", 8, 8, 0, 1, 0, 1, -1), L("add", 8, 8, 0, 1, 0, 2, 0)]
    assert _code(P.asteroid_stage_create, tap, 0, 3, 4, 4, 2, 1) == P.AST_ERR_UNSUPPORTED
    relu6_after_add = [L("conv", 8, 8, 1, 1, 0, -1, -1), L("add", 8, 8, 0, 1, 0, 0, -1), L("relu6", 8, 8, 0, 1, 0, 1, -1)]
    assert _code(P.asteroid_stage_create, relu6_after_add, 0, 2, 4, 4, 2, 1) == P.AST_ERR_UNSUPPORTED
    lin = [L("linear", 8, 4, 0, 1, 0, -1, -1)]
    assert _code(P.asteroid_stage_create, lin, 0, 0, 4, 4, 2, 1) == P.AST_ERR_UNSUPPORTED                # linear needs a pooled input


def test_bn_running_statistics_match_the_oracle_after_two_forwards():
    import torch
    import paper_2408_08015_b200 as P
    net = si.block_net(16, 6)
    first, last, h, w, B, M = 0, len(net) - 1, 12, 12, 4, 2
    xs, tg, params, _ = make_inputs(net, first, last, h, w, B, M, "mse", 4, False)
    params = si.randomize_bn(params, net, first, last, 4)
    st = O.Stage(net, first, last, B, M, params)
    for m in range(M):
        st.forward(m, xs[m])
    ref_mean = np.concatenate([st.running[i][0] for i in sorted(st.running)])
    ref_var = np.concatenate([st.running[i][1] for i in sorted(st.running)])
    hdl = P.asteroid_stage_create(net, first, last, h, w, B, M)
    try:
        P.asteroid_stage_import_state(hdl, params)
        y = torch.empty(B, h, w, 16, device="cuda:0")
        for m in range(M):
            x = torch.from_numpy(xs[m]).cuda()
            P.asteroid_stage_forward(hdl, m, x.data_ptr(), y.data_ptr())
        mean, var = np.empty(ref_mean.size, np.float32), np.empty(ref_var.size, np.float32)
        P.asteroid_stage_export_bn_running(hdl, mean, var)
    finally:
        P.asteroid_stage_destroy(hdl)
    assert np.abs(mean - ref_mean).max() <= 1e-5 * max(np.abs(ref_mean).max(), 1.0)
    assert np.abs(var - ref_var).max() <= 1e-5 * np.abs(ref_var).max()
    assert np.abs(ref_mean).max() > 1e-3 and np.abs(ref_var - 1).max() > 1e-3      # the statistics really moved


def test_one_forward_one_backward_order_against_the_oracle_in_bf16_and_its_memory_saving():
    """Section 3.2: stage p of P keeps K_p = 2(P-p)-1 micro-batches resident instead of M.  The same legal interleaving
    is handed to the oracle and to the library (bfloat16, one inverted-residual block of the MobileNetV2 stage at
    56x56); Eq. (3) gives the memory the smaller K saves."""
    import torch
    import paper_2408_08015_b200 as P
    net = si.block_net(24, 6)
    first, last, h, w, B, M = 0, len(net) - 1, 56, 56, 8, 6
    K = O.warmup_forwards(3, 1)                  # the middle stage of three: 3 resident micro-batches
    assert K == 3
    order = [("F", 0), ("F", 1), ("F", 2), ("B", 0), ("F", 3), ("B", 1), ("F", 4), ("B", 2), ("F", 5), ("B", 3), ("B", 4), ("B", 5)]
    xs, tg, params, _ = make_inputs(net, first, last, h, w, B, M, "mse", 2, True)
    plain = oracle_round(net, first, last, B, M, "mse", xs, tg, params, order=order)
    mirror = oracle_round(net, first, last, B, M, "mse", xs, tg, params, order=order, store=bf16_store)
    free0 = torch.cuda.mem_get_info()[0]
    gpu = gpu_round(net, first, last, h, w, B, M, "mse", xs, tg, params, True, order=order, slots=K)
    r = compare(gpu, plain, net, first, last, 2e-2, mirror=mirror, allow=(CONTRACT, MIRROR), outlier_frac=1e-4, case="f1b/block24/bf16")
    print(summary(r))
    full = gpu_round(net, first, last, h, w, B, M, "mse", xs, tg, params, True)        # all M resident, GPipe order
    assert np.array_equal(full["G"], gpu["G"]) and np.array_equal(full["w"], gpu["w"])
    # Eq. (3): Mem = MOD + OPT + K * ACT
    hdl = P.asteroid_stage_create(net, first, last, h, w, B, M, dtype=P.AST_BF16, slots=K)
    try:
        free_k = torch.cuda.mem_get_info()[0]
        rec = P.asteroid_stage_profile(hdl, first, B)
    finally:
        P.asteroid_stage_destroy(hdl)
    mem_k = O.stage_memory(rec["mem_mod"], rec["mem_opt"], rec["mem_act"], K)
    mem_m = O.stage_memory(rec["mem_mod"], rec["mem_opt"], rec["mem_act"], M)
    saving = mem_m - mem_k
    assert saving == (M - K) * rec["mem_act"] and saving > 0
    hdl = P.asteroid_stage_create(net, first, last, h, w, B, M, dtype=P.AST_BF16, slots=M)
    try:
        free_m = torch.cuda.mem_get_info()[0]
    finally:
        P.asteroid_stage_destroy(hdl)
    measured = free_k - free_m                                   # device memory the extra M-K slots took
    print("Eq.(3): K=%d of M=%d saves %.1f MB of %.1f MB (%.0f%%); device allocation differs by %.1f MB"
          % (K, M, saving / 2**20, (mem_m + rec["mem_work"]) / 2**20, 100.0 * saving / (mem_m + rec["mem_work"]), measured / 2**20))
    assert abs(measured - saving) <= 4 << 20
    del free0


def test_bounded_wait_gives_up_and_leaves_the_context_usable():
    import torch
    import paper_2408_08015_b200 as P
    assert P.asteroid_selftest_bounded_wait() == P.AST_ERR_TIMEOUT
    assert "wait" in P.asteroid_last_error()
    a = torch.arange(1000, device="cuda:0").sum().item()         # the context still works
    assert a == 499500
    net = si.block_net(16, 6)
    xs, tg, params, _ = make_inputs(net, 0, len(net) - 1, 8, 8, 2, 1, "mse", 0, True)
    out = gpu_round(net, 0, len(net) - 1, 8, 8, 2, 1, "mse", xs, tg, params, True)
    assert np.isfinite(out["w"]).all()


def test_arena_guard_bands_are_intact_after_ragged_rounds():
    """Runs ragged and full-tile rounds of every kernel family in a child process that has ASTEROID_CHECK_GUARDS=1: export_state
    then verifies the guard bands on both sides of every arena of the stage (the host-side stand-in for a memory checker)."""
    code = r'''
import sys
sys.path.insert(0, %r); sys.path.insert(0, %r)
import numpy as np, stage_inputs as si
from harness import gpu_round, make_inputs
cases = [(si.block_net(8, 3), 7, 5, 3, 2, "mse"), (si.stage_net_mbv2_4blocks(), 14, 14, 3, 2, "mse"),
         (si.bottleneck_net(64, [(64, 128, 1, 2)]), 9, 7, 2, 2, "mse"), (si.bottleneck_net(128, [(128, 128, 2, 1)]), 7, 12, 2, 1, "mse"),
         (si.small_mobilenet(10)[0], 32, 32, 4, 2, "xent"), (si.single_unit_net("conv", 512, 128, bn=True), 29, 27, 3, 1, "mse"),
         (si.single_unit_net("conv", 3, 32, k=3, stride=2, bn=True), 63, 65, 3, 2, "mse")]
for net, h, w, B, M, loss in cases:
    for bf16 in (False, True):
        xs, tg, params, _ = make_inputs(net, 0, len(net) - 1, h, w, B, M, loss, 0, bf16)
        out = gpu_round(net, 0, len(net) - 1, h, w, B, M, loss, xs, tg, params, bf16)     # export_state checks the guards
        assert np.isfinite(out["w"]).all()
print("guards ok")
''' % (ROOT, os.path.join(ROOT, "tests"))
    env = dict(os.environ, ASTEROID_CHECK_GUARDS="1")
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0 and "guards ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]
