"""Shared test harness: run one HPP-Round on the oracle and on the CUDA library from the same
seeded inputs, and compare tensor by tensor.  Imported by tests and the smoke check only."""
import numpy as np

import stage_inputs as si


def make_inputs(net, first, last, h, w, B, M, loss, seed, bf16):
    c_in = net[first].c_in
    shp = si.out_shape(net, first, last, h, w)[last]
    cast = si.round_to_bf16 if bf16 else (lambda a: a)
    xs = [cast(si.normal(seed, 100000 + m, (B, h, w, c_in)).astype(np.float32)) for m in range(M)]
    if loss == "mse":
        tg = [cast(si.normal(seed, 200000 + m, (B,) + shp).astype(np.float32)) for m in range(M)]
    else:
        tg = [si.labels(seed, 300000 + m, B, shp[2]) for m in range(M)]
    params = si.init_params(net, first, last, seed)
    return xs, tg, params, shp


def default_order(M):
    return [("F", m) for m in range(M)] + [("B", m) for m in range(M)]


def bf16_store(a):
    """Rounding applied at storage points, and to the operands of dense contractions, when mirroring
    bfloat16 activation storage with bfloat16 tensor-core inputs."""
    return si.round_to_bf16(np.asarray(a, np.float32)).astype(np.float64)


def oracle_round(net, first, last, B, M, loss, xs, tg, params, lr=0.01, mu=0.9, order=None, momentum0=None, rounds=1,
                 store=None):
    import oracle as O
    st = O.Stage(net, first, last, B, M, params, store=store, operand=store)
    if momentum0 is not None:
        off = 0
        for k in st.v:
            n = st.v[k].size
            st.v[k] = np.asarray(momentum0[off:off + n], dtype=np.float64).reshape(st.v[k].shape)
            off += n
    res = None
    for _ in range(rounds):
        ys, out = {}, {}
        for kind, m in (order or default_order(M)):
            if kind == "F":
                ys[m] = st.forward(m, xs[m])
            else:
                if loss == "mse":
                    Lm, dy = O.mse_loss(ys[m], tg[m])
                else:
                    Lm, dy = O.softmax_xent_loss(ys[m].reshape(B, -1), tg[m])
                if store is not None:
                    dy = store(dy)
                dx = st.backward(m, dy)
                st.accumulate(m)
                out[m] = (ys[m], dx, Lm)
        G = st.flat_grad_accum().copy()
        st.step(lr, mu)
        res = {"y": [out[m][0] for m in range(M)], "dx": [out[m][1] for m in range(M)],
               "loss": [out[m][2] for m in range(M)], "G": G, "w": st.flat_params().copy(), "v": st.flat_momentum().copy()}
    return res


def gpu_round(net, first, last, h, w, B, M, loss, xs, tg, params, bf16, lr=0.01, mu=0.9, order=None,
              slots=0, need_dx=1, momentum0=None, rounds=1, stream=None, export_micro=False):
    import torch
    import paper_2408_08015_b200 as P
    dev = torch.device("cuda:0")
    tdt = torch.bfloat16 if bf16 else torch.float32
    dt = P.AST_BF16 if bf16 else P.AST_F32
    hdl = P.asteroid_stage_create(net, first, last, h, w, B, M, dtype=dt, slots=slots, need_input_grad=need_dx)
    try:
        P.asteroid_stage_import_state(hdl, np.ascontiguousarray(params, np.float32),
                                      None if momentum0 is None else np.ascontiguousarray(momentum0, np.float32))
        n_out, shp = P.asteroid_stage_output_elems(hdl)
        xd = [torch.from_numpy(x).to(dev, tdt).contiguous() for x in xs]
        if loss == "mse":
            td = [torch.from_numpy(t).to(dev, tdt).contiguous() for t in tg]
        else:
            td = [torch.from_numpy(np.asarray(t, np.int32)).to(dev) for t in tg]
        yd = [torch.empty((B,) + shp, device=dev, dtype=tdt) for _ in range(M)]
        dyd = [torch.empty((B,) + shp, device=dev, dtype=tdt) for _ in range(M)]
        dxd = [torch.zeros_like(x) for x in xd]
        lossd = torch.zeros(M, device=dev, dtype=torch.float32)
        sp = 0 if stream is None else stream.cuda_stream
        torch.cuda.synchronize()
        micro = {}
        for _ in range(rounds):
            for kind, m in (order or default_order(M)):
                if kind == "F":
                    P.asteroid_stage_forward(hdl, m, xd[m].data_ptr(), yd[m].data_ptr(), sp)
                else:
                    lp = lossd.data_ptr() + 4 * m
                    if loss == "mse":
                        P.asteroid_loss_mse(yd[m].data_ptr(), td[m].data_ptr(), n_out, dt, dyd[m].data_ptr(), lp, sp)
                    else:
                        P.asteroid_loss_softmax_xent(yd[m].data_ptr(), td[m].data_ptr(), B, shp[2], dt, dyd[m].data_ptr(), lp, sp)
                    P.asteroid_stage_backward(hdl, m, dyd[m].data_ptr(), dxd[m].data_ptr() if need_dx else None, sp)
                    if export_micro:
                        gm = np.empty(P.asteroid_stage_param_count(hdl), np.float32)
                        P.asteroid_stage_export_state(hdl, micro_grad=gm)
                        micro[m] = gm
                    P.asteroid_stage_accumulate(hdl, m, sp)
            n = P.asteroid_stage_param_count(hdl)
            G = np.empty(n, np.float32)
            P.asteroid_stage_export_state(hdl, grad_accum=G)
            P.asteroid_stage_step(hdl, lr, mu, sp)
        wv, vv = np.empty(n, np.float32), np.empty(n, np.float32)
        P.asteroid_stage_export_state(hdl, params=wv, momentum=vv)
        torch.cuda.synchronize()
        return {"y": [t.float().cpu().numpy() for t in yd], "dx": [t.float().cpu().numpy() for t in dxd],
                "loss": lossd.cpu().numpy().tolist(), "G": G, "w": wv, "v": vv, "g": micro}
    finally:
        P.asteroid_stage_destroy(hdl)


def rel_err(a, b, floor=0.0):
    a = np.asarray(a, np.float64).ravel()
    b = np.asarray(b, np.float64).ravel()
    return float(np.abs(a - b).max() / max(np.abs(b).max(), floor, 1e-300))


def compare(gpu, ref, net, first, last, tol, need_dx=True, outlier_frac=0.0, outlier_cap=0.25, pure=None):
    """Per tensor (every y_m, dx_m, loss_m; accumulated gradient, momentum and weights per
    parameter tensor, denominators floored at 1% of the largest entry of their kind so that a
    tensor whose true value vanishes is judged on the scale of its siblings):

      primary    max|gpu-ref| / max|ref| <= tol, where up to `outlier_frac` of the elements may
                 exceed tol (never `outlier_cap`): a pre-activation within float rounding of a
                 ReLU/ReLU6 kink takes a different mask on the two sides.
      calibrated (only if `pure`, the plain float64 result, is given and the primary test
                 fails): with bfloat16 storage one-ulp differences between two correct
                 implementations multiply through the layers and flip masks, so deep stages
                 cannot agree element-wise on gradients.  Then the library must be no further
                 from the exact result than the storage format itself puts a float64
                 implementation: max-norm error vs `pure` <= 2x, and L2 error <= 1.5x, that of
                 `ref` (the float64 oracle rounding at the storage points).

    Returns worst ratios per kind plus counts of outlier elements and calibrated tensors."""
    worst = {"outliers": 0, "calibrated": 0}

    def note(kind, a, b, floor=0.0, p=None):
        a = np.asarray(a, np.float64).ravel()
        b = np.asarray(b, np.float64).ravel()
        scale = max(np.abs(b).max(), floor, 1e-300)
        err = np.abs(a - b) / scale
        assert np.isfinite(a).all(), "%s: non-finite values" % kind
        bad = int((err > tol).sum())
        e = float(err.max())
        if bad and bad <= outlier_frac * err.size and e <= outlier_cap:
            worst["outliers"] += bad
            e = float(err[err <= tol].max())
        if e > tol and p is not None:
            p = np.asarray(p, np.float64).ravel()
            ps = max(np.abs(p).max(), floor, 1e-300)
            g_max, r_max = np.abs(a - p).max() / ps, np.abs(b - p).max() / ps
            pn = max(np.linalg.norm(p), floor * np.sqrt(p.size), 1e-300)
            g_l2, r_l2 = np.linalg.norm(a - p) / pn, np.linalg.norm(b - p) / pn
            ok = g_max <= 2.0 * r_max and g_l2 <= 1.5 * r_l2
            assert ok, ("%s: %.3e vs storage-mirroring oracle; vs float64: max %.3e (mirror %.3e), L2 %.3e (mirror %.3e)"
                        % (kind, e, g_max, r_max, g_l2, r_l2))
            worst["calibrated"] += 1
            worst[kind + "_vs_f64"] = max(worst.get(kind + "_vs_f64", 0.0), float(g_max))
            return
        worst[kind] = max(worst.get(kind, 0.0), e)
        assert e <= tol, "%s: relative error %.3e exceeds %.1e (%d of %d elements)" % (kind, e, tol, bad, err.size)

    P = pure
    for m in range(len(ref["y"])):
        note("y", gpu["y"][m], ref["y"][m], p=P and P["y"][m])
        if need_dx:
            note("dx", gpu["dx"][m], ref["dx"][m], p=P and P["dx"][m])
        note("loss", [gpu["loss"][m]], [ref["loss"][m]], p=P and [P["loss"][m]])
    # parameter tensors: primary criterion tensor by tensor; if one misses and `pure` is given, the
    # calibrated criterion is applied once to the whole flat vector of that kind (single small
    # tensors are too few samples for a ratio of two error norms to be stable)
    for kind in ("G", "v", "w"):
        kmax = np.abs(ref[kind]).max()
        off, missed = 0, False
        for i, name, shape in si.param_layout(net, first, last):
            n = int(np.prod(shape))
            sl = slice(off, off + n)
            off += n
            try:
                note(kind, gpu[kind][sl], ref[kind][sl], floor=1e-2 * kmax)
            except AssertionError:
                if P is None:
                    raise
                missed = True
        if missed:
            note(kind, gpu[kind], ref[kind], p=P[kind])
    return worst


def sampled_round_check(net, first, last, h, w, B, M, loss, bf16, sample, tol, seed=0, need_dx=1, lr=0.01, mu=0.9,
                        outlier_frac=1e-3, deep=True):
    """Full-size round on the GPU (all M micro-batches); the oracle computes only the micro-batches
    in `sample` (micro-batches are independent given the weights: BatchNorm statistics are per
    micro-batch), and the rest of the round is checked through what holds at any size:
    G is the float32 running sum of the per-micro-batch gradients in backward order (bit-exact),
    v = G/M and w = w0 - lr*v from zero momentum."""
    xs, tg, params, _ = make_inputs(net, first, last, h, w, B, M, loss, seed, bf16)
    gpu = gpu_round(net, first, last, h, w, B, M, loss, xs, tg, params, bf16, lr=lr, mu=mu, need_dx=need_dx, export_micro=True)
    acc = np.zeros_like(gpu["G"])
    for m in range(M):
        acc = acc + gpu["g"][m]                      # float32, same order as the library
    assert np.array_equal(acc, gpu["G"]), "accumulated gradient is not the running float32 sum of the micro-batch gradients"
    v_expect = gpu["G"].astype(np.float64) / M
    assert np.abs(gpu["v"] - v_expect).max() <= 1e-6 * max(np.abs(v_expect).max(), 1e-30)
    w_expect = params.astype(np.float64) - lr * v_expect
    assert np.abs(gpu["w"] - w_expect).max() <= 2e-7 * np.abs(w_expect).max()
    S = len(sample)
    sx, st = [xs[m] for m in sample], [tg[m] for m in sample]
    ref = oracle_round(net, first, last, B, S, loss, sx, st, params, lr=lr, mu=mu, store=bf16_store if bf16 else None)
    pure = oracle_round(net, first, last, B, S, loss, sx, st, params, lr=lr, mu=mu) if (bf16 and deep) else None
    Gs = np.sum([gpu["g"][m].astype(np.float64) for m in sample], axis=0)
    sub = {"y": [gpu["y"][m] for m in sample], "dx": [gpu["dx"][m] for m in sample], "loss": [gpu["loss"][m] for m in sample],
           "G": Gs, "v": Gs / S, "w": params.astype(np.float64) - lr * Gs / S}
    return compare(sub, ref, net, first, last, tol, need_dx=need_dx != 0, outlier_frac=outlier_frac, pure=pure)
