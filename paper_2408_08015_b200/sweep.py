"""Stage-partition sweep: the planner's cost profile measured on this GPU.

The full MobileNetV2 layer sequence is cut into P contiguous stages at block boundaries
(P in 2, 3, 4, 6; cut points minimise the largest stage's forward MACs); every stage is run alone
at micro-batch sizes 4..64 with M = 8 in bfloat16.  Per stage: samples/s of a whole round
(CUDA events).  Per layer (with --layers): the profile record t_f, t_b, a_l, w_l, FLOPs and the
algorithmic GB/s of its kernels.

    python -m paper_2408_08015_b200.sweep [--parts 2 3 4 6] [--batches 4 8 16 32 64] [--layers] [--out FILE]
    python -m paper_2408_08015_b200.sweep --unit conv:128:512:1:1:28:28:32:none [--out FILE]      (one unit, per-kernel trace)
    python -m paper_2408_08015_b200.sweep --plan [--batches 4 8 16 32 64] [--out FILE]            (planner on the measured tables)
"""
import argparse
import json
import sys

import numpy as np


def time_stage(P, torch, si, net, first, last, h, w, B, M, rounds=5, warm=3, trace=None, xent=None, need_dx=None):
    dev = torch.device("cuda:0")
    bf = torch.bfloat16
    is_last = (last == len(net) - 1) if xent is None else xent      # softmax cross-entropy head, else MSE
    hdl = P.asteroid_stage_create(net, first, last, h, w, B, M, dtype=P.AST_BF16, need_input_grad=int(first > 0) if need_dx is None else need_dx)
    try:
        P.asteroid_stage_import_state(hdl, si.init_params(net, first, last, 0))
        n_out, shp = P.asteroid_stage_output_elems(hdl)
        c_in = net[first].c_in
        x = [torch.randn((B, h, w, c_in), device=dev).to(bf) for _ in range(M)]
        y = [torch.empty((B,) + shp, device=dev, dtype=bf) for _ in range(M)]
        dy = [torch.empty((B,) + shp, device=dev, dtype=bf) for _ in range(M)]
        dx = torch.empty_like(x[0])
        loss = torch.zeros(M, device=dev)
        if is_last:
            tgt = [torch.randint(0, shp[2], (B,), device=dev, dtype=torch.int32) for _ in range(M)]
        else:
            tgt = [torch.randn((B,) + shp, device=dev).to(bf) for _ in range(M)]
        st = torch.cuda.current_stream()
        sp = st.cuda_stream

        def one_round():
            for m in range(M):
                P.asteroid_stage_forward(hdl, m, x[m].data_ptr(), y[m].data_ptr(), sp)
                if is_last:
                    P.asteroid_loss_softmax_xent(y[m].data_ptr(), tgt[m].data_ptr(), B, shp[2], P.AST_BF16, dy[m].data_ptr(), loss.data_ptr() + 4 * m, sp)
                else:
                    P.asteroid_loss_mse(y[m].data_ptr(), tgt[m].data_ptr(), n_out, P.AST_BF16, dy[m].data_ptr(), loss.data_ptr() + 4 * m, sp)
            for m in range(M):
                P.asteroid_stage_backward(hdl, m, dy[m].data_ptr(), dx.data_ptr(), sp)
                P.asteroid_stage_accumulate(hdl, m, sp)
            P.asteroid_stage_step(hdl, 0.01, 0.9, sp)

        for _ in range(warm):
            one_round()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for _ in range(rounds):
            one_round()
        e1.record(st)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / rounds
        if trace is not None:
            # per-kernel device times of the same round (every kernel alone on the stream, CUDA events around each launch)
            P.asteroid_trace_start()
            for _ in range(rounds):
                one_round()
            trace.extend(P.asteroid_trace_stop())
        return hdl, ms
    except Exception:
        P.asteroid_stage_destroy(hdl)
        raise


def measured_peaks():
    """(HBM GB/s, dense bf16 TFLOP/s sustained) measured on this machine if the record is present, else the stated fall-back figures."""
    import os
    p = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    try:
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d["bf16_tflops_sustained"])
    except Exception:
        return 6650.0, 1400.0


def unit_cost_tables(P, si, net, unit_last, h, w, batches):
    """The planner's cost tables measured on this GPU (Section 3.3: the profiler records FP / BP time of each layer for
    various batch sizes, output size and weight size): one planning "layer" per block-level unit of `net`.
    Returns (t_f[unit][k], t_b[unit][k] in ms, a[unit] output bytes per sample, w[unit] parameter bytes,
    act[unit] bytes kept per sample for BP: the stored tensors of the unit)."""
    first_of = [0] + [u + 1 for u in unit_last[:-1]]
    hdl = P.asteroid_stage_create(net, 0, len(net) - 1, h, w, batches[0], 1, dtype=P.AST_BF16, need_input_grad=0)
    try:
        P.asteroid_stage_import_state(hdl, si.init_params(net, 0, len(net) - 1, 0))
        recs = {b: [P.asteroid_stage_profile(hdl, l, b) for l in range(len(net))] for b in batches}
    finally:
        P.asteroid_stage_destroy(hdl)
    t_f = [[sum(recs[b][l]["t_f_ms"] for l in range(f, u + 1)) for b in batches] for f, u in zip(first_of, unit_last)]
    t_b = [[sum(recs[b][l]["t_b_ms"] for l in range(f, u + 1)) for b in batches] for f, u in zip(first_of, unit_last)]
    b0 = batches[0]
    a = [recs[b0][u]["a_l_bytes"] / b0 for u in unit_last]
    wv = [float(sum(recs[b0][l]["w_l_bytes"] for l in range(f, u + 1))) for f, u in zip(first_of, unit_last)]
    stored = ("conv", "dwconv", "add", "gap", "linear")
    act = [sum(recs[b0][l]["a_l_bytes"] for l in range(f, u + 1) if net[l].op in stored) / b0 for f, u in zip(first_of, unit_last)]
    return t_f, t_b, a, wv, act


def plan_problem(t_f, t_b, a, wv, act, batches, slow=(1.0, 2.0, 4.0), devices=((0, 8e9), (1, 4e9), (1, 4e9), (2, 2e9), (2, 2e9), (2, 2e9)),
                 bytes_per_ms=125e3, B=64, M=8, block=4):
    """A synthetic device pool on top of measured tables: device types are this GPU slowed down by the factors in `slow`;
    `devices` lists (type, memory budget in bytes); every link has `bytes_per_ms` (125e3 = 1 Gbit/s)."""
    N = len(devices)
    return {"L": len(a), "B": B, "M": M, "block": block, "bs": list(batches),
            "t_f": [[[f * x for x in row] for row in t_f] for f in slow], "t_b": [[[f * x for x in row] for row in t_b] for f in slow],
            "a": a, "w": wv, "act": act, "mod_factor": 3.0, "opt_factor": 1.0,
            "devices": [{"type": t, "mem": m} for t, m in devices], "bw": [[0.0 if i == j else bytes_per_ms for j in range(N)] for i in range(N)]}


def main(argv=None):
    import torch
    import paper_2408_08015_b200 as P
    import stage_inputs as si
    ap = argparse.ArgumentParser()
    ap.add_argument("--parts", type=int, nargs="+", default=[2, 3, 4, 6])
    ap.add_argument("--batches", type=int, nargs="+", default=[4, 8, 16, 32, 64])
    ap.add_argument("--layers", action="store_true", help="also print the per-layer profile records")
    ap.add_argument("--out", default=None)
    ap.add_argument("--plan", action="store_true",
                    help="instead of the sweep: measure the per-unit cost tables of MobileNetV2 at the given batch sizes and run the planner "
                         "(Section 3.3) on them for a few synthetic device pools")
    ap.add_argument("--unit", nargs="+", default=None, metavar="KIND:CIN:COUT:K:STRIDE:H:W:BATCH:ACT",
                    help="instead of the sweep: single conv->BN->activation units (KIND conv|dwconv, ACT relu|relu6|none), each as a one-unit "
                         "stage with M=1, with the per-kernel trace of its round; e.g. conv:128:512:1:1:28:28:32:none")
    args = ap.parse_args(argv)
    if args.plan:
        # the planner on this GPU's measured cost tables (MobileNetV2 at 224x224, block-level units) and synthetic device pools
        import time
        net, units = si.mobilenetv2_net(), si.mobilenetv2_units()
        tabs = unit_cost_tables(P, si, net, units, 224, 224, args.batches)
        out = open(args.out, "w") if args.out else sys.stdout
        pools = {"1 fast + 2 medium + 3 slow, 1 Gbit/s": {}, "same, 100 Mbit/s": {"bytes_per_ms": 12.5e3},
                 "4 equal devices, 1 Gbit/s": {"devices": ((0, 4e9),) * 4}, "8 slow devices with 1 GB, 100 Mbit/s": {"devices": ((2, 1e9),) * 8, "bytes_per_ms": 12.5e3}}
        for name, kw in pools.items():
            prob = plan_problem(*tabs, args.batches, **kw)
            t0 = time.perf_counter()
            r = P.asteroid_plan(prob)
            dt = time.perf_counter() - t0
            rec = {"pool": name, "planning_ms": round(1e3 * dt, 2), "B": prob["B"], "M": prob["M"],
                   "latency_ms": None if r is None else round(r["latency"], 3),
                   "samples_per_s": None if r is None else round(prob["B"] * prob["M"] / (r["latency"] * 1e-3), 1),
                   "stages": None if r is None else [{"units": list(s["layers"]), "devices": s["devices"], "samples": s["y"],
                                                      "e_f_ms": round(s["ef"], 3), "e_b_ms": round(s["eb"], 3), "t_a_ms": round(s["ta"], 3)} for s in r["stages"]]}
            out.write(json.dumps(rec) + "\n")
            out.flush()
        return
    if args.unit:
        # one conv -> BatchNorm -> activation unit as a stage of its own: per-kernel device times of its round
        for spec in args.unit:
            kind, ci, co, k, stride, h, w, B, act = spec.split(":")
            net = si.single_unit_net(kind, int(ci), int(co), k=int(k), stride=int(stride), bn=True, act=None if act == "none" else act)
            out = open(args.out, "a") if args.out else sys.stdout
            trace = []
            hdl, ms = time_stage(P, torch, si, net, 0, len(net) - 1, int(h), int(w), int(B), 1, rounds=10, trace=trace, xent=False, need_dx=1)
            P.asteroid_stage_destroy(hdl)
            rec = {"unit": spec, "ms_per_round": round(ms, 4),
                   "kernels": [{"name": k_["name"], "launches_per_round": k_["launches"] // 10, "us_per_launch": round(1e3 * k_["total_ms"] / k_["launches"], 1),
                                "tflops": round(k_["flops"] / (k_["total_ms"] * 1e-3) / 1e12, 1) if k_["total_ms"] > 0 else 0.0,
                                "alg_gbs": round(k_["alg_bytes"] / (k_["total_ms"] * 1e-3) / 1e9, 1) if k_["total_ms"] > 0 else 0.0}
                               for k_ in sorted(trace, key=lambda q: -q["total_ms"])]}
            out.write(json.dumps(rec) + "\n")
            out.flush()
        return
    peaks = measured_peaks()
    net = si.mobilenetv2_net()
    units = si.mobilenetv2_units()
    shapes = si.out_shape(net, 0, len(net) - 1, 224, 224)
    out = open(args.out, "w") if args.out else sys.stdout
    M = 8
    for parts in args.parts:
        cuts = si.partition_units(net, units, parts, 224, 224)
        for p, (first, last) in enumerate(cuts):
            h, w, _ = shapes[first - 1] if first > 0 else (224, 224, 3)
            macs = sum(si.forward_macs(net, first, last, h, w).values())
            for B in args.batches:
                hdl, ms = time_stage(P, torch, si, net, first, last, h, w, B, M)
                rec = {"P": parts, "stage": p, "layers": [first, last], "B": B, "M": M, "ms_per_round": round(ms, 4),
                       "samples_per_s": round(B * M / (ms * 1e-3), 1), "fwd_mmacs_per_sample": round(macs / 1e6, 2)}
                # whole-stage roofline fraction: forward + backward + weight-gradient multiply-adds (3x forward) against the tensor peak
                rec["stage_tensor_frac"] = round(3 * 2 * macs * B * M / (ms * 1e-3) / 1e12 / peaks[1], 4)
                if args.layers:
                    layers = []
                    for l in range(first, last + 1):
                        r = P.asteroid_stage_profile(hdl, l, B)
                        if r["t_f_ms"] > 0 or r["t_b_ms"] > 0:
                            f_gbs = r["alg_bytes_f"] / (r["t_f_ms"] * 1e6) if r["t_f_ms"] > 0 else None
                            b_gbs = r["alg_bytes_b"] / (r["t_b_ms"] * 1e6) if r["t_b_ms"] > 0 else None
                            f_tf = r["flops"] / (r["t_f_ms"] * 1e9) if r["t_f_ms"] > 0 else None
                            b_tf = 2 * r["flops"] / (r["t_b_ms"] * 1e9) if r["t_b_ms"] > 0 else None
                            # roofline fraction of a layer: the larger of its memory and its tensor-pipe fraction (whichever bounds it)
                            frac = lambda g, t: None if g is None else round(max(g / peaks[0], (t or 0.0) / peaks[1]), 4)
                            layers.append({"layer": l, "op": net[l].op, "t_f_ms": round(r["t_f_ms"], 4), "t_b_ms": round(r["t_b_ms"], 4),
                                           "a_l": r["a_l_bytes"], "w_l": r["w_l_bytes"], "flops": r["flops"], "fused_into": r["fused_into"],
                                           "f_gbs": None if f_gbs is None else round(f_gbs, 1), "b_gbs": None if b_gbs is None else round(b_gbs, 1),
                                           "f_roofline": frac(f_gbs, f_tf), "b_roofline": frac(b_gbs, b_tf)})
                    rec["per_layer"] = layers
                P.asteroid_stage_destroy(hdl)
                out.write(json.dumps(rec) + "\n")
                out.flush()


if __name__ == "__main__":
    main()
