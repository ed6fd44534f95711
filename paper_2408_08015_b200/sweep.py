"""Stage-partition sweep: the planner's cost profile measured on this GPU.

The full MobileNetV2 layer sequence is cut into P contiguous stages at block boundaries
(P in 2, 3, 4, 6; cut points minimise the largest stage's forward MACs); every stage is run alone
at micro-batch sizes 4..64 with M = 8 in bfloat16.  Per stage: samples/s of a whole round
(CUDA events).  Per layer (with --layers): the profile record t_f, t_b, a_l, w_l, FLOPs and the
algorithmic GB/s of its kernels.

    python -m paper_2408_08015_b200.sweep [--parts 2 3 4 6] [--batches 4 8 16 32 64] [--layers] [--out FILE]
    python -m paper_2408_08015_b200.sweep --resnet --batches 32 [--out FILE]      (ResNet-50 conv2_x+conv3_x stage, kernel trace)
"""
import argparse
import json
import sys

import numpy as np


def time_stage(P, torch, si, net, first, last, h, w, B, M, rounds=5, warm=3, trace=None, xent=None):
    dev = torch.device("cuda:0")
    bf = torch.bfloat16
    is_last = (last == len(net) - 1) if xent is None else xent      # softmax cross-entropy head, else MSE
    hdl = P.asteroid_stage_create(net, first, last, h, w, B, M, dtype=P.AST_BF16, need_input_grad=int(first > 0))
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


def main(argv=None):
    import torch
    import paper_2408_08015_b200 as P
    import stage_inputs as si
    ap = argparse.ArgumentParser()
    ap.add_argument("--parts", type=int, nargs="+", default=[2, 3, 4, 6])
    ap.add_argument("--batches", type=int, nargs="+", default=[4, 8, 16, 32, 64])
    ap.add_argument("--layers", action="store_true", help="also print the per-layer profile records")
    ap.add_argument("--out", default=None)
    ap.add_argument("--resnet", action="store_true",
                    help="instead of the sweep: the ResNet-50 conv2_x+conv3_x stage (56x56x64 input) as one stage at the given batches, with its kernel trace")
    args = ap.parse_args(argv)
    if args.resnet:
        net = si.resnet50_c2c3_net()
        out = open(args.out, "w") if args.out else sys.stdout
        for B in args.batches:
            trace = []
            hdl, ms = time_stage(P, torch, si, net, 0, len(net) - 1, 56, 56, B, 8, trace=trace, xent=False)
            P.asteroid_stage_destroy(hdl)
            tot = sum(k["total_ms"] for k in trace) or 1.0
            rec = {"net": "resnet50_c2c3", "B": B, "M": 8, "ms_per_round": round(ms, 4), "samples_per_s": round(B * 8 / (ms * 1e-3), 1),
                   "kernels": [{"name": k["name"], "launches": k["launches"], "us_per_launch": round(1e3 * k["total_ms"] / k["launches"], 1),
                                "share": round(k["total_ms"] / tot, 4),
                                "tflops": round(k["flops"] / (k["total_ms"] * 1e-3) / 1e12, 1) if k["total_ms"] > 0 else 0.0,
                                "alg_gbs": round(k["alg_bytes"] / (k["total_ms"] * 1e-3) / 1e9, 1) if k["total_ms"] > 0 else 0.0}
                               for k in sorted(trace, key=lambda k: -k["total_ms"])]}
            out.write(json.dumps(rec) + "\n")
            out.flush()
        return
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
                if args.layers:
                    layers = []
                    for l in range(first, last + 1):
                        r = P.asteroid_stage_profile(hdl, l, B)
                        if r["t_f_ms"] > 0 or r["t_b_ms"] > 0:
                            layers.append({"layer": l, "op": net[l].op, "t_f_ms": round(r["t_f_ms"], 4), "t_b_ms": round(r["t_b_ms"], 4),
                                           "a_l": r["a_l_bytes"], "w_l": r["w_l_bytes"], "flops": r["flops"],
                                           "f_gbs": round(r["alg_bytes_f"] / (r["t_f_ms"] * 1e6), 1) if r["t_f_ms"] > 0 else None,
                                           "b_gbs": round(r["alg_bytes_b"] / (r["t_b_ms"] * 1e6), 1) if r["t_b_ms"] > 0 else None})
                    rec["per_layer"] = layers
                P.asteroid_stage_destroy(hdl)
                out.write(json.dumps(rec) + "\n")
                out.flush()


if __name__ == "__main__":
    main()
