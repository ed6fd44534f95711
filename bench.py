#!/usr/bin/env python
"""Benchmark of the per-stage training round (stage training samples/s on B200).

One step = one HPP-Round of the stage on one batch of synthetic input: M forwards (+ the loss head), M backwards,
M gradient accumulations and one SGD-momentum update, all enqueued on one stream through the C ABI.

    python bench.py [--config 1|2|3|4|6|all] [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workloads (synthetic tensors of the shapes of the paper's compact vision models):
  1  one inverted-residual block 16->96->16 at 32x32, float32, micro-batch 8, M=4, MSE
  2  MobileNetV2-style stage of four inverted-residual blocks at 56x56x24, bfloat16, micro-batch 32, M=8, MSE
  3  full MobileNetV2 at 224x224x3, bfloat16, micro-batch 16, M=4, softmax cross-entropy
  4  ResNet-50 conv2_x + conv3_x bottleneck stage at 56x56x64, bfloat16, micro-batch 32, M=8, MSE
  6  EfficientNet-B1-style stage of five MBConv6 blocks at 56x56x24, bfloat16, micro-batch 32, M=8, MSE (only on request)
`--config all` (the default) prints one JSON line per workload; the LAST line is the headline: workload 4, the
largest of the single-GPU workloads.  The timed region is repeated until it lasts about two seconds
(`steps_timed` = steps x repeats; `ms_per_step` is the mean over all of them).

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the stage on its own GPU
(the path has no exchange step); the time is the maximum over ranks.  `--impl reference` times the float64 CPU
oracle on a bounded sample of the headline workload.
"""
import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import stage_inputs as si  # noqa: E402

METRIC = "stage training samples/sec"
UNIT = "samples/s"
LR, MU = 0.01, 0.9
MIN_TIMED_S = 2.0


class Workload:
    def __init__(self, cfg):
        self.cfg = cfg
        if cfg == 1:
            self.net, self.H, self.W, self.B, self.M, self.bf16, self.loss = si.block_net(16, 6), 32, 32, 8, 4, False, "mse"
            self.name = "config 1: one inverted-residual block 16->96->16 at 32x32, micro-batch 8, M=4, float32, MSE"
            self.cpu_sample, self.ref_sample = 8, 8
        elif cfg == 2:
            self.net, self.H, self.W, self.B, self.M, self.bf16, self.loss = si.stage_net_mbv2_4blocks(), 56, 56, 32, 8, True, "mse"
            self.name = "config 2: MobileNetV2-style stage, 4 inverted-residual blocks at 56x56x24 (expand 6), micro-batch 32, M=8, bf16, MSE"
            self.cpu_sample, self.ref_sample = 32, 4
        elif cfg == 3:
            self.net, self.H, self.W, self.B, self.M, self.bf16, self.loss = si.mobilenetv2_net(), 224, 224, 16, 4, True, "xent"
            self.name = "config 3: full MobileNetV2 1.0 at 224x224x3, micro-batch 16, M=4, bf16, softmax cross-entropy"
            self.cpu_sample, self.ref_sample = 16, 2
        elif cfg == 4:
            self.net, self.H, self.W, self.B, self.M, self.bf16, self.loss = si.resnet50_c2c3_net(), 56, 56, 32, 8, True, "mse"
            self.name = "config 4: ResNet-50 conv2_x+conv3_x bottleneck stage at 56x56x64, micro-batch 32, M=8, bf16, MSE"
            self.cpu_sample, self.ref_sample = 8, 1
        elif cfg == 6:
            self.net, self.H, self.W, self.B, self.M, self.bf16, self.loss = si.efficientnet_b1_stage_net(), 56, 56, 32, 8, True, "mse"
            self.name = ("EfficientNet-B1-style stage: 5 MBConv6 blocks (5x5 then 3x3 depthwise, squeeze-excite, SiLU) at 56x56x24, "
                         "micro-batch 32, M=8, bf16, MSE")
            self.cpu_sample, self.ref_sample = 16, 4
        else:
            raise ValueError("config must be 1, 2, 3, 4 or 6")
        self.first, self.last = 0, len(self.net) - 1
        self.need_dx = 0 if cfg == 3 else 1          # the full network is the first stage of itself: no input gradient
        self.shp = si.out_shape(self.net, self.first, self.last, self.H, self.W)[self.last]
        self.dtype = "bf16" if self.bf16 else "f32"

    def host_inputs(self, seed, batch, n_micro):
        cast = si.round_to_bf16 if self.bf16 else (lambda a: a)
        c_in = self.net[self.first].c_in
        xs = [cast(si.normal(seed, 100000 + m, (batch, self.H, self.W, c_in)).astype(np.float32)) for m in range(n_micro)]
        if self.loss == "mse":
            ts = [cast(si.normal(seed, 200000 + m, (batch,) + self.shp).astype(np.float32)) for m in range(n_micro)]
        else:
            ts = [si.labels(seed, 300000 + m, batch, self.shp[2]).astype(np.int32) for m in range(n_micro)]
        return xs, ts, si.init_params(self.net, self.first, self.last, seed)


HEADLINE = 4
# compatibility names for the multi-rank host-logic test: samples per step of the headline workload
B, M = Workload(HEADLINE).B, Workload(HEADLINE).M


# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi sampled every 200 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.path = tempfile.mktemp(suffix=".csv")
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                                          "-lms", "200"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except OSError:
            pass
        if sm:
            busy = [s for s in sm if s >= 0.5 * max(sm)]
            out.update(sm_mhz=statistics.median(busy), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def ncu_traffic(cfg, kernel):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of a kernel kind from the committed ncu
    summary, or None when there is no capture of the kernel's current source."""
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "ncu_traffic.json")))["config%d" % cfg][kernel]
        cur = hashlib.sha256(open(os.path.join(ROOT, rec["file"]), "rb").read()).hexdigest()[:16]
        return rec["bytes_per_launch"] if cur == rec["sha"] else None
    except (OSError, KeyError, ValueError):
        return None


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        d = json.load(open(p))
        return {"hbm": float(d["hbm_gbs"]), "tensor": float(d["bf16_tflops_sustained"]), "how": "measured"}
    except Exception:
        return {"hbm": 6650.0, "tensor": 1400.0, "how": "fallback"}


# kernel kinds whose layers sit above the ridge point (dense 3x3 convolutions of 64 and 128 channels): judged on the tensor pipe
TENSOR_BOUND = ("conv3x3_fwd_tcgen05", "conv3x3_bwd_data_tcgen05", "conv3x3_bwd_weight_tcgen05")


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([d.get("num_threads", 1) for d in threadpool_info()] or [1])
    except Exception:
        n = 1
    return int(n)


def time_oracle(wl, batch, steps, warmup):
    """Seconds per (forward + loss + backward + accumulate + update) of one micro-batch of `batch` samples on the CPU oracle."""
    import oracle as O
    xs, ts, params = wl.host_inputs(0, batch, 1)
    st = O.Stage(wl.net, wl.first, wl.last, batch, 1, params)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        y = st.forward(0, xs[0])
        if wl.loss == "mse":
            _, dy = O.mse_loss(y, ts[0])
        else:
            _, dy = O.softmax_xent_loss(y.reshape(batch, -1), ts[0])
        st.backward(0, dy)
        st.accumulate(0)
        st.step(LR, MU)
        if it >= warmup:
            times.append(time.perf_counter() - t0)
    return times


# ------------------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = Workload(HEADLINE if args.config == "all" else int(args.config))
    sample = wl.ref_sample
    times = time_oracle(wl, sample, args.steps, args.warmup)
    sec = sum(times) / len(times)
    val = sample / sec
    cores = oracle_threads()
    desc = "one micro-batch of %d samples (of %d x %d per step): forward, loss, backward, accumulate, update" % (sample, wl.M, wl.B)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sec, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": wl.name, "sample": desc},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def max_over_ranks_ms(dist, ms, device):
    """The slowest rank's time: every rank contributes its own device-timed milliseconds."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_samples_per_s(world, steps, ms_max, samples_per_step=None):
    """Replicas only: every rank runs its own B*M samples per step; the job's rate uses the slowest rank's time."""
    return (samples_per_step or B * M) * world * steps / (ms_max * 1e-3)


def bench_config(wl, args, torch, P, dist, dev, rank, world):
    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    Bn, Mn = wl.B, wl.M
    tdt = torch.bfloat16 if wl.bf16 else torch.float32
    adt = P.AST_BF16 if wl.bf16 else P.AST_F32
    xs, ts, params = wl.host_inputs(rank, Bn, Mn)               # each replica draws its own batch
    hx = [torch.from_numpy(x).to(tdt).pin_memory() for x in xs]
    ht = [(torch.from_numpy(t).to(tdt) if wl.loss == "mse" else torch.from_numpy(t)).pin_memory() for t in ts]
    n_out = int(np.prod((Bn,) + wl.shp))

    def dev_set():
        return {"x": [torch.empty(h.shape, device=dev, dtype=h.dtype) for h in hx],
                "t": [torch.empty(h.shape, device=dev, dtype=h.dtype) for h in ht],
                "y": [torch.empty((Bn,) + wl.shp, device=dev, dtype=tdt) for _ in range(Mn)],
                "dx": [torch.empty(hx[0].shape, device=dev, dtype=tdt) for _ in range(Mn if wl.need_dx else 0)],
                "loss": torch.zeros(Mn, device=dev, dtype=torch.float32)}
    sets = [dev_set(), dev_set()]
    for s in sets:
        for m in range(Mn):
            s["x"][m].copy_(hx[m])
            s["t"][m].copy_(ht[m])
    dy = [torch.empty((Bn,) + wl.shp, device=dev, dtype=tdt) for _ in range(Mn)]
    # host side of the end-to-end step: what the stage's neighbours in a pipeline receive (Section 3.3: output
    # activations go to the next stage, input gradients to the previous one) and the losses
    hy = [torch.empty((Bn,) + wl.shp, dtype=tdt).pin_memory() for _ in range(Mn)]
    hdx = [torch.empty(hx[0].shape, dtype=tdt).pin_memory() for _ in range(Mn if wl.need_dx else 0)]
    hloss = torch.zeros(Mn, dtype=torch.float32).pin_memory()

    hdl = P.asteroid_stage_create(wl.net, wl.first, wl.last, wl.H, wl.W, Bn, Mn, dtype=adt, need_input_grad=wl.need_dx)
    P.asteroid_stage_import_state(hdl, np.ascontiguousarray(params))
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream

    def one_round(s, sp=sp):
        for m in range(Mn):
            P.asteroid_stage_forward(hdl, m, s["x"][m].data_ptr(), s["y"][m].data_ptr(), sp)
            lp = s["loss"].data_ptr() + 4 * m
            if wl.loss == "mse":
                P.asteroid_loss_mse(s["y"][m].data_ptr(), s["t"][m].data_ptr(), n_out, adt, dy[m].data_ptr(), lp, sp)
            else:
                P.asteroid_loss_softmax_xent(s["y"][m].data_ptr(), s["t"][m].data_ptr(), Bn, wl.shp[2], adt, dy[m].data_ptr(), lp, sp)
        for m in range(Mn):
            P.asteroid_stage_backward(hdl, m, dy[m].data_ptr(), s["dx"][m].data_ptr() if wl.need_dx else None, sp)
            P.asteroid_stage_accumulate(hdl, m, sp)
        P.asteroid_stage_step(hdl, LR, MU, sp)

    # End-to-end step: this step's inputs and targets go host -> device from pinned memory on a copy stream into one of
    # two device buffer sets; the round waits for them; every micro-batch's output y_m, every input gradient dx_m and the
    # losses go device -> host on a third stream.  The copies of step i+1 and of step i-1 overlap the compute of step i.
    h2d, d2h = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    copied = [torch.cuda.Event() for _ in range(2)]
    computed = [torch.cuda.Event() for _ in range(2)]
    drained = [torch.cuda.Event() for _ in range(2)]
    e2e_step = [0]

    def one_round_e2e():
        b = e2e_step[0] % 2
        s = sets[b]
        if e2e_step[0] >= 2:
            h2d.wait_event(computed[b])          # the round that last read this set's inputs
            stream.wait_event(drained[b])        # the copies that last read this set's outputs
        with torch.cuda.stream(h2d):
            for m in range(Mn):
                s["x"][m].copy_(hx[m], non_blocking=True)
                s["t"][m].copy_(ht[m], non_blocking=True)
            copied[b].record(h2d)
        stream.wait_event(copied[b])
        if graphs[b] is not None:
            graphs[b].replay()                   # the same round, captured once per buffer set
        else:
            one_round(s)
        computed[b].record(stream)
        d2h.wait_event(computed[b])
        with torch.cuda.stream(d2h):
            for m in range(Mn):
                hy[m].copy_(s["y"][m], non_blocking=True)
                if wl.need_dx:
                    hdx[m].copy_(s["dx"][m], non_blocking=True)
            hloss.copy_(s["loss"], non_blocking=True)
            drained[b].record(d2h)
        e2e_step[0] += 1

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        barrier()
        return max_over_ranks_ms(dist, e0.elapsed_time(e1), dev)

    warm = max(args.warmup, 3)
    for _ in range(warm):
        one_round(sets[0])
    # The device-timed steps replay one captured CUDA graph of the round (the stage calls only enqueue: the same kernels, in
    # the same order, on the same two streams, without the per-launch submission cost).  If the capture is refused the steps
    # are issued call by call, on a fresh stage (a capture that stopped half-way leaves the stage's bookkeeping mid-round).
    run_round, launch_mode, launches_per_round = (lambda: one_round(sets[0])), "call by call", None
    graphs = [None, None]                         # one per device buffer set (the end-to-end leg alternates between the two)
    if not args.no_graph:
        torch.cuda.synchronize()
        try:
            made = []
            for b in range(2):
                n_cap = P.asteroid_launch_count()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, capture_error_mode="thread_local"):
                    one_round(sets[b], torch.cuda.current_stream().cuda_stream)
                launches_per_round = P.asteroid_launch_count() - n_cap
                made.append(graph)
            for _ in range(2):
                made[0].replay()
            torch.cuda.synchronize()
            graphs = made
            run_round, launch_mode = graphs[0].replay, "one captured CUDA graph of the round, replayed"
        except Exception as exc:                                     # noqa: BLE001 (any refusal means: no graph)
            launches_per_round = None
            sys.stderr.write("graph capture refused (%s): steps issued call by call\n" % (str(exc).splitlines() or [""])[0])
            torch.cuda.synchronize()
            P.asteroid_stage_destroy(hdl)
            hdl = P.asteroid_stage_create(wl.net, wl.first, wl.last, wl.H, wl.W, Bn, Mn, dtype=adt, need_input_grad=wl.need_dx)
            P.asteroid_stage_import_state(hdl, np.ascontiguousarray(params))
            for _ in range(warm):
                one_round(sets[0])
    # repeats: the timed region lasts about MIN_TIMED_S (every rank takes the same count: it comes from rank 0's probe)
    probe = timed(run_round, 2) / 2
    rep = max(1, int(np.ceil(args.min_seconds * 1e3 / max(probe * args.steps, 1e-3))))
    if dist is not None:
        t = torch.tensor([rep], device=dev)
        dist.broadcast(t, 0)
        rep = int(t.item())
    steps_timed = args.steps * rep
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev.index).uuid)
    except Exception:
        gpu_id = str(dev.index)
    sampler = ClockSampler(gpu_id)
    n0 = P.asteroid_launch_count()
    ms = timed(run_round, steps_timed)
    launches = P.asteroid_launch_count() - n0 if launches_per_round is None else launches_per_round * steps_timed
    clocks = sampler.stop()

    def e2e_timed(steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            one_round_e2e()
        stream.wait_stream(d2h)                  # the step is over when its results are on the host
        e1.record(stream)
        barrier()
        return max_over_ranks_ms(dist, e0.elapsed_time(e1), dev)
    for _ in range(2):
        one_round_e2e()
    ms_e2e = e2e_timed(steps_timed)
    if not np.isfinite(hloss.numpy()).all():
        raise SystemExit("non-finite loss")

    # per-kernel device times of further steps, every launch bracketed by CUDA events on the launching stream
    roofline, kernels = None, []
    if rank == 0:
        torch.cuda.synchronize()
        P.asteroid_trace_start()
        for _ in range(min(args.steps, 5)):
            one_round(sets[0])
        kernels = P.asteroid_trace_stop()
        tot = sum(k["total_ms"] for k in kernels)
        pk = measured_peaks()
        for k in kernels:
            sec = k["total_ms"] * 1e-3
            k["gbs"] = k["alg_bytes"] / sec / 1e9 if sec > 0 else 0.0
            k["tflops"] = k["flops"] / sec / 1e12 if sec > 0 else 0.0
            k["share"] = k["total_ms"] / tot if tot > 0 else 0.0
            k["bound"] = "tensor" if k["name"] in TENSOR_BOUND else "hbm"
            k["frac"] = k["tflops"] / pk["tensor"] if k["bound"] == "tensor" else k["gbs"] / pk["hbm"]
        top = max(kernels, key=lambda k: k["total_ms"])
        tensor = top["bound"] == "tensor"
        roofline = {"bound": top["bound"], "kernel": top["name"], "achieved": top["tflops"] if tensor else top["gbs"],
                    "peak": pk["tensor"] if tensor else pk["hbm"], "unit": "TFLOP/s" if tensor else "GB/s", "frac": top["frac"],
                    "peak_source": "of " + pk["how"] + (" (sustained bf16)" if tensor else " (copy)"), "traffic": ncu_traffic(wl.cfg, top["name"]),
                    "avg_launch_us": 1e3 * top["total_ms"] / top["launches"], "share_of_step": top["share"],
                    ("flops_per_launch" if tensor else "alg_bytes_per_launch"): (top["flops"] if tensor else top["alg_bytes"]) / top["launches"]}
    barrier()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        t = time_oracle(wl, wl.cpu_sample, 1, 0)[0]
        cpu = {"value": wl.cpu_sample / t, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
               "sample": "one micro-batch of %d samples (a step has %d x %d): forward, loss, backward, accumulate, update; %.1f s"
                         % (wl.cpu_sample, Mn, Bn, t)}

    P.asteroid_stage_destroy(hdl)
    out = None
    if rank == 0:
        esz = 2 if wl.bf16 else 4
        h2d_bytes = sum(h.numel() * h.element_size() for h in hx) + sum(h.numel() * h.element_size() for h in ht)
        d2h_bytes = sum(h.numel() * esz for h in hy) + sum(h.numel() * esz for h in hdx) + hloss.numel() * 4
        out = {
            "metric": METRIC, "value": whole_job_samples_per_s(world, steps_timed, ms, Bn * Mn), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms / steps_timed, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": wl.name, "samples_per_step_per_gpu": Bn * Mn, "parallelism": "replicas only" if world > 1 else "single GPU",
                       "steps_timed": steps_timed, "launch": launch_mode,
                       "timed_region": "%d x %d steps so that it lasts about %.0f s; ms_per_step is their mean" % (rep, args.steps, args.min_seconds),
                       "l2": ("no flush: each step streams its activation slots and gradients, far beyond the 126 MB L2" if wl.cfg != 1 else
                              "no flush and smaller than L2: a step touches about 30 MB, so this workload is launch- and latency-bound by construction")},
            "clocks": clocks,
            "e2e": {"value": Bn * Mn * world * steps_timed / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d_bytes),
                    "d2h_bytes_per_step": int(d2h_bytes),
                    "moves": "H2D: every x_m and target; D2H: every y_m, every dx_m, the losses; copies on their own streams, double-buffered"},
            "gpu_launches": int(launches),
            "roofline": roofline,
            "cpu_baseline": cpu,
            "kernels": [{"name": k["name"], "launches": k["launches"], "ms": round(k["total_ms"], 3), "share": round(k["share"], 4),
                         "alg_gbs": round(k["gbs"], 1), "tflops": round(k["tflops"], 1), "bound": k["bound"], "frac": round(k["frac"], 4)}
                        for k in sorted(kernels, key=lambda k: -k["total_ms"])],
        }
    return out


def run_ours(args):
    import torch
    import paper_2408_08015_b200 as P

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the stage library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    cfgs = [1, 2, 3, HEADLINE] if args.config == "all" else [int(args.config)]
    for c in cfgs:
        out = bench_config(Workload(c), args, torch, P, dist, dev, rank, world)
        if rank == 0:
            if c != cfgs[-1]:
                out["headline"] = False
            print(json.dumps(out), flush=True)
        torch.cuda.empty_cache()
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="all", choices=["1", "2", "3", "4", "6", "all"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="issue the device-timed steps call by call instead of replaying a captured graph")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_S,
                    help="the K timed steps are repeated until the timed region lasts about this long (0: exactly K steps)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
