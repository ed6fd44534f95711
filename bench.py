#!/usr/bin/env python
"""Benchmark of the per-stage training round (stage training samples/s on B200).

One step = one HPP-Round of the stage on one batch of synthetic input: M forwards (+ the MSE
loss head), M backwards, M gradient accumulations and one SGD-momentum update, all enqueued on
one stream through the C ABI.  Workload: the MobileNetV2-style stage of four inverted-residual
blocks at 56x56 (24->24 x2, 24->32 stride 2, 32->32; expand 6), bfloat16 activations,
micro-batch 32, M = 8, i.e. 256 samples per step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the
stage on its own GPU (the path has no exchange step); the time is the maximum over ranks.
`--impl reference` times the float64 CPU oracle on a bounded sample of the same workload.
"""
import argparse
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
B, M, H, W = 32, 8, 56, 56
LR, MU = 0.01, 0.9
WORKLOAD = "config 2: MobileNetV2-style stage, 4 inverted-residual blocks at 56x56x24 (expand 6), micro-batch 32, M=8, bf16, MSE"


def workload():
    net = si.stage_net_mbv2_4blocks()
    return net, 0, len(net) - 1


def make_host_inputs(seed, batch, n_micro):
    net, first, last = workload()
    shp = si.out_shape(net, first, last, H, W)[last]
    xs = [si.round_to_bf16(si.normal(seed, 100000 + m, (batch, H, W, net[first].c_in)).astype(np.float32)) for m in range(n_micro)]
    ts = [si.round_to_bf16(si.normal(seed, 200000 + m, (batch,) + shp).astype(np.float32)) for m in range(n_micro)]
    return xs, ts, si.init_params(net, first, last, seed), shp


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


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel kinds, from the
# ncu capture summarised in profiles/ncu_top_kernels_config2.md: mean over the launches of one micro-batch's
# pass (the capture runs the benchmark's per-launch shapes); valid only while the kernel's source is the one
# that was captured.  A kernel measured alone keeps its output in the 126 MB L2, so the figure is mostly reads.
NCU_TRAFFIC = {
    "pw_bwd_data_tcgen05": {"bytes": (13.0 + 22.6 + 10.5 + 62.8 + 38.7 + 67.6 + 38.7 + 62.7) * 1e6 / 8,
                            "file": "paper_2408_08015_b200/csrc/pw_tc.cu", "sha": "fb3cf8d5c1ddd9a4"},
    "pw_bwd_weight_tcgen05": {"bytes": (12.9 + 20.9 + 10.5 + 62.7 + 38.6 + 62.7 + 38.6 + 62.7) * 1e6 / 8,
                              "file": "paper_2408_08015_b200/csrc/pw_tc.cu", "sha": "fb3cf8d5c1ddd9a4"},
    "dw_bwd_fused": {"bytes": 93.1e6, "file": "paper_2408_08015_b200/csrc/dwconv.cu", "sha": "e3b826da5053a2a8"},
}


def ncu_traffic(kernel):
    import hashlib
    rec = NCU_TRAFFIC.get(kernel)
    if not rec:
        return None
    try:
        cur = hashlib.sha256(open(os.path.join(ROOT, rec["file"]), "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    return rec["bytes"] if cur == rec["sha"] else None


def measured_peak_hbm():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([d.get("num_threads", 1) for d in threadpool_info()] or [1])
    except Exception:
        n = 1
    return int(n)


def time_oracle(batch, steps, warmup):
    """Seconds per (forward + backward + accumulate) of one micro-batch of `batch` samples on the CPU oracle."""
    import oracle as O
    from harness import bf16_store
    net, first, last = workload()
    xs, ts, params, _ = make_host_inputs(0, batch, 1)
    st = O.Stage(net, first, last, batch, 1, params, store=bf16_store, operand=bf16_store)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        y = st.forward(0, xs[0])
        _, dy = O.mse_loss(y, ts[0])
        st.backward(0, bf16_store(dy))
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
    sample = 4
    times = time_oracle(sample, args.steps, args.warmup)
    sec = sum(times) / len(times)
    val = sample / sec
    cores = oracle_threads()
    desc = "one micro-batch of %d samples (of %d): forward, loss, backward, accumulate, update" % (sample, B)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sec, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "sample": desc},
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


def whole_job_samples_per_s(world, steps, ms_max):
    """Replicas only: every rank runs its own B*M samples per step; the job's rate uses the slowest rank's time."""
    return B * M * world * steps / (ms_max * 1e-3)


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

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return max_over_ranks_ms(dist, ms, dev)

    net, first, last = workload()
    xs, ts, params, shp = make_host_inputs(rank, B, M)          # each replica draws its own batch
    bf = torch.bfloat16
    hx = [torch.from_numpy(x).to(bf).pin_memory() for x in xs]
    ht = [torch.from_numpy(t).to(bf).pin_memory() for t in ts]
    dx_in = [h.to(dev) for h in hx]
    dt_in = [h.to(dev) for h in ht]
    y = [torch.empty((B,) + shp, device=dev, dtype=bf) for _ in range(M)]
    dy = [torch.empty((B,) + shp, device=dev, dtype=bf) for _ in range(M)]
    dx = torch.empty_like(dx_in[0])
    loss = torch.zeros(M, device=dev, dtype=torch.float32)
    hloss = torch.zeros(M, dtype=torch.float32).pin_memory()
    n_out = int(np.prod((B,) + shp))

    hdl = P.asteroid_stage_create(net, first, last, H, W, B, M, dtype=P.AST_BF16, need_input_grad=1)
    P.asteroid_stage_import_state(hdl, np.ascontiguousarray(params))
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream

    def one_round(xd, td):
        for m in range(M):
            P.asteroid_stage_forward(hdl, m, xd[m].data_ptr(), y[m].data_ptr(), sp)
            P.asteroid_loss_mse(y[m].data_ptr(), td[m].data_ptr(), n_out, P.AST_BF16, dy[m].data_ptr(), loss.data_ptr() + 4 * m, sp)
        for m in range(M):
            P.asteroid_stage_backward(hdl, m, dy[m].data_ptr(), dx.data_ptr(), sp)
            P.asteroid_stage_accumulate(hdl, m, sp)
        P.asteroid_stage_step(hdl, LR, MU, sp)

    # End-to-end step: this step's inputs and targets go host -> device from pinned memory on a copy stream into one
    # of two device buffer sets, the round waits for them, the losses go device -> host.  The copies of step i+1
    # overlap the compute of step i (they wait until step i-1, the last user of their buffer set, has finished).
    copy_stream = torch.cuda.Stream(device=dev)
    in_sets = [(dx_in, dt_in), ([torch.empty_like(t) for t in dx_in], [torch.empty_like(t) for t in dt_in])]
    copied = [torch.cuda.Event() for _ in range(2)]
    consumed = [torch.cuda.Event() for _ in range(2)]
    e2e_step = [0]

    def one_round_e2e():
        b = e2e_step[0] % 2
        xd, td = in_sets[b]
        if e2e_step[0] >= 2:
            copy_stream.wait_event(consumed[b])
        with torch.cuda.stream(copy_stream):
            for m in range(M):
                xd[m].copy_(hx[m], non_blocking=True)
                td[m].copy_(ht[m], non_blocking=True)
            copied[b].record(copy_stream)
        stream.wait_event(copied[b])
        one_round(xd, td)
        consumed[b].record(stream)
        hloss.copy_(loss, non_blocking=True)
        e2e_step[0] += 1

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1))

    for _ in range(max(args.warmup, 3)):
        one_round(dx_in, dt_in)
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        gpu_id = str(local)
    sampler = ClockSampler(gpu_id)
    n0 = P.asteroid_launch_count()
    ms = timed(lambda: one_round(dx_in, dt_in), args.steps)
    launches = P.asteroid_launch_count() - n0
    clocks = sampler.stop()
    ms_e2e = timed(one_round_e2e, args.steps)
    if not np.isfinite(hloss.numpy()).all():
        raise SystemExit("non-finite loss")

    # per-kernel device times of the same steps, bracketed by CUDA events on the launching stream
    roofline = None
    kernels = []
    if rank == 0:
        torch.cuda.synchronize()
        P.asteroid_trace_start()
        for _ in range(args.steps):
            one_round(dx_in, dt_in)
        kernels = P.asteroid_trace_stop()
        tot = sum(k["total_ms"] for k in kernels)
        peak, how = measured_peak_hbm()
        for k in kernels:
            k["gbs"] = k["alg_bytes"] / (k["total_ms"] * 1e-3) / 1e9 if k["total_ms"] > 0 else 0.0
            k["share"] = k["total_ms"] / tot if tot > 0 else 0.0
        top = max(kernels, key=lambda k: k["total_ms"])
        roofline = {"bound": "hbm", "kernel": top["name"], "achieved": top["gbs"], "peak": peak, "unit": "GB/s",
                    "frac": top["gbs"] / peak, "peak_source": "of " + how, "traffic": ncu_traffic(top["name"]),
                    "avg_launch_us": 1e3 * top["total_ms"] / top["launches"], "share_of_step": top["share"],
                    "alg_bytes_per_launch": top["alg_bytes"] / top["launches"]}
    barrier()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = B
        t = time_oracle(sample, 1, 0)[0]
        cpu = {"value": sample / t, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
               "sample": "one micro-batch of %d samples (1 of the %d per step): forward, loss, backward, accumulate, update; %.1f s" % (sample, M, t)}

    P.asteroid_stage_destroy(hdl)
    if rank == 0:
        samples = B * M * world * args.steps
        out = {
            "metric": METRIC, "value": whole_job_samples_per_s(world, args.steps, ms), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "samples_per_step_per_gpu": B * M, "parallelism": "replicas only" if world > 1 else "single GPU",
                       "l2": "no flush: each step streams ~1.5 GB of activation slots plus gradients, far beyond the 126 MB L2"},
            "clocks": clocks,
            "e2e": {"value": samples / (ms_e2e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(sum(h.numel() * 2 for h in hx) + sum(h.numel() * 2 for h in ht)),
                    "d2h_bytes_per_step": int(hloss.numel() * 4)},
            "gpu_launches": int(launches),
            "roofline": roofline,
            "cpu_baseline": cpu,
            "kernels": [{"name": k["name"], "launches": k["launches"], "ms": round(k["total_ms"], 3), "share": round(k["share"], 4),
                         "alg_gbs": round(k["gbs"], 1)} for k in sorted(kernels, key=lambda k: -k["total_ms"])],
        }
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--m-override", type=int, default=0,
                    help="profiling captures only: run M' micro-batches per step instead of 8 (smaller device footprint); not a benchmark configuration")
    args = ap.parse_args()
    if args.m_override > 0:
        global M, WORKLOAD
        M = args.m_override
        WORKLOAD += " [profiling capture with M=%d]" % M
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
