"""Seeded synthetic planning problems: per-layer cost tables of a few device types, device pools with memory budgets and
pairwise bandwidths.  Descriptions and random draws only; none of the planner's arithmetic lives here.

A problem is a dict:
  L, B, M, block           layers, micro-batch size, micro-batches per round, samples moved per offloading step
  bs[k]                    profiled batch sizes, ascending
  t_f[type][l][k], t_b     FP / BP milliseconds of layer l at batch size bs[k] on a device of that type
  a[l], w[l], act[l]       output bytes per sample, parameter bytes, bytes kept per sample for BP
  mod_factor, opt_factor   Mem_MOD and Mem_OPT as multiples of the parameter bytes
  devices[d]               {"type": t, "mem": bytes}
  bw[d][d']                bytes per millisecond between devices d and d'
"""
from .rng import uniform


def synthetic_problem(seed, L=6, n_types=2, N=3, B=16, M=4, bs=(1, 2, 4, 8, 16, 32), block=1, tight_memory=False, sublinear=0.7):
    u = list(uniform(seed, 77, 8 * L + 4 * N + N * N + 16))
    it = iter(u)
    speed = [1.0 + 1.5 * t for t in range(n_types)]          # type 0 fastest
    base_f = [0.2 + next(it) for _ in range(L)]
    base_b = [1.5 * x * (0.8 + 0.4 * next(it)) for x in base_f]
    fixed = [0.05 + 0.1 * next(it) for _ in range(L)]         # launch-like fixed cost: time is not linear in the batch
    t_f = [[[speed[t] * (fixed[l] + base_f[l] * (b ** sublinear)) for b in bs] for l in range(L)] for t in range(n_types)]
    t_b = [[[speed[t] * (fixed[l] + base_b[l] * (b ** sublinear)) for b in bs] for l in range(L)] for t in range(n_types)]
    a = [1e4 * (1 + int(8 * next(it))) for _ in range(L)]
    w = [1e5 * (1 + int(20 * next(it))) for _ in range(L)]
    act = [3e4 * (1 + int(6 * next(it))) for _ in range(L)]
    devices = []
    for d in range(N):
        t = int(next(it) * n_types) % n_types
        full = 4.0 * sum(w) + 7 * B * sum(act)
        mem = full * ((0.25 + 0.5 * next(it)) if tight_memory else 4.0) * (1.0 + 0.01 * d)
        devices.append({"type": t, "mem": mem})
    bw = [[0.0] * N for _ in range(N)]
    for i in range(N):
        for j in range(i + 1, N):
            bw[i][j] = bw[j][i] = 1e4 * (1 + int(9 * next(it)))
    return {"L": L, "B": B, "M": M, "block": block, "bs": list(bs), "t_f": t_f, "t_b": t_b, "a": a, "w": w, "act": act,
            "mod_factor": 3.0, "opt_factor": 1.0, "devices": devices, "bw": bw}
