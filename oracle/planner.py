"""Parallelism planning of Section 3.3 in plain Python.  Test infrastructure only.

The planner takes the profiler's per-layer cost tables (FP / BP time per batch size, output bytes a_l, weight bytes
w_l), a pool of devices with memory budgets and pairwise bandwidths, and picks the hybrid pipeline (model cut points,
device groups, per-device share of a micro-batch) with the smallest estimated HPP-Round latency:

  allocate()        Algorithm 1: MemoryAwareBalancing, then StragglerWorkloadOffloading; Eq. (7)-(9)
  round_latency()   Eq. (4)-(6): waiting, execution and AllReduce phase of every step, the dominant step
  plan()            Algorithm 2: dynamic programming over (layers l, devices n, stages p); Eq. (10)-(11)

Everything is lists and loops; nothing is cached or reordered beyond what the algorithms state.  Readings of points the
paper leaves open are marked "reading:" and listed in the design notes.
"""
import math

__all__ = ["interp_time", "stage_time", "max_batch", "allocate", "dominant_step", "round_latency", "comm_step", "plan", "INF"]

INF = float("inf")


def interp_time(bs, t, y):
    """Time of a layer at batch size y from its profile t[k] at the ascending batch sizes bs[k] (Section 3.3: the profiler
    records FP / BP time for various batch sizes; the relation is not linear).  reading: 0 at y = 0, straight lines between
    profiled sizes (and from the origin to the first), the last segment's line beyond the largest profiled size."""
    if y <= 0:
        return 0.0
    if y <= bs[0]:
        return t[0] * y / bs[0]
    for k in range(1, len(bs)):
        if y <= bs[k]:
            return t[k - 1] + (t[k] - t[k - 1]) * (y - bs[k - 1]) / (bs[k] - bs[k - 1])
    if len(bs) == 1:
        return t[0] * y / bs[0]
    return t[-1] + (t[-1] - t[-2]) * (y - bs[-1]) / (bs[-1] - bs[-2])


def stage_time(prob, dev_type, i, j, y):
    """(sum of FP times, sum of BP times) of layers i..j on a device of `dev_type` with y samples."""
    f = b = 0.0
    for l in range(i, j + 1):
        f += interp_time(prob["bs"], prob["t_f"][dev_type][l], y)
        b += interp_time(prob["bs"], prob["t_b"][dev_type][l], y)
    return f, b


def max_batch(prob, budget, i, j, k_p):
    """Largest number of samples whose footprint Mem = MOD + OPT + K_p * ACT(y) fits `budget` (Eq. (3)); ACT is linear in y."""
    w = sum(prob["w"][l] for l in range(i, j + 1))
    act = sum(prob["act"][l] for l in range(i, j + 1))
    fixed = (prob["mod_factor"] + prob["opt_factor"]) * w
    if budget < fixed:
        return -1                     # not even the model fits
    if act <= 0:
        return 10 ** 9
    return int(math.floor((budget - fixed) / (k_p * act)))


def allocate(prob, group, i, j, k_p):
    """Algorithm 1 for the device list `group` (indices into prob["devices"]) and layers i..j: y_d per device with
    sum y_d = B under every device's memory budget, or None if the micro-batch does not fit.  Returns (y, E_f, E_b)
    with E_f, E_b by Eq. (8)."""
    B = prob["B"]
    devs = prob["devices"]
    cap = {d: max_batch(prob, devs[d]["mem"], i, j, k_p) for d in group}
    if any(c < 0 for c in cap.values()):
        return None
    y = {d: 0 for d in group}
    # Eq. (9): computing capacity = inverse of the FP + BP time of a whole micro-batch
    v = {}
    for d in group:
        f, b = stage_time(prob, devs[d]["type"], i, j, B)
        v[d] = 1.0 / (f + b) if f + b > 0 else INF

    # ---- phase 1: MemoryAwareBalancing(G, beta)
    def balance(G, beta):
        if beta == 0:
            return True
        if len(G) == 0:
            return False
        vs = sum(v[d] for d in G)
        given = 0
        for d in G:
            share = int(math.floor(v[d] / vs * beta)) if vs < INF else beta // len(G)
            take = min(share, cap[d] - y[d])
            y[d] += take
            given += take
        left = beta - given
        if given == 0:
            # reading: shares that all round down to zero would never end the recursion; the fastest device with
            # memory left takes one sample
            cands = [d for d in G if cap[d] - y[d] > 0]
            if not cands:
                return False
            best = cands[0]
            for d in cands[1:]:
                if v[d] > v[best]:
                    best = d
            y[best] += 1
            left -= 1
        return balance([d for d in G if cap[d] - y[d] > 0], left)

    if not balance(list(group), B):
        return None

    def lat(d):
        f, b = stage_time(prob, devs[d]["type"], i, j, y[d])
        return f + b

    # ---- phase 2: StragglerWorkloadOffloading
    block = prob["block"]
    while True:
        order = sorted(group, key=lambda d: (lat(d), d))
        straggler = order[-1]
        old = lat(straggler)
        moved = None
        for d in order[:-1]:                       # fastest first
            n = min(block, y[straggler])
            if n > 0 and cap[d] - y[d] >= n:
                y[straggler] -= n
                y[d] += n
                moved = (d, n)
                break
        if moved is None:
            break
        new = max(lat(d) for d in group)
        if not new < old:
            # the transfer made the slowest device slower (or no faster): take it back and stop
            y[moved[0]] -= moved[1]
            y[straggler] += moved[1]
            break
    ef = eb = 0.0
    for d in group:
        f, b = stage_time(prob, devs[d]["type"], i, j, y[d])
        ef = max(ef, f)
        eb = max(eb, b)
    return [y[d] for d in group], ef, eb


def comm_step(prob, g_a, g_b, cut_layer):
    """Communication step between consecutive stages: (E_f, E_b) = bytes of the boundary tensor of one micro-batch over the
    bandwidth between the groups (Section 3.3).  reading: the slowest link between any device of one group and any of the
    other; FP sends activations, BP the gradient of the same size."""
    bw = min(prob["bw"][a][b] for a in g_a for b in g_b)
    t = prob["B"] * prob["a"][cut_layer] / bw
    return t, t


def dominant_step(steps, M):
    """Index of the step with the fewest bubbles: the largest M (E_f + E_b) after alignment, i.e. plus the FP + BP time of
    every step in front of it (Eq. (11) written for all steps at once; ties go to the earliest step)."""
    best, best_v, pre = 0, -1.0, 0.0
    for s, st in enumerate(steps):
        v = M * (st["ef"] + st["eb"]) + pre
        if v > best_v:
            best, best_v = s, v
        pre += st["ef"] + st["eb"]
    return best


def round_latency(steps, M, dm):
    """Eq. (4): max over steps of T_w + T_e + T_a, with T_w by Eq. (5) and T_e by Eq. (6) for dominant step dm."""
    worst = 0.0
    for s in range(len(steps)):
        tw = sum(steps[i]["ef"] for i in range(s))
        te = M * (steps[dm]["ef"] + steps[dm]["eb"])
        if s < dm:
            te += sum(steps[i]["ef"] + steps[i]["eb"] for i in range(s, dm))
        else:
            te -= sum(steps[i]["ef"] + steps[i]["eb"] for i in range(dm, s))
        worst = max(worst, tw + te + steps[s]["ta"])
    return worst


def allreduce_time(prob, group, i, j):
    """Eq. (5): T_a = 2 (|G| - 1) sum w_l / (|G| min bandwidth inside the group); 0 for a single device."""
    if len(group) < 2:
        return 0.0
    w = sum(prob["w"][l] for l in range(i, j + 1))
    bw = min(prob["bw"][a][b] for a in group for b in group if a != b)
    return 2.0 * (len(group) - 1) * w / (len(group) * bw)


def exec_step(prob, group, i, j, k_p):
    r = allocate(prob, group, i, j, k_p)
    if r is None:
        return None
    y, ef, eb = r
    return {"kind": "exec", "layers": (i, j), "group": list(group), "y": y, "ef": ef, "eb": eb, "ta": allreduce_time(prob, group, i, j)}


def plan(prob):
    """Algorithm 2.  Devices are taken in descending order of memory (earlier stages keep more activations); Q[l][n][p] is
    the best pipeline of the LAST l layers in p stages on the LAST n devices of that order.  Returns the best entry of
    min_p Q(L, N, p): {"latency", "steps", "dm", "stages"} or None if nothing fits."""
    L, N, M = prob["L"], len(prob["devices"]), prob["M"]
    order = sorted(range(N), key=lambda d: (-prob["devices"][d]["mem"], d))
    Q = {}
    for p in range(1, min(L, N) + 1):
        k_p = 2 * p - 1                          # the new head stage is the p-th from the end: K = 2 (P - 0) - 1 with P = p
        for n in range(1, N + 1):
            for l in range(1, L + 1):
                best = None
                for n2 in range(0, n):
                    for l2 in range(0, l):
                        if p == 1:
                            if n2 != 0 or l2 != 0:
                                continue
                            sub = None
                        else:
                            if n2 == 0 or l2 == 0:
                                continue
                            sub = Q.get((l2, n2, p - 1))
                            if sub is None:
                                continue
                        group = order[N - n:N - n2]
                        i, j = L - l, L - l2 - 1
                        ne = exec_step(prob, group, i, j, k_p)
                        if ne is None:
                            continue
                        if sub is None:
                            steps, dm = [ne], 0
                        else:
                            cf, cb = comm_step(prob, group, sub["steps"][0]["group"], j)
                            nc = {"kind": "comm", "ef": cf, "eb": cb, "ta": 0.0}
                            steps = [ne, nc] + sub["steps"]
                            # Eq. (11): the old dominant step (now two places further back), the new execution step
                            # and the new communication step, each aligned by the steps in front of it
                            od = sub["dm"] + 2
                            va = M * (steps[od]["ef"] + steps[od]["eb"]) + sum(s["ef"] + s["eb"] for s in steps[:od])
                            vb = M * (ne["ef"] + ne["eb"])
                            vc = M * (nc["ef"] + nc["eb"]) + (ne["ef"] + ne["eb"])
                            dm = 0
                            top = vb
                            if vc > top:
                                dm, top = 1, vc
                            if va > top:
                                dm, top = od, va
                        lat = round_latency(steps, M, dm)
                        if best is None or lat < best["latency"]:
                            best = {"latency": lat, "steps": steps, "dm": dm}
                if best is not None:
                    Q[(l, n, p)] = best
    out = None
    for p in range(1, min(L, N) + 1):
        c = Q.get((L, N, p))
        if c is not None and (out is None or c["latency"] < out["latency"]):
            out = dict(c, p=p)
    if out is None:
        return None
    out["stages"] = [{"layers": s["layers"], "devices": s["group"], "y": s["y"]} for s in out["steps"] if s["kind"] == "exec"]
    return out
