"""Pins of the planning oracle (Section 3.3: Algorithm 1, Algorithm 2, Eq. (4)-(11)) against closed forms and exhaustive
search on instances small enough to enumerate."""
import itertools

import pytest

import stage_inputs as si
from oracle import planner as PL


def linear_problem(N, B, M, L=3, mem=1e12, t=1.0):
    """Identical devices whose layer time is exactly proportional to the batch size, ample memory, one fat link."""
    bs = [1, 64]
    tf = [[[t * (l + 1) * b for b in bs] for l in range(L)]]
    tb = [[[2 * t * (l + 1) * b for b in bs] for l in range(L)]]
    return {"L": L, "B": B, "M": M, "block": 1, "bs": bs, "t_f": tf, "t_b": tb, "a": [1e3] * L, "w": [1e4] * L, "act": [1e3] * L,
            "mod_factor": 3.0, "opt_factor": 1.0, "devices": [{"type": 0, "mem": mem} for _ in range(N)],
            "bw": [[0.0 if i == j else 1e6 for j in range(N)] for i in range(N)]}


def test_interpolation_is_piecewise_linear_through_the_profile():
    bs, t = [2, 4, 8], [1.0, 1.5, 4.0]
    assert PL.interp_time(bs, t, 0) == 0.0
    assert PL.interp_time(bs, t, 1) == 0.5                 # from the origin to the first profiled size
    assert PL.interp_time(bs, t, 2) == 1.0 and PL.interp_time(bs, t, 4) == 1.5 and PL.interp_time(bs, t, 8) == 4.0
    assert PL.interp_time(bs, t, 3) == 1.25 and PL.interp_time(bs, t, 6) == 2.75
    assert PL.interp_time(bs, t, 12) == 6.5                # the last segment's line continued


def test_single_device_is_one_stage_with_the_whole_micro_batch():
    p = linear_problem(1, 8, 5)
    r = PL.plan(p)
    ef, eb = 8 * (1 + 2 + 3), 2 * 8 * (1 + 2 + 3)
    assert r["p"] == 1 and r["stages"] == [{"layers": (0, 2), "devices": [0], "y": [8]}]
    assert r["latency"] == pytest.approx(5 * (ef + eb))    # Eq. (4)-(6): no waiting, no AllReduce, M compact FP+BP


def test_identical_linear_devices_share_a_micro_batch_equally():
    p = linear_problem(4, 16, 3)
    y, ef, eb = PL.allocate(p, [0, 1, 2, 3], 0, 2, 1)
    assert y == [4, 4, 4, 4] and ef == pytest.approx(4 * 6) and eb == pytest.approx(8 * 6)
    # Eq. (5): 2 (|G|-1)/|G| * sum w / min bandwidth
    assert PL.allreduce_time(p, [0, 1, 2, 3], 0, 2) == pytest.approx(2 * 3 / 4 * 3e4 / 1e6)
    assert PL.allreduce_time(p, [2], 0, 2) == 0.0


def test_memory_budget_caps_a_device_and_an_impossible_budget_fails():
    p = linear_problem(2, 12, 2)
    w, act = 3e4, 3e3
    # device 0 can hold the model plus K * 2 samples only; device 1 is ample
    p["devices"][0]["mem"] = 4.0 * w + 3 * 2 * act + 1.0
    assert PL.max_batch(p, p["devices"][0]["mem"], 0, 2, 3) == 2
    y, _, _ = PL.allocate(p, [0, 1], 0, 2, 3)
    assert y == [2, 10]
    p["devices"][1]["mem"] = 4.0 * w + 3 * 5 * act + 1.0           # 2 + 5 < 12: the micro-batch does not fit
    assert PL.allocate(p, [0, 1], 0, 2, 3) is None
    p["devices"][1]["mem"] = 4.0 * w - 1.0                         # not even the model fits
    assert PL.max_batch(p, p["devices"][1]["mem"], 0, 2, 3) == -1 and PL.allocate(p, [0, 1], 0, 2, 3) is None


def brute_allocation(p, group, i, j, k_p):
    best = None
    caps = [PL.max_batch(p, p["devices"][d]["mem"], i, j, k_p) for d in group]
    for y in itertools.product(*[range(0, min(c, p["B"]) + 1) for c in caps]):
        if sum(y) != p["B"]:
            continue
        t = max(sum(PL.stage_time(p, p["devices"][d]["type"], i, j, yy)) for d, yy in zip(group, y))
        if best is None or t < best:
            best = t
    return best


@pytest.mark.parametrize("seed", range(8))
def test_algorithm1_against_exhaustive_allocation(seed):
    """Algorithm 1 is a heuristic: never better than the optimum of Eq. (7), feasible, complete; with one-sample blocks it
    ends within one sample's worth of time of it on these instances; its second phase never hurts."""
    p = si.synthetic_problem(seed, L=4, N=3, B=9, n_types=2, tight_memory=(seed % 2 == 1))
    group = [0, 1, 2]
    opt = brute_allocation(p, group, 0, 3, 3)
    r = PL.allocate(p, group, 0, 3, 3)
    if opt is None:
        assert r is None
        return
    y, ef, eb = r
    assert sum(y) == p["B"] and all(v >= 0 for v in y)
    for d, yy in zip(group, y):
        assert yy <= PL.max_batch(p, p["devices"][d]["mem"], 0, 3, 3)
    t = max(sum(PL.stage_time(p, p["devices"][d]["type"], 0, 3, yy)) for d, yy in zip(group, y))
    assert t >= opt - 1e-12
    big = dict(p, block=10 ** 6)                                # a block nobody can give away: phase 1 alone
    y1, _, _ = PL.allocate(big, group, 0, 3, 3)
    t1 = max(sum(PL.stage_time(p, p["devices"][d]["type"], 0, 3, yy)) for d, yy in zip(group, y1))
    assert t <= t1 + 1e-12
    assert ef == max(PL.stage_time(p, p["devices"][d]["type"], 0, 3, yy)[0] for d, yy in zip(group, y))      # Eq. (8)


def test_offloading_repairs_a_split_that_ignores_nonlinear_time():
    """Two device types whose full-micro-batch times are equal (equal capacity v_d, Eq. (9)) but whose time curves differ:
    the proportional split of phase 1 is even, phase 2 moves samples off the device that is slow at half a batch."""
    bs = [1, 4, 8]
    p = {"L": 1, "B": 8, "M": 2, "block": 1, "bs": bs, "t_f": [[[1.0, 4.0, 8.0]], [[6.0, 7.0, 8.0]]], "t_b": [[[0.0, 0.0, 0.0]], [[0.0, 0.0, 0.0]]],
         "a": [1.0], "w": [1.0], "act": [1.0], "mod_factor": 1.0, "opt_factor": 0.0,
         "devices": [{"type": 0, "mem": 1e9}, {"type": 1, "mem": 1e9}], "bw": [[0, 1e3], [1e3, 0]]}
    y1, ef1, _ = PL.allocate(dict(p, block=100), [0, 1], 0, 0, 1)
    assert y1 == [4, 4] and ef1 == 7.0
    y, ef, _ = PL.allocate(p, [0, 1], 0, 0, 1)
    assert y == [6, 2] and ef == pytest.approx(6.0 + 1.0 / 3.0)      # type 1 at 2 samples: 6 + 1/3; type 0 at 6: 6
    assert brute_allocation(p, [0, 1], 0, 0, 1) == pytest.approx(6.0 + 1.0 / 3.0)


def test_dominant_step_update_equals_the_all_steps_formula_and_execution_phase_is_a_trapezoid():
    import random
    rnd = random.Random(5)
    for _ in range(200):
        M = rnd.randint(1, 6)
        steps = [{"ef": rnd.random(), "eb": rnd.random(), "ta": rnd.random() * 0.1} for _ in range(rnd.choice([1, 3, 5, 7]))]
        dm = PL.dominant_step(steps, M)
        # brute force of the definition: aligned total FP+BP time, largest first
        vals = [M * (s["ef"] + s["eb"]) + sum(t["ef"] + t["eb"] for t in steps[:k]) for k, s in enumerate(steps)]
        assert vals[dm] == max(vals)
        # Eq. (6): T_e of the dominant step is M compact FP+BP; a step in front starts earlier by what lies between, one behind later
        lat = PL.round_latency(steps, M, dm)
        te = [M * (steps[dm]["ef"] + steps[dm]["eb"]) + (sum(steps[i]["ef"] + steps[i]["eb"] for i in range(s, dm)) if s < dm else
                                                        -sum(steps[i]["ef"] + steps[i]["eb"] for i in range(dm, s))) for s in range(len(steps))]
        tw = [sum(t["ef"] for t in steps[:s]) for s in range(len(steps))]
        assert lat == pytest.approx(max(a + b + s["ta"] for a, b, s in zip(tw, te, steps)))


def exhaustive_plan(p, max_stages):
    """Every contiguous cut of the layers into at most max_stages stages and every contiguous grouping of the devices (in
    descending order of memory), each stage allocated by Algorithm 1, the round judged by Eq. (4)-(6)."""
    L, N, M = p["L"], len(p["devices"]), p["M"]
    order = sorted(range(N), key=lambda d: (-p["devices"][d]["mem"], d))
    best = None
    for P in range(1, min(L, N, max_stages) + 1):
        for lc in itertools.combinations(range(1, L), P - 1):
            for dc in itertools.combinations(range(1, N), P - 1):
                lb, db = (0,) + lc + (L,), (0,) + dc + (N,)
                steps, ok = [], True
                for s in range(P):
                    ne = PL.exec_step(p, order[db[s]:db[s + 1]], lb[s], lb[s + 1] - 1, 2 * (P - s) - 1)
                    if ne is None:
                        ok = False
                        break
                    if steps:
                        cf, cb = PL.comm_step(p, steps[-1]["group"], ne["group"], lb[s] - 1)
                        steps.append({"kind": "comm", "ef": cf, "eb": cb, "ta": 0.0})
                    steps.append(ne)
                if not ok:
                    continue
                lat = PL.round_latency(steps, M, PL.dominant_step(steps, M))
                if best is None or lat < best:
                    best = lat
    return best


@pytest.mark.parametrize("seed", range(6))
def test_dynamic_program_against_exhaustive_search(seed):
    """With two devices (at most two stages) the dynamic program sees every configuration: it must return the exhaustive
    optimum.  With four it composes optimal sub-pipelines, which the latency of Eq. (4) does not strictly allow: it
    may not beat the exhaustive optimum and stays close to it."""
    p2 = si.synthetic_problem(seed, L=5, N=2, B=8, M=4)
    r2 = PL.plan(p2)
    assert r2["latency"] == pytest.approx(exhaustive_plan(p2, 2), rel=1e-12)
    p4 = si.synthetic_problem(100 + seed, L=5, N=4, B=8, M=4, tight_memory=(seed % 2 == 0))
    r4, ex = PL.plan(p4), exhaustive_plan(p4, 4)
    if ex is None:
        assert r4 is None
        return
    assert r4 is not None and r4["latency"] >= ex * (1 - 1e-12) and r4["latency"] <= 1.25 * ex
    # the returned plan is self-consistent: every layer once, every device once, every micro-batch whole
    assert [s["layers"][0] for s in r4["stages"]] == [0] + [s["layers"][1] + 1 for s in r4["stages"][:-1]] and r4["stages"][-1]["layers"][1] == 4
    assert sorted(d for s in r4["stages"] for d in s["devices"]) == [0, 1, 2, 3]
    assert all(sum(s["y"]) == 8 for s in r4["stages"])
    assert r4["dm"] == PL.dominant_step(r4["steps"], 4)          # Eq. (11), applied stage by stage, agrees with the all-steps form
