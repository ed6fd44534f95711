"""The per-layer profile record and the partitioned (config-5 style) stages at full resolution."""
import numpy as np
import pytest

import oracle as O
import stage_inputs as si
from harness import ALL, bf16_store, compare, gpu_round, make_inputs, oracle_round, summary

pytestmark = pytest.mark.gpu


def test_profile_record_closed_forms_and_memory_terms():
    import torch
    import paper_2408_08015_b200 as P
    net = si.stage_net_mbv2_4blocks()
    first, last, h, w, B, M, K = 0, len(net) - 1, 56, 56, 8, 4, 3
    free0 = torch.cuda.mem_get_info()[0]
    hdl = P.asteroid_stage_create(net, first, last, h, w, B, M, dtype=P.AST_BF16, slots=K)
    free1 = torch.cuda.mem_get_info()[0]
    try:
        P.asteroid_stage_import_state(hdl, si.init_params(net, first, last, 0))
        recs = {l: P.asteroid_stage_profile(hdl, l, B) for l in range(first, last + 1)}
        for l, r in recs.items():
            ref = O.layer_profile(net, first, last, h, w, l, B, 2)
            assert r["a_l_bytes"] == ref["a_l"] and r["w_l_bytes"] == ref["w_l"] and r["flops"] == ref["flops"], (l, r, ref)
            if net[l].op in ("conv", "dwconv"):
                assert r["t_f_ms"] > 0 and r["t_b_ms"] > 0 and r["alg_bytes_f"] > 0 and r["alg_bytes_b"] > r["alg_bytes_f"]
            # no record may claim more than the memory system can deliver (a fused BatchNorm reports its finishing kernel only)
            for t, nb in ((r["t_f_ms"], r["alg_bytes_f"]), (r["t_b_ms"], r["alg_bytes_b"])):
                if t > 0:
                    assert nb / (t * 1e-3) < 8e12, (l, net[l].op, r)
            if net[l].op in ("relu6", "relu"):
                assert r["t_f_ms"] == 0 and r["fused_into"] == l - 1
        r0 = recs[first]
        # Eq. (3): Mem = MOD + OPT + K * ACT(beta); with the transient workspace it is what the stage allocated
        total = O.stage_memory(r0["mem_mod"], r0["mem_opt"], r0["mem_act"], K) + r0["mem_work"]
        assert abs((free0 - free1) - total) <= 48 << 20, (free0 - free1, total)
        # activation memory is proportional to the micro-batch size (up to alignment and the statistics vectors)
        r2 = P.asteroid_stage_profile(hdl, first, 2 * B)
        assert abs(r2["mem_act"] - 2 * r0["mem_act"]) <= 0.01 * r2["mem_act"]
        # time is not linear in the batch size: a tiny batch under-uses the GPU (Section 3.3)
        conv = [l for l in range(first, last + 1) if net[l].op == "dwconv"][0]
        t1 = P.asteroid_stage_profile(hdl, conv, 1)["t_f_ms"]
        t32 = P.asteroid_stage_profile(hdl, conv, 32)["t_f_ms"]
        assert t32 < 16 * t1
    finally:
        P.asteroid_stage_destroy(hdl)


@pytest.mark.parametrize("parts", [2, 6])
def test_full_resolution_partitions_match_oracle(parts):
    """MobileNetV2 at 224x224 cut into `parts` stages, each run alone at micro-batch 4 (M=2, bfloat16)."""
    net = si.mobilenetv2_net()
    cuts = si.partition_units(net, si.mobilenetv2_units(), parts, 224, 224)
    shapes = si.out_shape(net, 0, len(net) - 1, 224, 224)
    B, M = 4, 2
    for first, last in cuts:
        h, w, _ = shapes[first - 1] if first > 0 else (224, 224, 3)
        loss = "xent" if last == len(net) - 1 else "mse"
        xs, tg, params, _ = make_inputs(net, first, last, h, w, B, M, loss, 1, True)
        mirror = oracle_round(net, first, last, B, M, loss, xs, tg, params, store=bf16_store)
        plain = oracle_round(net, first, last, B, M, loss, xs, tg, params)
        gpu = gpu_round(net, first, last, h, w, B, M, loss, xs, tg, params, True, need_dx=int(first > 0))
        print((first, last), summary(compare(gpu, plain, net, first, last, 2e-2, need_dx=first > 0, mirror=mirror, allow=ALL, outlier_frac=5e-4,
                                             case="config5/P%d/%d-%d/B4" % (parts, first, last),
                                             contract_kinds=("loss",) if parts == 2 else ("y", "loss"))))


def test_planner_on_measured_cost_tables_equals_the_oracle():
    """Section 3.3 end to end: profile a small network's block-level units on this GPU at three batch sizes, hand the tables
    to the library's planner and to the planning oracle with the same synthetic device pool: same pipeline, same latency."""
    import paper_2408_08015_b200 as P
    from paper_2408_08015_b200.sweep import plan_problem, unit_cost_tables
    from oracle import planner as PL
    net, units = si.small_mobilenet(10)
    batches = [2, 4, 8]
    tabs = unit_cost_tables(P, si, net, units, 32, 32, batches)
    assert all(t > 0 for row in tabs[0] for t in row) and all(t > 0 for row in tabs[1] for t in row)
    for kw in ({"devices": ((0, 1e9), (1, 1e9), (2, 1e9)), "B": 8, "M": 4, "block": 1},
               {"devices": ((0, 2e5), (1, 1.5e5), (1, 1.5e5), (2, 1e5)), "B": 8, "M": 4, "block": 1, "bytes_per_ms": 1e3}):
        prob = plan_problem(*tabs, batches, **kw)
        got, ref = P.asteroid_plan(prob), PL.plan(prob)
        assert (got is None) == (ref is None)
        if ref is not None:
            assert got["latency"] == pytest.approx(ref["latency"], rel=1e-12)
            assert [(tuple(s["layers"]), s["devices"], s["y"]) for s in got["stages"]] == [(tuple(s["layers"]), s["devices"], s["y"]) for s in ref["stages"]]
            print(kw["devices"], "->", [(s["layers"], s["devices"], s["y"]) for s in got["stages"]], "%.3f ms" % got["latency"])
