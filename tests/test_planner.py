"""The library's planner (host C++ behind the C ABI) against the planning oracle: the same hybrid pipeline and the same
estimated HPP-Round latency on seeded synthetic problems, plus the ABI's argument checks.  Needs no GPU."""
import numpy as np
import pytest

import paper_2408_08015_b200 as P
import stage_inputs as si
from oracle import planner as PL


@pytest.fixture(scope="module", autouse=True)
def library():
    P.build()


def same_plan(got, ref):
    if ref is None:
        assert got is None
        return
    assert got is not None
    assert got["latency"] == pytest.approx(ref["latency"], rel=1e-12)
    assert got["dm"] == ref["dm"] and got["n_steps"] == len(ref["steps"])
    assert [(tuple(s["layers"]), s["devices"], s["y"]) for s in got["stages"]] == [(tuple(s["layers"]), s["devices"], s["y"]) for s in ref["stages"]]
    execs = [s for s in ref["steps"] if s["kind"] == "exec"]
    for g, r in zip(got["stages"], execs):
        assert g["ef"] == pytest.approx(r["ef"], rel=1e-12) and g["eb"] == pytest.approx(r["eb"], rel=1e-12) and g["ta"] == pytest.approx(r["ta"], rel=1e-12)


@pytest.mark.parametrize("seed", range(12))
def test_library_plan_equals_the_oracle_plan(seed):
    kw = [dict(L=6, N=3, B=16, M=4), dict(L=8, N=5, B=32, M=8, n_types=3, block=2), dict(L=5, N=4, B=8, M=4, tight_memory=True),
          dict(L=10, N=6, B=24, M=6, n_types=2, tight_memory=True, block=3)][seed % 4]
    prob = si.synthetic_problem(seed, **kw)
    same_plan(P.asteroid_plan(prob), PL.plan(prob))


def test_nothing_fits_and_single_device():
    prob = si.synthetic_problem(3, L=4, N=2, B=8, M=2)
    for d in prob["devices"]:
        d["mem"] = 1.0
    assert P.asteroid_plan(prob) is None and PL.plan(prob) is None
    one = si.synthetic_problem(4, L=4, N=1, B=8, M=3)
    got = P.asteroid_plan(one)
    assert len(got["stages"]) == 1 and got["stages"][0]["y"] == [8] and got["stages"][0]["layers"] == (0, 3)
    ef, eb = PL.stage_time(one, one["devices"][0]["type"], 0, 3, 8)
    assert got["latency"] == pytest.approx(3 * (ef + eb), rel=1e-12)


def test_argument_errors():
    prob = si.synthetic_problem(0, L=4, N=2, B=8, M=2)
    bad = dict(prob, bs=[4, 2, 8, 16, 32, 64])
    with pytest.raises(P.binding.AsteroidError) as e:
        P.asteroid_plan(bad)
    assert e.value.code == P.AST_ERR_ARG
    bad = dict(prob, devices=[{"type": 9, "mem": 1e12}, {"type": 0, "mem": 1e12}])
    with pytest.raises(P.binding.AsteroidError) as e:
        P.asteroid_plan(bad)
    assert e.value.code == P.AST_ERR_ARG
    bad = dict(prob, B=0)
    with pytest.raises(P.binding.AsteroidError) as e:
        P.asteroid_plan(bad)
    assert e.value.code == P.AST_ERR_ARG
