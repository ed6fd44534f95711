"""The seeded input generators: mixing function against published values, distributions,
bfloat16 rounding, network descriptions."""
import os

import numpy as np

import stage_inputs as si
from stage_inputs.rng import _mix, _GOLDEN

HERE = os.path.dirname(os.path.abspath(__file__))


def test_splitmix64_published_sequence():
    want = [int(l, 16) for l in open(os.path.join(HERE, "golden", "splitmix64.txt")) if not l.startswith("#")]
    with np.errstate(over="ignore"):
        got = [int(_mix(_GOLDEN * np.uint64(i + 1))) for i in range(3)]
    assert got == want


def test_streams_are_deterministic_and_distinct():
    a = si.normal(0, 5, (4, 3)); b = si.normal(0, 5, (4, 3)); c = si.normal(0, 6, (4, 3)); d = si.normal(1, 5, (4, 3))
    assert (a == b).all() and (a != c).any() and (a != d).any()
    z = si.normal(0, 1, (400000,))
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01 and abs((z ** 3).mean()) < 0.02 and abs((z ** 4).mean() - 3) < 0.05
    u = si.uniform(0, 2, 200000)
    assert 0 < u.min() and u.max() < 1 and abs(u.mean() - 0.5) < 0.005
    lab = si.labels(0, 3, 100000, 1000)
    assert lab.min() >= 0 and lab.max() <= 999 and len(np.unique(lab)) == 1000


def test_bf16_rounding_is_nearest_even():
    one = np.float32(1.0)
    eps = np.float32(2.0 ** -7)          # bf16 spacing at 1.0
    v = np.array([1.0, 1.0 + eps / 2, 1.0 + eps * 1.5, 1.0 + eps * 0.75, -3.1415926], np.float32)
    r = si.round_to_bf16(v)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == one + 2 * eps and r[3] == one + eps
    assert abs(r[4] + 3.140625) < 1e-7
    x = si.normal(0, 9, (1000,)).astype(np.float32)
    assert (si.round_to_bf16(si.round_to_bf16(x)) == si.round_to_bf16(x)).all()
    assert np.abs(si.round_to_bf16(x) - x).max() <= np.abs(x).max() * 2.0 ** -8


def test_workload_descriptions():
    sizes = {"c1": (si.block_net(), 32, 4352, 4.03e6), "c2": (si.stage_net_mbv2_4blocks(), 56, 42512, 77.9e6),
             "c3": (si.mobilenetv2_net(), 224, 3504872, 300.8e6), "c4": (si.resnet50_c2c3_net(), 56, 1435392, 1695.5e6)}
    for name, (net, h, params, macs) in sizes.items():
        n = len(net)
        assert si.param_count(net, 0, n - 1) == params
        assert abs(sum(si.forward_macs(net, 0, n - 1, h, h).values()) - macs) / macs < 1e-3
    net = si.mobilenetv2_net()
    assert sum(1 for l in net if l.op == "add") == 10 and sum(1 for l in net if l.op in ("conv", "dwconv")) == 52
    units = si.mobilenetv2_units()
    assert len(units) == 19
    for P in (2, 3, 4, 6):
        cuts = si.partition_units(net, units, P, 224, 224)
        assert len(cuts) == P and cuts[0][0] == 0 and cuts[-1][1] == len(net) - 1
        assert all(cuts[i][1] + 1 == cuts[i + 1][0] for i in range(P - 1))
        for f, l in cuts:          # a cut never separates a residual add from its block input
            assert all(net[i].src >= f - 1 and (net[i].op != "add" or net[i].add_from >= f - 1) for i in range(f, l + 1))
