"""CPU-side checks of the product: the C-ABI library loads, exports every declared symbol, and
fails loudly without a device."""
import os
import re

import pytest

import paper_2408_08015_b200 as P
import stage_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def library():
    P.build()
    return P.lib()


def test_every_declared_symbol_is_exported(library):
    hdr = open(os.path.join(ROOT, "include", "asteroid.h")).read()
    declared = set(re.findall(r"\b(asteroid_[a-z0-9_]+)\s*\(", hdr))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(library, name), name
    assert declared == set(P.binding.EXPORTS)


def test_op_codes_agree_with_header():
    hdr = open(os.path.join(ROOT, "include", "asteroid.h")).read()
    for name, code in P.binding.OP_CODES.items():
        cname = {"add": "AST_ADD"}.get(name, "AST_" + name.upper())
        assert re.search(r"%s\s*=\s*%d\b" % (cname, code), hdr), name
    assert si.OPS == P.binding.OP_CODES


def test_no_device_is_a_loud_error(library):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(P.binding.AsteroidError) as e:
        P.asteroid_stage_create(si.block_net(), 0, 8, 32, 32, 8, 4)
    assert e.value.code == P.AST_ERR_CUDA
    assert P.asteroid_stage_param_count(None) == 0
