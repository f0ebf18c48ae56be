"""CPU checks of the C-ABI library: it loads, exports every symbol the header declares, and its
pure-host entry points behave (no compute calls without a GPU)."""
import re
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
from paper_2608_02989_b200 import acm, build as acm_build

HEADER = Path(__file__).resolve().parent.parent / "include" / "acm.h"


@pytest.fixture(scope="module")
def lib():
    acm_build.build_library()
    return acm.load_library()


def test_every_declared_symbol_is_exported(lib):
    text = re.sub(r"/\*.*?\*/", "", HEADER.read_text(), flags=re.S)
    declared = set(re.findall(r"\b(acm_[a-z0-9_]+)\s*\(", text))
    assert declared == set(acm.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert acm.status_string(acm.OK) == "ok"
    assert "wait" in acm.status_string(acm.ERR_TIMEOUT)
    assert len({acm.status_string(c) for c in range(7)}) == 7


def test_default_select_params(lib):
    p = acm.SelectParams(demand=2, use_anchors=0, fixed_budget=9, ceil_guard=0.0, residency=2, max_remove=1)
    lib.acm_default_select_params(p)
    assert (p.demand, p.use_anchors, p.fixed_budget, p.residency, p.max_remove) == (0, 1, 0, 0, 128)
    assert p.ceil_guard == 2.0 ** -10


def test_node_weights_host_helper_matches_oracle_bitwise(lib):
    rng = np.random.default_rng(0)
    for _ in range(50):
        D = int(rng.integers(1, 9))
        T = int(rng.integers(1, 65))
        depth = torch.tensor(np.sort(rng.integers(0, D + 1, T)), dtype=torch.int32)
        p = torch.tensor(rng.uniform(0.01, 1.0, D + 1), dtype=torch.float32)
        beta = float(rng.choice([0.0, 0.25, 0.5, 1.0, 2.0]))
        wn = bool(rng.integers(0, 2))
        got = acm.node_weights(depth, p, beta, wn).numpy()
        want = oracle.node_weights(depth.numpy(), p.numpy(), beta, wn)
        np.testing.assert_array_equal(got, want)


def test_node_weights_rejects_bad_depth(lib):
    with pytest.raises(acm.AcmError) as e:
        acm.node_weights(torch.tensor([0, 5], dtype=torch.int32), torch.tensor([1.0, 0.5]))
    assert e.value.code == acm.ERR_INVALID


def test_create_rejects_bad_descriptions_before_touching_the_gpu(lib):
    def create(**kw):
        d = dict(hidden=256, n_experts=16, top_k=2, inter=128, n_shared=0, max_nodes=64, n_layers=1, dtype=acm.BF16,
                 weighting=0, routed_scale=1.0)
        d.update(kw)
        desc = acm.ModelDesc(*d.values())
        h = acm.c_void_p()
        return lib.acm_create(acm.byref(desc), acm.byref(h))

    assert create(top_k=17) == acm.ERR_INVALID
    assert create(n_experts=0) == acm.ERR_INVALID
    assert create(dtype=7) == acm.ERR_INVALID
    assert create(n_experts=129) == acm.ERR_UNSUPPORTED
    assert create(top_k=9) == acm.ERR_UNSUPPORTED
    assert create(max_nodes=65) == acm.ERR_UNSUPPORTED
    assert create(hidden=192) == acm.ERR_UNSUPPORTED
    assert create(inter=96) == acm.ERR_UNSUPPORTED
    assert lib.acm_create(None, None) == acm.ERR_INVALID


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_no_silent_fallback_without_a_gpu(lib):
    with pytest.raises(acm.AcmError) as e:
        acm.Context(256, 16, 2, 128)
    assert e.value.code in (acm.ERR_CUDA, acm.ERR_UNSUPPORTED)
