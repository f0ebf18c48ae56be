"""Pins for the oracle's elementary pieces: series exp/log against libm in double, the
expert-axis tree sum against exact sums, node weights (Eq. 3) against closed forms."""
import math

import numpy as np
import pytest

import oracle

ULP32 = 2.0 ** -23


def test_series_exp_matches_double_exp():
    x = np.concatenate([np.linspace(-87.0, 5.0, 600_001), -np.logspace(-8, 1.9, 200_000),
                        [0.0, -0.0, 1.0, -1.0]]).astype(np.float32)
    got = oracle.expf(x).astype(np.float64)
    ref = np.exp(x.astype(np.float64))
    assert np.max(np.abs(got - ref) / ref) <= 1.0 * ULP32   # measured 0.64 ulp-units
    assert oracle.expf(0.0)[0] == 1.0


def test_series_exp_is_monotone_on_a_fine_grid():
    x = np.linspace(-20.0, 0.0, 400_001).astype(np.float32)
    y = oracle.expf(x)
    assert np.all(np.diff(y.astype(np.float64)) >= -2 * ULP32 * y[1:])


def test_series_log_matches_double_log():
    rng = np.random.default_rng(7)
    q = np.concatenate([np.exp(rng.uniform(-86.0, 0.0, 600_000)),
                        np.linspace(0.5, 1.0, 200_001)[:-1],
                        [0.5, 0.25, 2.0 ** -126, 0.75, 0.7071, 0.70711, 1.0 - 2.0 ** -24]]).astype(np.float32)
    got = oracle.logf(q).astype(np.float64)
    ref = np.log(q.astype(np.float64))
    assert np.max(np.abs(got - ref) / np.abs(ref)) <= 2.0 * ULP32   # measured 1.6
    assert oracle.logf(1.0)[0] == 0.0
    # exact powers of two: the series part vanishes, e*ln2 rounded once
    for e in range(-126, 1):
        assert oracle.logf(2.0 ** e)[0] == np.float32(e * np.float32(math.log(2.0)))


def test_exp_of_log_roundtrip():
    q = np.linspace(0.01, 1.0, 10_001).astype(np.float32)
    back = oracle.expf(oracle.logf(q)).astype(np.float64)
    assert np.max(np.abs(back - q) / q) < 6 * ULP32


def test_tree_sum_exact_on_dyadic_values():
    rng = np.random.default_rng(3)
    for n in (1, 2, 5, 16, 63, 64, 100, 128):
        v = rng.integers(0, 1024, n).astype(np.float32) / 1024.0   # sums are exact in fp32
        assert oracle.tree_sum(v) == float(np.sum(v.astype(np.float64)))


def test_tree_sum_order_is_the_halving_tree():
    # 1 + 2^-24 + 2^-24 depends on association: the halving tree adds slots 0 and 64 first.
    v = np.zeros(128, dtype=np.float32)
    v[0], v[64], v[1] = 1.0, 2.0 ** -24, 2.0 ** -24
    # (1 + 2^-24) rounds to 1 (ties-to-even); then + 2^-24 (slot 1 joins at the last level) -> 1
    assert oracle.tree_sum(v) == 1.0
    v = np.zeros(128, dtype=np.float32)
    v[0], v[1], v[65] = 1.0, 2.0 ** -24, 2.0 ** -24
    # slots 1 and 65 meet at the first level (2^-23), reach slot 0 at the last: 1 + 2^-23 exactly
    assert oracle.tree_sum(v) == 1.0 + 2.0 ** -23


def test_node_weights_closed_forms():
    # toy tree: widths 1,2,2,3; p_d = 0.8^d with p_0 = 1; beta = 0.5
    depth = [0, 1, 1, 2, 2, 3, 3, 3]
    p = [1.0, 0.8, 0.64, 0.512]
    a = oracle.node_weights(depth, p, beta=0.5, width_norm=True).astype(np.float64)
    want = [1.0] + [math.sqrt(0.8 / 2)] * 2 + [math.sqrt(0.64 / 2)] * 2 + [math.sqrt(0.512 / 3)] * 3
    np.testing.assert_allclose(a, want, rtol=3e-7)
    # aggregate weight of a level grows like sqrt(N_d): sum over level = p^beta * sqrt(N_d)
    assert abs(a[5:].sum() - math.sqrt(0.512) * math.sqrt(3)) < 1e-6
    # beta = 0, no width factor: uniform weights (0^0 = 1 included)
    a0 = oracle.node_weights(depth, [0.0, 0.3, 0.2, 0.1], beta=0.0, width_norm=False)
    assert np.all(a0 == 1.0)
    # beta = 1, no width factor: the table itself
    a1 = oracle.node_weights(depth, p, beta=1.0, width_norm=False)
    np.testing.assert_array_equal(a1, np.float32(p)[depth])
    # chain draft: every level has one node, width factor is 1
    ac = oracle.node_weights([0, 1, 2, 3], [1.0, 0.25, 0.0625, 0.015625], beta=0.5)
    np.testing.assert_array_equal(ac, np.float32([1.0, 0.5, 0.25, 0.125]))


def test_node_weights_rejects_depth_outside_table():
    with pytest.raises(ValueError):
        oracle.node_weights([0, 1, 4], [1.0, 0.5, 0.25, 0.125])
