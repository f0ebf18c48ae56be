"""Pins for the oracle's router stage (Section 3.1): logits against a double dot product,
softmax against its definition, natural top-k against brute force."""
import numpy as np
import torch

import oracle
from tests.helpers import topk_brute


def _bf16_bits(a):
    return torch.tensor(a, dtype=torch.float32).to(torch.bfloat16)


def test_logits_match_double_dot_product_fp32():
    rng = np.random.default_rng(0)
    T, H, E, k = 8, 256, 16, 2
    x = rng.standard_normal((T, H)).astype(np.float32)
    w = (0.02 * rng.standard_normal((E, H))).astype(np.float32)
    b = rng.standard_normal(E).astype(np.float32)
    z, r, nat = oracle.router(x, w, b, k)
    ref = x.astype(np.float64) @ w.astype(np.float64).T + b.astype(np.float64)
    np.testing.assert_allclose(z, ref, rtol=0, atol=2e-6)
    z0, _, _ = oracle.router(x, w, None, k)
    np.testing.assert_allclose(z0, ref - b, rtol=0, atol=1e-6)
    # transposed operands would not even agree in shape-compatible cases: check one entry by hand
    assert abs(z0[3, 5] - float(np.dot(x[3].astype(np.float64), w[5].astype(np.float64)))) < 1e-6


def test_logits_match_double_dot_product_bf16():
    rng = np.random.default_rng(1)
    T, H, E, k = 5, 192, 12, 3
    x = _bf16_bits(rng.standard_normal((T, H)))
    w = _bf16_bits(0.02 * rng.standard_normal((E, H)))
    z, _, _ = oracle.router(x, w, None, k)
    ref = x.to(torch.float64).numpy() @ w.to(torch.float64).numpy().T
    np.testing.assert_allclose(z, ref, rtol=0, atol=2e-6)


def test_logits_exact_on_small_integers():
    # integer-valued inputs: every partial sum is exact, so any summation order gives the same
    rng = np.random.default_rng(2)
    x = rng.integers(-8, 9, (4, 96)).astype(np.float32)
    w = rng.integers(-8, 9, (6, 96)).astype(np.float32)
    z, _, _ = oracle.router(x, w, None, 2)
    np.testing.assert_array_equal(z, (x.astype(np.int64) @ w.astype(np.int64).T).astype(np.float32))


def test_logit_summation_order_is_32_interleaved_partials():
    # x.w = 2^24 + 1 + 1 with the three terms placed so that the outcome depends on association.
    # partial 0 gets 2^24 (h=0) then +1 (h=32): 2^24+1 rounds to 2^24 (tie to even).
    # partial 1 gets 1 (h=1).  tree: slot0 + slot1 at the last level -> 2^24 + 1 -> 2^24.
    H = 64
    x = np.zeros((1, H), dtype=np.float32)
    w = np.ones((1, H), dtype=np.float32)
    x[0, 0], x[0, 32], x[0, 1] = 2.0 ** 24, 1.0, 1.0
    z, _, _ = oracle.router(x, w, None, 1)
    assert z[0, 0] == 2.0 ** 24
    # moving the second unit from h=32 to h=17 puts it in partial 17, which meets partial 1
    # at the first tree level (1+1 = 2) and reaches slot 0 as 2: 2^24 + 2 exactly.
    x[0, 32], x[0, 17] = 0.0, 1.0
    z, _, _ = oracle.router(x, w, None, 1)
    assert z[0, 0] == 2.0 ** 24 + 2.0


def test_softmax_and_topk():
    rng = np.random.default_rng(3)
    T, H, E, k = 16, 128, 24, 4
    x = rng.standard_normal((T, H)).astype(np.float32)
    w = (0.3 * rng.standard_normal((E, H))).astype(np.float32)
    z, r, nat = oracle.router(x, w, None, k)
    zd = z.astype(np.float64)
    ref = np.exp(zd - zd.max(1, keepdims=True))
    ref /= ref.sum(1, keepdims=True)
    # |z - max| reaches ~20 here, so rounding that difference to fp32 alone moves exp by ~1e-6 relative
    np.testing.assert_allclose(r, ref, rtol=2e-6, atol=0)
    assert np.all(np.abs(r.astype(np.float64).sum(1) - 1.0) < 1e-6)
    for t in range(T):
        assert list(nat[t]) == topk_brute(z[t], k)
        # softmax is monotone: ordering of probabilities never contradicts ordering of logits
        order = np.argsort(-z[t], kind="stable")
        assert np.all(np.diff(r[t][order]) <= 0)


def test_topk_ties_go_to_lower_index():
    H, E = 32, 8
    x = np.ones((1, H), dtype=np.float32)
    w = np.zeros((E, H), dtype=np.float32)
    w[[1, 4, 6], 0] = 1.0          # three experts tie at logit 1, the rest at 0
    _, r, nat = oracle.router(x, w, None, 5)
    assert list(nat[0]) == [1, 4, 6, 0, 2]
    assert r[0, 1] == r[0, 4] == r[0, 6]
