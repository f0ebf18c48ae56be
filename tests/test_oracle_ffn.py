"""Pins for the oracle's expert FFN: it reduces to a dense SwiGLU MLP (library matmul in
double) for a single expert with weight one; it is linear in the combine weights; permuting
the nodes permutes the outputs; shared experts add with weight one."""
import numpy as np
import torch

import oracle


def _weights(rng, E, H, I, bf16):
    gu = 0.05 * rng.standard_normal((E, 2 * I, H))
    dn = 0.05 * rng.standard_normal((E, H, I))
    if bf16:
        return torch.tensor(gu).to(torch.bfloat16), torch.tensor(dn).to(torch.bfloat16)
    return gu.astype(np.float32), dn.astype(np.float32)


def _f64(a):
    return a.to(torch.float64).numpy() if isinstance(a, torch.Tensor) else a.astype(np.float64)


def _dense_mlp(x, gu, dn, e):
    I = dn.shape[2]
    g = _f64(x) @ _f64(gu)[e, :I].T
    u = _f64(x) @ _f64(gu)[e, I:].T
    return ((g / (1.0 + np.exp(-g))) * u) @ _f64(dn)[e].T


def test_single_expert_is_a_dense_swiglu_mlp():
    rng = np.random.default_rng(0)
    for bf16 in (False, True):
        T, H, I, E = 5, 96, 64, 3
        gu, dn = _weights(rng, E, H, I, bf16)
        x = rng.standard_normal((T, H))
        x = torch.tensor(x).to(torch.bfloat16) if bf16 else x.astype(np.float32)
        idx = np.full((T, 1), 2, dtype=np.int32)
        out = oracle.expert_ffn(x, idx, np.ones((T, 1)), gu, dn)
        np.testing.assert_allclose(out, _dense_mlp(x, gu, dn, 2), rtol=1e-10, atol=1e-12)


def test_gate_and_up_halves_are_not_interchangeable():
    # silu(g)*u with g and u swapped differs: guards against reading rows I..2I-1 as the gate
    rng = np.random.default_rng(1)
    gu, dn = _weights(rng, 1, 32, 16, False)
    x = rng.standard_normal((2, 32)).astype(np.float32)
    out = oracle.expert_ffn(x, np.zeros((2, 1), np.int32), np.ones((2, 1)), gu, dn)
    swapped = np.concatenate([gu[:, 16:], gu[:, :16]], axis=1)
    assert np.max(np.abs(out - _dense_mlp(x, swapped, dn, 0))) > 1e-4


def test_weighted_combine_linearity_and_permutation():
    rng = np.random.default_rng(2)
    T, H, I, E, k = 6, 64, 32, 5, 3
    gu, dn = _weights(rng, E, H, I, False)
    x = rng.standard_normal((T, H)).astype(np.float32)
    idx = np.array([rng.permutation(E)[:k] for _ in range(T)], dtype=np.int32)
    w = rng.uniform(0.1, 1.0, (T, k))
    out = oracle.expert_ffn(x, idx, w, gu, dn)
    want = np.zeros((T, H))
    for t in range(T):
        for j in range(k):
            want[t] += w[t, j] * _dense_mlp(x[t:t + 1], gu, dn, idx[t, j])[0]
    np.testing.assert_allclose(out, want, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(oracle.expert_ffn(x, idx, 3.0 * w, gu, dn), 3.0 * out, rtol=1e-12)
    perm = rng.permutation(T)
    np.testing.assert_array_equal(oracle.expert_ffn(x[perm], idx[perm], w[perm], gu, dn), out[perm])
    # an empty slot (-1) contributes nothing
    idx2, w2 = idx.copy(), w.copy()
    idx2[:, 2] = -1
    w0 = w.copy()
    w0[:, 2] = 0.0
    np.testing.assert_allclose(oracle.expert_ffn(x, idx2, w2, gu, dn), oracle.expert_ffn(x, idx, w0, gu, dn),
                               rtol=1e-12, atol=1e-15)


def test_shared_experts_add_with_weight_one():
    rng = np.random.default_rng(3)
    T, H, I, E = 4, 64, 32, 3
    gu, dn = _weights(rng, E, H, I, True)
    sgu, sdn = _weights(rng, 2, H, I, True)
    x = torch.tensor(rng.standard_normal((T, H))).to(torch.bfloat16)
    idx = np.array([[0], [1], [2], [1]], dtype=np.int32)
    w = rng.uniform(0.2, 1.0, (T, 1))
    out = oracle.expert_ffn(x, idx, w, gu, dn, sgu, sdn)
    want = oracle.expert_ffn(x, idx, w, gu, dn)
    want = want + _dense_mlp(x, sgu, sdn, 0) + _dense_mlp(x, sgu, sdn, 1)
    np.testing.assert_allclose(out, want, rtol=1e-10, atol=1e-12)


def test_moe_verify_chains_the_stages():
    rng = np.random.default_rng(4)
    T, H, I, E, k = 6, 64, 32, 8, 2
    gu, dn = _weights(rng, E, H, I, False)
    x = rng.standard_normal((T, H)).astype(np.float32)
    wr = (0.2 * rng.standard_normal((E, H))).astype(np.float32)
    alpha = oracle.node_weights([0, 1, 1, 2, 2, 2], [1.0, 0.8, 0.64])
    res = oracle.moe_verify(x, wr, None, gu, dn, alpha, k)
    z, r, nat = oracle.router(x, wr, None, k)
    sel = oracle.select_eligible(r, nat, alpha)
    idx, w = oracle.route_restricted(z, sel["mask"], k)
    np.testing.assert_array_equal(res["idx"], idx)
    np.testing.assert_array_equal(res["out"], oracle.expert_ffn(x, idx, w, gu, dn))
    # override with every expert eligible = natural routing
    full = np.array([(1 << E) - 1], dtype=np.uint32)
    nat_res = oracle.moe_verify(x, wr, None, gu, dn, alpha, k, mask_override=full)
    np.testing.assert_array_equal(nat_res["idx"], nat)
