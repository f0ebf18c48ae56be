"""Pins for the oracle's selector (Sections 3.2-3.4): closed forms for demand (Eq. 4) and the
effective-rank cardinality (Eq. 6), the stated special cases, the invariants the method
fixes, and brute force for the pruning rule (Eq. 7) -- all on tiny inputs."""
from itertools import combinations
from pathlib import Path

import numpy as np
import pytest

import oracle
from oracle import SelectParams
from tests.helpers import full_mask, mask_to_set, set_to_mask, topk_brute

GOLDEN = Path(__file__).parent / "golden" / "effective_rank_cases.txt"


def _softmax_rows(rng, T, E, scale=2.0):
    z = (scale * rng.standard_normal((T, E))).astype(np.float32)
    p = np.exp(z.astype(np.float64) - z.max(1, keepdims=True))
    return z, (p / p.sum(1, keepdims=True)).astype(np.float32)


def _nat(z, k):
    return np.array([topk_brute(row, k) for row in z], dtype=np.int32)


# ------------------------------------------------------------------ demand (Eq. 4)
def test_demand_closed_form_on_dyadic_inputs():
    # 3 nodes, 4 experts, k = 2.  alpha and r are powers of two so every fp32 operation is exact.
    r = np.array([[0.5, 0.25, 0.125, 0.125],
                  [0.125, 0.5, 0.25, 0.125],
                  [0.25, 0.125, 0.5, 0.125]], dtype=np.float32)
    nat = np.array([[0, 1], [1, 2], [2, 0]], dtype=np.int32)
    alpha = np.array([1.0, 0.5, 0.25], dtype=np.float32)
    prm = SelectParams(use_anchors=0)
    d = oracle.select_eligible(r, nat, alpha, prm)["demand"]
    # only entries inside each node's natural top-k count
    want = [1.0 * 0.5 + 0.25 * 0.25, 1.0 * 0.25 + 0.5 * 0.5, 0.5 * 0.25 + 0.25 * 0.5, 0.0]
    assert list(d) == want
    # full-mass mode drops the indicator
    d1 = oracle.select_eligible(r, nat, alpha, SelectParams(demand=1, use_anchors=0))["demand"]
    np.testing.assert_array_equal(d1, (alpha[:, None].astype(np.float64) * r).sum(0).astype(np.float32))
    # vote mode counts natural assignments
    d2 = oracle.select_eligible(r, nat, alpha, SelectParams(demand=2, use_anchors=0))["demand"]
    assert list(d2) == [2.0, 2.0, 2.0, 0.0]


def test_demand_accumulates_in_node_order_in_fp32():
    # u = fma(a2, r2, fma(a1, r1, fma(a0, r0, 0))): 2^24, then +1 (lost to rounding), then +1 (lost)
    r = np.array([[1.0], [1.0], [1.0]], dtype=np.float32)
    nat = np.zeros((3, 1), dtype=np.int32)
    up = oracle.select_eligible(r, nat, np.float32([2.0 ** 24, 1.0, 1.0]), SelectParams(use_anchors=0))
    assert up["demand"][0] == 2.0 ** 24
    down = oracle.select_eligible(r, nat, np.float32([1.0, 1.0, 2.0 ** 24]), SelectParams(use_anchors=0))
    assert down["demand"][0] == 2.0 ** 24 + 2.0


def test_scaling_alpha_by_two_leaves_the_set_unchanged():
    rng = np.random.default_rng(5)
    for _ in range(50):
        T, E, k = 6, 12, 2
        z, r = _softmax_rows(rng, T, E)
        nat = _nat(z, k)
        alpha = rng.uniform(0.1, 1.0, T).astype(np.float32)
        a = oracle.select_eligible(r, nat, alpha)
        for s in (2.0, 0.5, 8.0):
            b = oracle.select_eligible(r, nat, (alpha * np.float32(s)).astype(np.float32))
            np.testing.assert_array_equal(a["mask"], b["mask"])
            assert a["stats"]["n_er"] == b["stats"]["n_er"]


# ------------------------------------------------------------------ effective rank (Eq. 6)
def _golden_cases():
    for line in GOLDEN.read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        lhs, rhs = line.split("->")
        yield [float(v) for v in lhs.split()], int(rhs)


@pytest.mark.parametrize("demands,want", list(_golden_cases()))
def test_effective_rank_golden(demands, want):
    # one node, full-mass demand, no anchors: u_e equals the given vector; two zero-demand experts appended
    u = np.array(demands + [0.0, 0.0], dtype=np.float32)
    r = u[None, :]
    nat = np.array([[int(np.argmax(u))]], dtype=np.int32)
    res = oracle.select_eligible(r, nat, np.float32([1.0]), SelectParams(demand=1, use_anchors=0))
    assert res["stats"]["n_er"] == want
    assert res["count"] == want
    order = sorted(range(len(u)), key=lambda e: (-u[e], e))
    assert mask_to_set(res["mask"], len(u)) == set(order[:want])


@pytest.mark.parametrize("E", [8, 40, 128])
def test_uniform_demand_over_m_experts_gives_m(E):
    for m in range(1, E + 1):
        u = np.zeros(E, dtype=np.float32)
        u[:m] = 0.37
        res = oracle.select_eligible(u[None, :], np.zeros((1, 1), np.int32), np.float32([1.0]),
                                     SelectParams(demand=1, use_anchors=0))
        assert res["stats"]["n_er"] == m, m


def test_ceiling_guard_at_integer_boundary():
    # exp(H) = 4 analytically (H = 2 ln 2); a sixth expert with positive demand keeps the clamp
    # to the number of positive experts out of the way.
    exact = np.float32([0.5, 0.125, 0.125, 0.125, 0.125, 0.0])
    res = oracle.select_eligible(exact[None, :], np.zeros((1, 1), np.int32), np.float32([1.0]),
                                 SelectParams(demand=1, use_anchors=0))
    assert res["stats"]["n_er"] == 4
    assert abs(res["stats"]["perplexity"] - 4.0) < 1e-4
    assert abs(res["stats"]["entropy"] - 2 * np.log(2.0)) < 1e-6
    # the literal rule (guard 0) is ceil of whatever fp32 value exp(H) took
    overshoot = 0
    for m in range(2, 100):
        u = np.zeros(128, dtype=np.float32)
        u[:m] = 0.37
        u[m] = 2.0 ** -60          # positive but negligible: allows n_er = m + 1
        lit = oracle.select_eligible(u[None, :], np.zeros((1, 1), np.int32), np.float32([1.0]),
                                     SelectParams(demand=1, use_anchors=0, ceil_guard=0.0))
        grd = oracle.select_eligible(u[None, :], np.zeros((1, 1), np.int32), np.float32([1.0]),
                                     SelectParams(demand=1, use_anchors=0))
        assert grd["stats"]["n_er"] == m
        assert lit["stats"]["n_er"] == int(np.ceil(np.float32(lit["stats"]["perplexity"])))
        overshoot += lit["stats"]["n_er"] == m + 1
    assert overshoot > 0     # rounding does push exp(H) above the integer for some m: the guard matters


def test_zero_residual_keeps_only_what_min_size_needs():
    # every node routes to the root's experts: residual demand is zero, S = A
    E, k, T = 8, 2, 4
    r = np.zeros((T, E), dtype=np.float32)
    r[:, 3], r[:, 5] = 0.6, 0.4
    nat = np.tile(np.int32([3, 5]), (T, 1))
    res = oracle.select_eligible(r, nat, np.ones(T, np.float32))
    assert mask_to_set(res["mask"], E) == {3, 5} and res["stats"]["n_er"] == 0
    assert res["stats"]["residual_mass"] == 0.0
    # without anchors the min-size rule fills up with the lowest-index zero-demand experts
    zero = np.zeros((T, E), dtype=np.float32)
    res = oracle.select_eligible(zero, nat, np.ones(T, np.float32), SelectParams(use_anchors=0))
    assert mask_to_set(res["mask"], E) == {0, 1} and res["count"] == k


def test_single_node_block_is_vanilla_decoding():
    rng = np.random.default_rng(11)
    z, r = _softmax_rows(rng, 1, 16)
    nat = _nat(z, 4)
    res = oracle.select_eligible(r, nat, np.float32([1.0]))
    assert mask_to_set(res["mask"], 16) == set(nat[0])
    idx, w = oracle.route_restricted(z, res["mask"], 4)
    assert list(idx[0]) == list(nat[0])
    assert abs(w.sum() - 1.0) < 1e-12


# ------------------------------------------------------------------ invariants on random tiny blocks
def test_invariants_brute_force():
    rng = np.random.default_rng(2024)
    for trial in range(3000):
        E = int(rng.integers(3, 9))
        k = int(rng.integers(1, min(E, 4) + 1))
        T = int(rng.integers(1, 6))
        z, r = _softmax_rows(rng, T, E, scale=float(rng.uniform(0.2, 4.0)))
        nat = _nat(z, k)
        alpha = rng.uniform(0.05, 1.0, T).astype(np.float32)
        res = oracle.select_eligible(r, nat, alpha)
        S = mask_to_set(res["mask"], E)
        st = res["stats"]
        # (i) the root's natural top-k is always eligible; (v) |S| >= |A|, |S| >= k
        assert set(nat[0]) <= S
        assert len(S) == res["count"] == st["n_eligible"] >= max(st["n_anchor"], k)
        assert st["n_anchor"] == k
        assert len(S) == (k + st["n_er"] if st["residual_mass"] > 0.0 else k)
        # every retained non-anchor outranks every dropped one
        u = res["demand"]
        kept = [e for e in S if e not in set(nat[0])]
        dropped = [e for e in range(E) if e not in S]
        for a in kept:
            for b in dropped:
                assert (u[a], -a) > (u[b], -b)
        # (ii) restricted routes stay inside S, and equal brute-force top-k over S
        idx, w = oracle.route_restricted(z, res["mask"], k)
        for t in range(T):
            assert set(idx[t]) <= S
            assert list(idx[t]) == topk_brute(z[t], k, S)
            assert abs(w[t].sum() - 1.0) < 1e-9
        # (iii) with every expert eligible, restricted routing is natural routing
        idx_all, _ = oracle.route_restricted(z, full_mask(E), k)
        np.testing.assert_array_equal(idx_all, nat)
        # displaced assignments a(S) by set algebra
        votes = np.bincount(nat.ravel(), minlength=E)
        assert st["displaced_aS"] == sum(int(votes[e]) for e in range(E) if e not in S)
        assert st["n_natural_union"] == int((votes > 0).sum())


def test_uniform_weights_fixed_budget_full_mass_is_equal_weight_top_b():
    """Uniform node weights + fixed budget B + full router mass (anchors off) is the
    equal-weight aggregation of router mass over the block, top B (the MoE-Spec rule)."""
    rng = np.random.default_rng(77)
    for trial in range(2000):
        E = int(rng.integers(3, 9))
        k = int(rng.integers(1, min(E, 3) + 1))
        T = int(rng.integers(1, 6))
        B = int(rng.integers(k, E + 1))
        # dyadic probabilities: column sums are exact in any order, so ranks are unambiguous
        r = (rng.integers(0, 256, (T, E)) / 256.0).astype(np.float32)
        z = r.copy()
        nat = _nat(z, k)
        res = oracle.select_eligible(r, nat, np.ones(T, np.float32),
                                     SelectParams(demand=1, use_anchors=0, fixed_budget=B))
        mass = r.astype(np.float64).sum(0)
        top_b = set(sorted(range(E), key=lambda e: (-mass[e], e))[:B])
        assert mask_to_set(res["mask"], E) == top_b
        # with anchors on, the identity holds exactly when the anchors are inside that top-B
        res_a = oracle.select_eligible(r, nat, np.ones(T, np.float32),
                                       SelectParams(demand=1, use_anchors=1, fixed_budget=B))
        Sa = mask_to_set(res_a["mask"], E)
        assert set(nat[0]) <= Sa and len(Sa) == max(B, k)
        if set(nat[0]) <= top_b:
            assert Sa == top_b


def test_fixed_budget_holds_total_size_with_anchors():
    rng = np.random.default_rng(9)
    z, r = _softmax_rows(rng, 5, 16)
    nat = _nat(z, 2)
    alpha = np.float32([1.0, 0.8, 0.8, 0.6, 0.6])
    for B in range(1, 17):
        res = oracle.select_eligible(r, nat, alpha, SelectParams(fixed_budget=B))
        assert res["count"] == max(B, 2)
        assert set(nat[0]) <= mask_to_set(res["mask"], 16)


# ------------------------------------------------------------------ anchors over several nodes (Eq. 5)
def test_anchor_set_is_the_union_over_the_listed_nodes_hand_case():
    # 3 nodes, 8 experts, k = 2.  Anchor nodes {0, 2}: A = K_0 u K_2 = {0, 1, 4, 5}.  The residual is what the other
    # experts collect: node 1 alone chooses experts 2 and 3, so R's demand is u_2 = 1/2, u_3 = 1/4 and zero elsewhere
    # (6, 7): q = (2/3, 1/3), exp(H) = 1.89 -> n_er = 2, S = A u {2, 3}.  Experts 4 and 5 collect the largest demand
    # of all (node 2 has alpha 4), yet they must not take residual ranks: they are anchors, outside R.
    r = np.zeros((3, 8), dtype=np.float32)
    nat = np.int32([[0, 1], [2, 3], [4, 5]])
    r[0, 0], r[0, 1] = 0.5, 0.25
    r[1, 2], r[1, 3] = 0.5, 0.25
    r[2, 4], r[2, 5] = 0.5, 0.25
    alpha = np.float32([1.0, 1.0, 4.0])
    res = oracle.select_eligible(r, nat, alpha, SelectParams(), anchor_nodes=np.int32([0, 2]))
    assert res["stats"]["n_anchor"] == 4 and res["stats"]["n_er"] == 2
    assert mask_to_set(res["mask"], 8) == {0, 1, 2, 3, 4, 5}
    assert res["stats"]["residual_mass"] == 0.75
    # the default (root only): A = {0, 1}; R now holds 2, 3, 4, 5 with demand (1/2, 1/4, 2, 1): q = (2/15, 1/15, 8/15,
    # 4/15), exp(H) = 3.14 -> n_er = 4 and the same set results, but through a different count
    root = oracle.select_eligible(r, nat, alpha, SelectParams())
    assert root["stats"]["n_anchor"] == 2 and root["stats"]["n_er"] == 4
    assert mask_to_set(root["mask"], 8) == {0, 1, 2, 3, 4, 5}
    # a fixed budget tells the two apart: B = 4 keeps the four anchors and nothing else, or the root's two anchors
    # plus the two residual experts with the largest demand (4 and 5)
    four = oracle.select_eligible(r, nat, alpha, SelectParams(fixed_budget=4), anchor_nodes=np.int32([0, 2]))
    assert mask_to_set(four["mask"], 8) == {0, 1, 4, 5}
    four_root = oracle.select_eligible(r, nat, alpha, SelectParams(fixed_budget=4))
    assert mask_to_set(four_root["mask"], 8) == {0, 1, 4, 5}
    three = oracle.select_eligible(r, nat, np.float32([1.0, 4.0, 1.0]), SelectParams(fixed_budget=3), anchor_nodes=np.int32([0, 2]))
    assert mask_to_set(three["mask"], 8) == {0, 1, 4, 5}       # the budget never cuts into the anchors: |S| >= |A|
    # a listed node twice, or in another order, changes nothing; an empty list is not the default
    again = oracle.select_eligible(r, nat, alpha, SelectParams(), anchor_nodes=np.int32([2, 0, 2]))
    np.testing.assert_array_equal(again["mask"], res["mask"])


def test_every_listed_anchor_node_keeps_its_natural_top_k():
    rng = np.random.default_rng(515)
    differs = 0
    for trial in range(3000):
        E = int(rng.integers(3, 10))
        k = int(rng.integers(1, min(E, 3) + 1))
        T = int(rng.integers(2, 7))
        z, r = _softmax_rows(rng, T, E, scale=float(rng.uniform(0.2, 4.0)))
        nat = _nat(z, k)
        alpha = rng.uniform(0.05, 1.0, T).astype(np.float32)
        nodes = sorted(rng.choice(T, size=int(rng.integers(1, T + 1)), replace=False).tolist())
        res = oracle.select_eligible(r, nat, alpha, SelectParams(), anchor_nodes=np.int32(nodes))
        S = mask_to_set(res["mask"], E)
        A = set().union(*[set(nat[t]) for t in nodes])
        st = res["stats"]
        assert A <= S and st["n_anchor"] == len(A)                      # Eq. 5 for every listed node
        assert len(S) == res["count"] >= max(len(A), k)
        # the residual ranking sees only experts outside A: every kept non-anchor outranks every dropped one
        u = res["demand"]
        kept = [e for e in S if e not in A]
        dropped = [e for e in range(E) if e not in S]
        assert all((u[a], -a) > (u[b], -b) for a in kept for b in dropped)
        assert len(kept) == (max(st["n_er"], k - len(A)) if st["residual_mass"] > 0.0 else max(0, k - len(A)))
        # residual mass by its definition: positive demand outside A, summed in double (the oracle's tree sum is fp32)
        want_z = sum(max(float(u[e]), 0.0) for e in range(E) if e not in A)
        assert abs(st["residual_mass"] - want_z) <= 1e-6 * max(want_z, 1.0)
        # routes of the listed nodes are their natural ones (their top-k is inside S)
        idx, _ = oracle.route_restricted(z, res["mask"], k)
        for t in nodes:
            assert list(idx[t]) == list(nat[t])
        root_only = oracle.select_eligible(r, nat, alpha, SelectParams())
        differs += not np.array_equal(root_only["mask"], res["mask"])
    assert differs > 100          # the list matters: it is not the default in disguise


# ------------------------------------------------------------------ residency-aware pruning (Eq. 7)
def _prune_brute(S, A, u, votes, resident, k, E):
    C = sorted((e for e in S if e not in resident), key=lambda e: (float(u[e]), e))
    aS = sum(int(votes[e]) for e in range(E) if votes[e] > 0 and e not in S)
    best = 0
    for m in range(0, len(C) + 1):
        if all(sum(int(votes[e]) for e in C[:j]) <= aS and len(S) - j >= k for j in range(1, m + 1)):
            best = m
    return S - set(C[:best]), best, aS


def test_pruning_matches_brute_force_and_special_cases():
    rng = np.random.default_rng(31)
    removed_total = 0
    for trial in range(3000):
        E = int(rng.integers(4, 9))
        k = int(rng.integers(1, 4))
        T = int(rng.integers(2, 7))
        z, r = _softmax_rows(rng, T, E, scale=float(rng.uniform(0.5, 4.0)))
        nat = _nat(z, k)
        alpha = rng.uniform(0.05, 1.0, T).astype(np.float32)
        resident = {e for e in range(E) if rng.random() < 0.4}
        base = oracle.select_eligible(r, nat, alpha)
        S = mask_to_set(base["mask"], E)
        res = oracle.select_eligible(r, nat, alpha, SelectParams(residency=1, max_remove=E),
                                     resident_mask=set_to_mask(resident, E))
        np.testing.assert_array_equal(res["unpruned_mask"], base["mask"])
        votes = np.bincount(nat.ravel(), minlength=E)
        want, m, aS = _prune_brute(S, set(nat[0]), res["demand"], votes, resident, k, E)
        assert mask_to_set(res["mask"], E) == want
        assert res["stats"]["pruned_m"] == m and res["stats"]["displaced_aS"] == aS
        assert res["count"] == len(want) >= k
        removed_total += m
        if aS == 0:
            assert m == 0
        # full residency: nothing to prune
        full = oracle.select_eligible(r, nat, alpha, SelectParams(residency=1), resident_mask=full_mask(E))
        np.testing.assert_array_equal(full["mask"], base["mask"])
        # strict variant: (S intersect resident) union anchors
        strict = oracle.select_eligible(r, nat, alpha, SelectParams(residency=2),
                                        resident_mask=set_to_mask(resident, E))
        assert mask_to_set(strict["mask"], E) == (S & resident) | set(nat[0])
    assert removed_total > 200      # the rule is exercised, not vacuous


def test_pruning_removal_cap():
    rng = np.random.default_rng(4)
    hits = 0
    for trial in range(500):
        E, k, T = 8, 1, 6
        z, r = _softmax_rows(rng, T, E, scale=3.0)
        nat = _nat(z, k)
        alpha = rng.uniform(0.05, 1.0, T).astype(np.float32)
        free = oracle.select_eligible(r, nat, alpha, SelectParams(residency=1, max_remove=E),
                                      resident_mask=set_to_mask([], E))
        capped = oracle.select_eligible(r, nat, alpha, SelectParams(residency=1, max_remove=1),
                                        resident_mask=set_to_mask([], E))
        assert capped["stats"]["pruned_m"] == min(1, free["stats"]["pruned_m"])
        hits += free["stats"]["pruned_m"] > 1
    assert hits > 0


def test_pruned_prefix_is_the_lowest_demand_nonresident_members():
    # hand-built case: S = {0,1,2,3}, anchors {0,1}; non-resident {1,2,3}; demands 1>... ; votes known
    E, k = 6, 2
    r = np.zeros((4, E), dtype=np.float32)
    nat = np.int32([[0, 1], [2, 3], [2, 4], [3, 5]])
    r[0, 0], r[0, 1] = 0.5, 0.25
    r[1, 2], r[1, 3] = 0.5, 0.25
    r[2, 2], r[2, 4] = 0.5, 0.03125
    r[3, 3], r[3, 5] = 0.5, 0.03125
    alpha = np.ones(4, np.float32)
    base = oracle.select_eligible(r, nat, alpha)
    # residual demand: u2 = 1.0, u3 = 0.75, u4 = u5 = 1/32 -> q = (.5517,.4138,.0172,.0172), exp(H) = 2.3 -> 3
    assert base["stats"]["n_er"] == 3
    assert mask_to_set(base["mask"], E) == {0, 1, 2, 3, 4}
    # a(S) = votes of expert 5 = 1.  Non-resident members ordered by demand: 4 (1/32, 1 vote), 1 (.25, 1 vote), ...
    res = oracle.select_eligible(r, nat, alpha, SelectParams(residency=1), resident_mask=set_to_mask({0, 2, 3}, E))
    assert mask_to_set(res["mask"], E) == {0, 1, 2, 3}      # expert 4 removed (budget 1), anchor 1 kept (budget spent)
    # all non-resident, budget still 1: only the lowest-demand member goes, even though it is not an anchor
    res = oracle.select_eligible(r, nat, alpha, SelectParams(residency=1), resident_mask=set_to_mask([], E))
    assert mask_to_set(res["mask"], E) == {0, 1, 2, 3}
    # anchors are not protected by the paper's rule: make the anchor the lowest-demand non-resident member
    r2 = r.copy()
    r2[0, 1] = 2.0 ** -8
    res = oracle.select_eligible(r2, nat, alpha, SelectParams(residency=1), resident_mask=set_to_mask({0, 2, 3, 4}, E))
    assert mask_to_set(res["mask"], E) == {0, 2, 3, 4}
    # the strict variant protects them
    res = oracle.select_eligible(r2, nat, alpha, SelectParams(residency=2), resident_mask=set_to_mask({0, 2, 3, 4}, E))
    assert mask_to_set(res["mask"], E) == {0, 1, 2, 3, 4}


# ------------------------------------------------------------------ routing weights
def test_routing_weight_modes():
    rng = np.random.default_rng(8)
    z, r = _softmax_rows(rng, 4, 10)
    S = {0, 2, 3, 7, 9}
    m = set_to_mask(S, 10)
    zd = z.astype(np.float64)
    p_all = np.exp(zd - zd.max(1, keepdims=True))
    p_all /= p_all.sum(1, keepdims=True)
    for mode in (0, 1, 2):
        idx, w = oracle.route_restricted(z, m, 3, weighting=mode, routed_scale=2.5)
        for t in range(4):
            sel = topk_brute(z[t], 3, S)
            assert list(idx[t]) == sel
            if mode == 0:
                want = p_all[t, sel] / p_all[t, sel].sum()
            elif mode == 1:
                want = p_all[t, sel]
            else:
                want = p_all[t, sel] / p_all[t, sorted(S)].sum()
            np.testing.assert_allclose(w[t], 2.5 * want, rtol=1e-12)


def test_fewer_eligible_than_k_pads_with_minus_one():
    z = np.float32([[0.1, 0.9, 0.5, 0.3]])
    idx, w = oracle.route_restricted(z, set_to_mask({2, 3}, 4), 3)
    assert list(idx[0]) == [2, 3, -1] and w[0, 2] == 0.0 and abs(w[0].sum() - 1.0) < 1e-12
