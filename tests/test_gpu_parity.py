"""GPU parity: every stage of the CUDA library, called through the C ABI, against the CPU oracle
on the same seeded inputs.  Sets, counts, indices, logits, probabilities and demand are compared
bit for bit; routing weights within 1e-5 relative; FFN outputs within 2e-2 x RMS(oracle output)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_02989_b200 import acm, workloads as wl
from tests.helpers import LruModel as _LruModel, full_mask, mask_to_set, set_to_mask

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
FFN_TOL = 2e-2


def _u32(t):
    return t.cpu().numpy().view(np.uint32)


def _take(t, rows):
    return t[torch.as_tensor(np.asarray(rows), device=t.device, dtype=torch.long)]


def _ctx(cfg, **kw):
    return acm.Context.for_config(cfg, n_layers=kw.pop("n_layers", 1), **kw)


def _block(cfg, layer=0, experts=True):
    w = wl.layer_weights(cfg, layer, DEV, experts=experts)
    x = wl.hidden_states(cfg, layer, DEV)
    depth, p = wl.tree_depths(cfg), wl.commitment_table(cfg)
    alpha = acm.node_weights(depth, p)
    np.testing.assert_array_equal(alpha.numpy(), oracle.node_weights(depth.numpy(), p.numpy()))
    return w, x, alpha


def _set_weights(ctx, w, layer=0):
    ctx.set_layer_weights(layer, w["w_router"], w["router_bias"], w["gate_up"], w["down"],
                          w["shared_gate_up"], w["shared_down"])


def _ffn_check(out, ref, what=""):
    out = out.double().cpu().numpy()
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = float(np.abs(out - ref).max())
    assert np.isfinite(out).all(), what
    assert err <= FFN_TOL * rms, f"{what}: max|d|={err:.3e} > {FFN_TOL} * rms={rms:.3e}"
    return err / rms


ROUTER_SHAPES = [
    # (dtype, T, H, E, k, bias)
    ("f32", 8, 256, 16, 2, False),
    ("f32", 5, 96, 13, 3, True),
    ("bf16", 64, 2048, 128, 8, True),
    ("bf16", 37, 1024, 60, 6, False),
    ("bf16", 1, 256, 8, 1, False),
    ("bf16", 64, 4096, 128, 8, False),
    ("bf16", 33, 384, 100, 8, True),
]


@pytest.mark.parametrize("dtype,T,H,E,k,bias", ROUTER_SHAPES)
def test_router_bit_exact(dtype, T, H, E, k, bias):
    g = torch.Generator(device=DEV).manual_seed(T * 1000 + E)
    td = torch.float32 if dtype == "f32" else torch.bfloat16
    x = torch.randn(T, H, generator=g, device=DEV).to(td)
    wr = (0.05 * torch.randn(E, H, generator=g, device=DEV)).to(td)
    b = torch.randn(E, generator=g, device=DEV) if bias else None
    ctx = acm.Context(H, E, k, 64, dtype=acm.F32 if dtype == "f32" else acm.BF16)
    ctx.set_layer_weights(0, wr, b, None, None)
    z, r, nat = ctx.router(0, x)
    assert ctx.device_status() == acm.OK
    zo, ro, nato = oracle.router(x, wr, b, k)
    np.testing.assert_array_equal(z.cpu().numpy(), zo)
    np.testing.assert_array_equal(r.cpu().numpy(), ro)
    np.testing.assert_array_equal(nat.cpu().numpy(), nato)
    ctx.close()


def test_router_flags_non_finite_logits():
    x = torch.randn(4, 256, device=DEV).to(torch.bfloat16)
    wr = torch.randn(8, 256, device=DEV).to(torch.bfloat16)
    b = torch.zeros(8, device=DEV)
    b[3] = float("inf")
    ctx = acm.Context(256, 8, 2, 64)
    ctx.set_layer_weights(0, wr, b, None, None)
    ctx.router(0, x)
    assert ctx.device_status() == acm.ERR_NONFINITE
    assert ctx.device_status() == acm.OK     # sticky until read, then cleared
    ctx.close()


def _random_routing_inputs(rng, T, E, k, scale):
    z = (scale * rng.standard_normal((T, E))).astype(np.float32)
    p = np.exp(z.astype(np.float64) - z.max(1, keepdims=True))
    r = (p / p.sum(1, keepdims=True)).astype(np.float32)
    nat = np.array([sorted(range(E), key=lambda e: (-float(row[e]), e))[:k] for row in z], dtype=np.int32)
    return z, r, nat


SELECT_MODES = [
    dict(),
    dict(demand=1),
    dict(demand=2),
    dict(use_anchors=0),
    dict(fixed_budget=20),
    dict(demand=1, use_anchors=0, fixed_budget=12),     # MoE-Spec (with uniform node weights, rep 5)
    dict(demand=2, use_anchors=0, fixed_budget=16),     # Count-B
    dict(ceil_guard=0.0),
    dict(residency=1),
    dict(residency=1, max_remove=2),
    dict(residency=2),
]


@pytest.mark.parametrize("mode_id", range(len(SELECT_MODES)))
def test_select_eligible_bit_exact(mode_id):
    mode = SELECT_MODES[mode_id]
    rng = np.random.default_rng(100 + mode_id)
    cases = [(64, 128, 8), (32, 64, 8), (48, 64, 6), (8, 16, 2), (1, 128, 8), (17, 33, 5), (64, 96, 1), (3, 8, 8)]
    for T, E, k in cases:
        ctx = acm.Context(256, E, k, 64)
        for rep in range(6):
            z, r, nat = _random_routing_inputs(rng, T, E, k, float(rng.choice([0.3, 1.0, 3.0])))
            alpha = rng.uniform(0.05, 1.0, T).astype(np.float32)
            if rep == 5:
                alpha[:] = 1.0
            resident = {e for e in range(E) if rng.random() < 0.4}
            rmask = set_to_mask(resident, E)
            anchors = None if rep % 3 else np.array(sorted(set([0, T // 2, T - 1])), dtype=np.int32)
            po = oracle.SelectParams(**mode)
            pg = acm.SelectParams(**mode)
            want = oracle.select_eligible(r, nat, alpha, po, anchors, rmask if mode.get("residency") else None)
            got = ctx.select_eligible(torch.tensor(r, device=DEV), torch.tensor(nat, device=DEV),
                                      torch.tensor(alpha, device=DEV), pg,
                                      None if anchors is None else torch.tensor(anchors, device=DEV),
                                      torch.tensor(rmask.view(np.int32), device=DEV) if mode.get("residency") else None)
            np.testing.assert_array_equal(_u32(got["mask"]), want["mask"])
            np.testing.assert_array_equal(_u32(got["unpruned_mask"]), want["unpruned_mask"])
            assert int(got["count"]) == want["count"]
            np.testing.assert_array_equal(got["demand"].cpu().numpy(), want["demand"])
            st = acm.stats_dict(got["stats"])
            for key in ("n_anchor", "n_er", "n_eligible", "n_eligible_pruned", "n_natural_union", "displaced_aS",
                        "pruned_m"):
                assert st[key] == want["stats"][key], (key, T, E, k, rep)
        ctx.close()


def test_select_closed_forms_on_gpu():
    # uniform residual demand over m experts -> n_er = m, for every m (Eq. 6 and the text below it)
    E = 128
    ctx = acm.Context(256, E, 1, 64)
    for m in list(range(1, 20)) + [33, 64, 100, 120, 128]:
        u = np.zeros((1, E), dtype=np.float32)
        u[0, :m] = 0.37
        got = ctx.select_eligible(torch.tensor(u, device=DEV), torch.zeros(1, 1, dtype=torch.int32, device=DEV),
                                  torch.ones(1, device=DEV), acm.SelectParams(demand=1, use_anchors=0))
        assert int(got["count"]) == m
        assert mask_to_set(_u32(got["mask"]), E) == set(range(m))
    ctx.close()


@pytest.mark.parametrize("weighting", [0, 1, 2])
def test_route_restricted(weighting):
    rng = np.random.default_rng(weighting)
    for T, E, k in [(64, 128, 8), (48, 64, 6), (8, 16, 2), (1, 8, 1), (19, 70, 7)]:
        ctx = acm.Context(256, E, k, 64, weighting=weighting, routed_scale=1.5)
        for rep in range(5):
            z, _, nat = _random_routing_inputs(rng, T, E, k, 2.0)
            if rep == 0:
                S = set(range(E))
            elif rep == 1:
                S = set(range(max(1, k - 2)))           # fewer eligible experts than k
            else:
                S = {e for e in range(E) if rng.random() < 0.3} | {0}
            mask = set_to_mask(S, E)
            idx, w = ctx.route_restricted(torch.tensor(z, device=DEV), torch.tensor(mask.view(np.int32), device=DEV))
            io, wo = oracle.route_restricted(z, mask, k, weighting, 1.5)
            np.testing.assert_array_equal(idx.cpu().numpy(), io)
            np.testing.assert_allclose(w.cpu().numpy(), wo, rtol=1e-5, atol=1e-7)
            if rep == 0:
                np.testing.assert_array_equal(idx.cpu().numpy(), nat)      # S = [E] is natural routing
        ctx.close()


FFN_SHAPES = [
    # (T, H, I, E, k, n_shared)
    (64, 256, 128, 8, 2, 0),
    (16, 128, 64, 4, 1, 0),
    (37, 512, 192, 12, 4, 0),       # ragged node count
    (48, 256, 320, 16, 6, 2),       # shared experts, intermediate not a power of two
    (1, 128, 64, 4, 2, 0),
    (64, 2048, 768, 128, 8, 0),     # the Qwen3-30B-A3B layer shape
]


@pytest.mark.parametrize("T,H,I,E,k,ns", FFN_SHAPES)
def test_expert_ffn_against_oracle(T, H, I, E, k, ns):
    cfg = wl.scaled(wl.CONFIGS[3], hidden=H, inter=I, n_experts=E, top_k=k, n_shared=ns, n_nodes=T, zipf_bias=False)
    w = wl.layer_weights(cfg, 7, DEV)
    # larger weights than the recipe's so that outputs are O(1) and errors are visible
    x = wl.hidden_states(cfg, 7, DEV)
    rng = np.random.default_rng(T + E)
    idx = np.array([rng.permutation(E)[:k] for _ in range(T)], dtype=np.int32)
    if T > 2:
        idx[1, -1] = -1                                # an empty slot
    wt = rng.uniform(0.05, 1.0, (T, k)).astype(np.float32)
    ctx = _ctx(cfg)
    _set_weights(ctx, w)
    out = ctx.expert_ffn(0, x, torch.tensor(idx, device=DEV), torch.tensor(wt, device=DEV))
    assert ctx.device_status() == acm.OK
    rows = np.arange(T)
    ref = oracle.expert_ffn(_take(x, rows), idx[rows], wt[rows].astype(np.float64), w["gate_up"], w["down"],
                            w["shared_gate_up"], w["shared_down"])
    _ffn_check(_take(out, rows), ref, f"ffn {T}x{H}x{I}")
    # twice in a row on the same context: workspace flags and counters are re-armed correctly
    out2 = ctx.expert_ffn(0, x, torch.tensor(idx, device=DEV), torch.tensor(wt, device=DEV))
    _ffn_check(_take(out2, rows), ref, "second call")
    ctx.close()


def test_expert_ffn_fp32_toy():
    cfg = wl.CONFIGS[1]
    w = wl.layer_weights(cfg, 0, DEV)
    x = wl.hidden_states(cfg, 0, DEV)
    rng = np.random.default_rng(0)
    idx = np.array([rng.permutation(cfg.n_experts)[:2] for _ in range(cfg.n_nodes)], dtype=np.int32)
    wt = rng.uniform(0.1, 1.0, idx.shape).astype(np.float32)
    ctx = _ctx(cfg)
    _set_weights(ctx, w)
    out = ctx.expert_ffn(0, x, torch.tensor(idx, device=DEV), torch.tensor(wt, device=DEV))
    ref = oracle.expert_ffn(x, idx, wt.astype(np.float64), w["gate_up"], w["down"])
    assert _ffn_check(out, ref, "fp32 toy") < 1e-4
    ctx.close()


def _verify_layer(cfg, layer, ctx, slot, params_kw=None, rows=None, natural=False):
    w, x, alpha = _block(cfg, layer)
    _set_weights(ctx, w, slot)
    E = cfg.n_experts
    pk = params_kw or {}
    if natural:
        mo = torch.tensor(full_mask(E).view(np.int32), device=DEV)
        out, idx, wt, mask, stats = ctx.moe_verify(slot, x, None, None, mask_override=mo, want=True)
        ref = oracle.moe_verify(x, w["w_router"], w["router_bias"], w["gate_up"], w["down"], alpha.numpy(),
                                cfg.top_k, weighting=cfg.weighting, shared_gate_up=w["shared_gate_up"],
                                shared_down=w["shared_down"], mask_override=full_mask(E), with_ffn=False)
    else:
        out, idx, wt, mask, stats = ctx.moe_verify(slot, x, alpha.to(DEV), acm.SelectParams(**pk), want=True)
        ref = oracle.moe_verify(x, w["w_router"], w["router_bias"], w["gate_up"], w["down"], alpha.numpy(),
                                cfg.top_k, oracle.SelectParams(**pk), weighting=cfg.weighting,
                                shared_gate_up=w["shared_gate_up"], shared_down=w["shared_down"], with_ffn=False)
    assert ctx.device_status() == acm.OK
    np.testing.assert_array_equal(_u32(mask), ref["mask"])
    np.testing.assert_array_equal(idx.cpu().numpy(), ref["idx"])
    np.testing.assert_allclose(wt.cpu().numpy(), ref["w"], rtol=1e-5, atol=1e-7)
    st = acm.stats_dict(stats)
    if not natural:
        assert st["n_eligible_pruned"] == ref["count"]
        for key in ("n_anchor", "n_er", "n_eligible", "n_natural_union", "displaced_aS"):
            assert st[key] == ref["stats"][key]
    assert st["n_activated"] == len(set(ref["idx"].ravel()) - {-1})
    if cfg.dtype == "bf16":
        # what the FFN launch streamed: with an early start every eligible expert -- the anchors it started on (ranked
        # by the router kernel's root CTAs from their own copy of the root's logits) must all be among them -- else
        # the activated ones
        assert st["n_streamed"] == (st["n_activated"] if natural else st["n_eligible_pruned"])
    rows = np.arange(cfg.n_nodes) if rows is None else np.asarray(rows)
    ffn = oracle.expert_ffn(_take(x, rows), ref["idx"][rows], ref["w"][rows], w["gate_up"], w["down"],
                            w["shared_gate_up"], w["shared_down"])
    rel = _ffn_check(_take(out, rows), ffn, f"C{cfg.index} layer {layer}")
    return st, rel


def test_config1_toy_fp32_end_to_end():
    cfg = wl.CONFIGS[1]
    ctx = _ctx(cfg)
    st, rel = _verify_layer(cfg, 0, ctx, 0)
    assert rel < 1e-4 and st["n_anchor"] == 2
    _verify_layer(cfg, 0, ctx, 0, natural=True)
    ctx.close()


@pytest.mark.parametrize("c", [2, 3, 4])
def test_full_size_configs_end_to_end(c):
    """Full layer shapes of the OLMoE-, Qwen3-30B-A3B- and DeepSeek-V2-Lite-shaped configurations:
    sets, routes and weights on every node; FFN outputs on every node (all accumulator columns)."""
    cfg = wl.CONFIGS[c]
    ctx = _ctx(cfg, n_layers=2)
    sizes = []
    for layer in (0, cfg.n_layers - 1):
        st, _ = _verify_layer(cfg, layer, ctx, layer % 2)
        sizes.append(st["n_eligible_pruned"])
    _verify_layer(cfg, 1, ctx, 1, natural=True)
    if c == 3:
        assert all(10 <= s <= 45 for s in sizes), sizes     # skewed routing: the set is far below E
    ctx.close()


def test_selection_and_routing_on_every_layer_of_the_qwen3_30b_stack():
    cfg = wl.CONFIGS[3]
    ctx = _ctx(cfg)
    depth, p = wl.tree_depths(cfg), wl.commitment_table(cfg)
    alpha = acm.node_weights(depth, p)
    alpha_dev = alpha.to(DEV)
    for layer in range(cfg.n_layers):
        w = wl.layer_weights(cfg, layer, DEV, experts=False)
        x = wl.hidden_states(cfg, layer, DEV)
        ctx.set_layer_weights(0, w["w_router"], w["router_bias"], None, None)
        z, r, nat = ctx.router(0, x)
        sel = ctx.select_eligible(r, nat, alpha_dev)
        idx, wt = ctx.route_restricted(z, sel["mask"])
        ref = oracle.moe_verify(x, w["w_router"], w["router_bias"], None, None, alpha.numpy(), cfg.top_k,
                                weighting=cfg.weighting, with_ffn=False)
        np.testing.assert_array_equal(z.cpu().numpy(), ref["logits"])
        np.testing.assert_array_equal(_u32(sel["mask"]), ref["mask"])
        np.testing.assert_array_equal(idx.cpu().numpy(), ref["idx"])
    ctx.close()


def test_invalid_arguments_are_rejected_on_the_host():
    cfg = wl.scaled(wl.CONFIGS[3], hidden=256, inter=64, n_experts=8, top_k=2, n_nodes=8, zipf_bias=False)
    w, x, alpha = _block(cfg)
    ctx = _ctx(cfg)
    out = torch.full((8, 256), 7.0, device=DEV)
    with pytest.raises(acm.AcmError) as e:          # weights not registered yet
        ctx.moe_verify(0, x, alpha.to(DEV), out=out)
    assert e.value.code == acm.ERR_INVALID
    _set_weights(ctx, w)
    for bad in (lambda: ctx.moe_verify(3, x, alpha.to(DEV), out=out),                    # layer out of range
                lambda: ctx.moe_verify(0, x[:0], alpha.to(DEV), out=out),                # T = 0
                lambda: ctx.moe_verify(0, x, None, out=out),                             # alpha missing
                lambda: ctx.moe_verify(0, x, alpha.to(DEV), acm.SelectParams(demand=5), out=out),
                lambda: ctx.moe_verify(0, x, alpha.to(DEV), acm.SelectParams(residency=1), out=out),
                lambda: ctx.moe_verify(0, x.view(-1)[1:1 + 7 * 256].view(7, 256), alpha.to(DEV), out=out)):  # misaligned x
        with pytest.raises(acm.AcmError) as e:
            bad()
        assert e.value.code == acm.ERR_INVALID
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())                  # outputs untouched by rejected calls
    ctx.close()


def test_deterministic_selection_and_routing_across_runs():
    cfg = wl.CONFIGS[3]
    w, x, alpha = _block(cfg, 5)
    ctx = _ctx(cfg)
    _set_weights(ctx, w)
    a = ctx.moe_verify(0, x, alpha.to(DEV), want=True)
    b = ctx.moe_verify(0, x, alpha.to(DEV), want=True)
    torch.cuda.synchronize()
    assert torch.equal(a[1], b[1]) and torch.equal(a[3], b[3]) and torch.equal(a[2], b[2])
    assert float((a[0] - b[0]).abs().max()) <= 1e-3 * float(a[0].abs().max())
    ctx.close()


@pytest.mark.parametrize("mode,full_shape", [(1, False), (2, False), (1, True), (2, True)])
def test_offload_variant_residency_and_on_demand_loads(mode, full_shape):
    """Config 5's mechanism, on a reduced layer and on the Qwen3-235B-A22B-shaped layer itself (hidden 4096,
    intermediate 1536, 128 experts, 64 nodes: 37.7 MB per expert copy, staging slots and the second work list at
    full extent): a seeded 40 % of the experts is GPU-resident, eligibility is conditioned on residency (Eq. 7, or the
    strict resident-plus-anchors variant), and activated non-resident experts are copied from pinned host memory.
    The device copies of non-resident experts are poisoned with NaN: a correct result proves they were never read.
    Sets and routes bit for bit, every output row in tolerance, host-to-device bytes exact."""
    cfg = wl.CONFIGS[5] if full_shape else \
        wl.scaled(wl.CONFIGS[5], hidden=512, inter=256, n_experts=32, top_k=4, n_nodes=32, max_depth=5, n_layers=1)
    w, x, alpha = _block(cfg, 2)
    E = cfg.n_experts
    rmask = wl.resident_mask(cfg, 2)
    resident = mask_to_set(rmask.numpy().view(np.uint32), E)
    assert len(resident) == round(0.4 * E)
    host_gu = w["gate_up"].cpu().pin_memory()
    host_dn = w["down"].cpu().pin_memory()
    dev_gu, dev_dn = w["gate_up"].clone(), w["down"].clone()
    for e in range(E):
        if e not in resident:
            dev_gu[e] = float("nan")
            dev_dn[e] = float("nan")
    ctx = _ctx(cfg)
    ctx.set_layer_weights(0, w["w_router"], w["router_bias"], dev_gu, dev_dn)
    ctx.set_resident(0, rmask, host_gu, host_dn)
    for rep in range(2):          # twice: staging slots and events are reused correctly
        ctx.h2d_bytes(reset=True)
        out, idx, wt, mask, stats = ctx.moe_verify(0, x, alpha.to(DEV), acm.SelectParams(residency=mode), want=True)
        assert ctx.device_status() == acm.OK
        ref = oracle.moe_verify(x, w["w_router"], w["router_bias"], w["gate_up"], w["down"], alpha.numpy(), cfg.top_k,
                                oracle.SelectParams(residency=mode), weighting=cfg.weighting,
                                resident_mask=rmask.numpy().view(np.uint32))
        np.testing.assert_array_equal(_u32(mask), ref["mask"])
        np.testing.assert_array_equal(idx.cpu().numpy(), ref["idx"])
        _ffn_check(out, ref["out"], f"offload mode {mode}")
        st = acm.stats_dict(stats)
        activated = set(ref["idx"].ravel()) - {-1}
        staged = activated - resident
        assert st["n_activated"] == len(activated) and st["n_staged"] == len(staged)
        assert st["pruned_m"] == ref["stats"]["pruned_m"]
        assert ctx.h2d_bytes() == len(staged) * cfg.expert_bytes
        if mode == 2:
            assert staged <= set(ref["nat_idx"][0])       # only the root's anchors can be non-resident
    # natural routing on the same offloaded layer: every activated non-resident expert is loaded
    ctx.h2d_bytes(reset=True)
    full = torch.tensor(full_mask(E).view(np.int32), device=DEV)
    out, idx, wt, mask, stats = ctx.moe_verify(0, x, None, None, mask_override=full, want=True)
    ref = oracle.moe_verify(x, w["w_router"], w["router_bias"], w["gate_up"], w["down"], alpha.numpy(), cfg.top_k,
                            weighting=cfg.weighting, mask_override=full_mask(E))
    _ffn_check(out, ref["out"], "offload natural")
    nat_staged = (set(ref["idx"].ravel()) - {-1}) - resident
    assert ctx.h2d_bytes() == len(nat_staged) * cfg.expert_bytes
    assert acm.stats_dict(stats)["n_staged"] == len(nat_staged)
    ctx.close()


def test_config5_shape_one_layer():
    """The Qwen3-235B-A22B-shaped layer at full size (4.8 GB of weights), restricted routing, all resident, every row."""
    cfg = wl.CONFIGS[5]
    ctx = _ctx(cfg)
    st, _ = _verify_layer(cfg, 0, ctx, 0)
    assert st["n_activated"] > cfg.top_k
    ctx.close()


def test_eligible_but_unchosen_experts_contribute_nothing():
    """The FFN kernel starts on the ELIGIBLE set before the routes exist.  With few nodes and a large fixed
    budget most eligible experts are chosen by no node: they must add nothing to the output, and the
    activated count must still be that of the routes."""
    cfg = wl.scaled(wl.CONFIGS[3], n_nodes=5)
    ctx = _ctx(cfg)
    st, _ = _verify_layer(cfg, 0, ctx, 0, params_kw={"fixed_budget": 96})
    assert st["n_eligible_pruned"] == 96 and st["n_activated"] <= 5 * cfg.top_k < st["n_eligible_pruned"]
    ctx.close()


def test_host_buffer_call_matches_the_device_call():
    """acm_moe_verify_host: pinned host x / alpha in, pinned host out back, through the two alternating
    buffer sets (five calls, so both sets are reused), against the device-pointer call on the same blocks."""
    cfg = wl.CONFIGS[3]
    ctx = _ctx(cfg, n_layers=2)
    depth, p = wl.tree_depths(cfg), wl.commitment_table(cfg)
    alpha = acm.node_weights(depth, p)
    alpha_pin = alpha.pin_memory()
    blocks = []
    for layer in range(2):
        w = wl.layer_weights(cfg, layer, DEV)
        _set_weights(ctx, w, layer)
        blocks.append(w)
    calls = [0, 1, 1, 0, 1]
    xs = [wl.hidden_states(cfg, 10 + i, DEV) for i in range(len(calls))]
    xs_pin = [x.cpu().pin_memory() for x in xs]
    outs_pin = [torch.full((cfg.n_nodes, cfg.hidden), float("nan")).pin_memory() for _ in calls]
    stats_pin = [torch.zeros(12, dtype=torch.int32).pin_memory() for _ in calls]
    for i, layer in enumerate(calls):
        ctx.moe_verify_host(layer, xs_pin[i], alpha_pin, outs_pin[i], stats_host=stats_pin[i])
    ctx.host_synchronize()
    assert ctx.device_status() == acm.OK
    for i, layer in enumerate(calls):
        out, idx, wt, mask, stats = ctx.moe_verify(layer, xs[i], alpha.to(DEV), acm.SelectParams(), want=True)
        ref = out.double().cpu().numpy()
        _ffn_check(outs_pin[i].to(DEV), ref, f"host call {i}")
        assert acm.stats_dict(stats_pin[i]) == acm.stats_dict(stats)
    ctx.close()


@pytest.mark.parametrize("level", [acm.OVERLAP_NONE, acm.OVERLAP_DEPENDENT, acm.OVERLAP_ELIGIBLE, acm.OVERLAP_ANCHORS])
def test_overlap_levels_agree_with_the_oracle(level):
    """The fused call's kernels overlap to a degree the caller chooses (plain stream order with a cooperative FFN
    launch; dependent launches; early start on the eligible set; early start on the anchors): every level must give
    the oracle's sets, routes and outputs, on every row, and switching levels on a live context must too."""
    cfg = wl.CONFIGS[3]
    ctx = _ctx(cfg, n_layers=2)
    ctx.set_overlap(level)
    for layer in (0, 1):
        _verify_layer(cfg, layer, ctx, layer)
    ctx.set_overlap((level + 2) % 4)
    _verify_layer(cfg, 1, ctx, 1)
    with pytest.raises(acm.AcmError):
        ctx.set_overlap(7)
    ctx.close()


def test_back_to_back_layers_without_host_synchronisation():
    """Sixteen layer calls enqueued without a host synchronisation in between (dependent launches overlap each
    kernel's set-up with the kernel before it; the per-call tags of the published eligible set must never be
    mistaken for the previous call's), with a changing number of nodes; every call's routes against the oracle."""
    cfg = wl.CONFIGS[3]
    ctx = _ctx(cfg, n_layers=4)
    depth, p = wl.tree_depths(cfg), wl.commitment_table(cfg)
    alpha_full = acm.node_weights(depth, p)
    ws, refs, outs = [], [], []
    for layer in range(4):
        w = wl.layer_weights(cfg, layer, DEV)
        _set_weights(ctx, w, layer)
        ws.append(w)
    calls = [(i % 4, [64, 33, 17, 64, 5, 48][i % 6]) for i in range(16)]
    xs = [wl.hidden_states(cfg, 20 + i, DEV)[:T].contiguous() for i, (_, T) in enumerate(calls)]
    res = []
    for (layer, T), x in zip(calls, xs):
        res.append(ctx.moe_verify(layer, x, alpha_full[:T].to(DEV), acm.SelectParams(), want=True))
    torch.cuda.synchronize()
    assert ctx.device_status() == acm.OK
    for (layer, T), x, (out, idx, wt, mask, stats) in zip(calls, xs, res):
        w = ws[layer]
        ref = oracle.moe_verify(x, w["w_router"], w["router_bias"], w["gate_up"], w["down"], alpha_full[:T].numpy(),
                                cfg.top_k, oracle.SelectParams(), weighting=cfg.weighting, with_ffn=False)
        np.testing.assert_array_equal(_u32(mask), ref["mask"])
        np.testing.assert_array_equal(idx.cpu().numpy(), ref["idx"])
        assert acm.stats_dict(stats)["n_activated"] == len(set(ref["idx"].ravel()) - {-1})
        ffn = oracle.expert_ffn(x, ref["idx"], ref["w"], w["gate_up"], w["down"])
        _ffn_check(out, ffn, f"call layer {layer} T {T}")
    ctx.close()


@pytest.mark.parametrize("mode,mx", [(1, False), (0, False), (1, True)])
def test_lru_expert_pool_over_a_sequence_of_blocks(mode, mx):
    """Section 3.4's X-slot pool on a reduced config-5 layer: the expert tensors exist on the device only as pool
    slots; eight blocks in a row, each against the oracle run with the resident set an LRU model predicts, plus the
    model's hit / miss counts, loaded bytes and final slot contents."""
    cfg = wl.scaled(wl.CONFIGS[5], hidden=512, inter=256, n_experts=64, top_k=4, n_nodes=24, max_depth=5, n_layers=1,
                    zipf_bias=True)            # skewed expert popularity: the activated set stays below the pool size
    w, _, alpha = _block(cfg, 3)
    E, X = cfg.n_experts, 24
    initial = list(range(0, 24, 2))                 # 12 of the 20 slots start occupied
    ctx = _ctx(cfg)
    expert_bytes = cfg.expert_bytes
    if mx:
        # the same layer with its experts in MXFP4: pool and host tensors hold tile records, the oracle sees the
        # dequantised weights
        m = _mx_layer(cfg, 3)
        w["gate_up"], w["down"] = m["gate_up_deq"], m["down_deq"]
        host_gu, host_dn = m["gate_up_tiles"].cpu().pin_memory(), m["down_tiles"].cpu().pin_memory()
        pool_gu = torch.full((X,) + tuple(host_gu.shape[1:]), 0xFF, dtype=torch.uint8, device=DEV)
        pool_dn = torch.full((X,) + tuple(host_dn.shape[1:]), 0xFF, dtype=torch.uint8, device=DEV)
        ctx.set_layer_weights_mxfp4(0, w["w_router"], w["router_bias"], None, None)
        expert_bytes = host_gu[0].numel() + host_dn[0].numel()
        assert expert_bytes * 32 == cfg.expert_bytes // 2 * 17        # 4 bits + 1/32 byte per weight
    else:
        host_gu, host_dn = w["gate_up"].cpu().pin_memory(), w["down"].cpu().pin_memory()
        pool_gu = torch.full((X,) + tuple(w["gate_up"].shape[1:]), float("nan"), dtype=w["gate_up"].dtype, device=DEV)
        pool_dn = torch.full((X,) + tuple(w["down"].shape[1:]), float("nan"), dtype=w["down"].dtype, device=DEV)
        ctx.set_layer_weights(0, w["w_router"], w["router_bias"], None, None)
    ctx.set_slot_pool(0, pool_gu, pool_dn, host_gu, host_dn, initial)
    model = _LruModel(X, initial)
    tot_hits = tot_misses = 0
    for blk in range(8):
        x = wl.hidden_states(cfg, 40 + blk, DEV)
        rset = model.resident()
        rmask = np.zeros(2, dtype=np.uint32)
        for e in rset:
            rmask[e >> 5] |= np.uint32(1) << np.uint32(e & 31)
        out, idx, wt, mask, stats = ctx.moe_verify(0, x, alpha.to(DEV), acm.SelectParams(residency=mode), want=True)
        assert ctx.device_status() == acm.OK
        ref = oracle.moe_verify(x, w["w_router"], w["router_bias"], w["gate_up"], w["down"], alpha.numpy(), cfg.top_k,
                                oracle.SelectParams(residency=mode), weighting=cfg.weighting, resident_mask=rmask)
        np.testing.assert_array_equal(_u32(mask), ref["mask"])
        np.testing.assert_array_equal(idx.cpu().numpy(), ref["idx"])
        _ffn_check(out, ref["out"], f"pool block {blk}")
        activated = {int(e) for e in set(ref["idx"].ravel()) - {-1}}
        hits, misses = model.block(activated)
        tot_hits += hits
        tot_misses += misses
        st = acm.stats_dict(stats)
        assert st["n_activated"] == len(activated) and st["n_staged"] == misses
    ps = ctx.pool_stats(0)
    assert (ps["hits"], ps["misses"]) == (tot_hits, tot_misses)
    assert ps["h2d_bytes"] == tot_misses * expert_bytes
    assert ps["slot_expert"] == model.slot_expert
    assert tot_misses > 0 and tot_hits > 0
    ctx.close()


def test_expert_pool_smaller_than_the_routed_union_runs_in_waves():
    """Natural routing activates more experts than the pool has slots: the loads and their FFN launches go in
    several waves; the output is still the oracle's and every activated expert outside the pool is loaded once."""
    cfg = wl.scaled(wl.CONFIGS[5], hidden=512, inter=256, n_experts=64, top_k=4, n_nodes=24, max_depth=5, n_layers=1)
    w, _, alpha = _block(cfg, 4)
    E, X = cfg.n_experts, 10
    host_gu, host_dn = w["gate_up"].cpu().pin_memory(), w["down"].cpu().pin_memory()
    pool_gu = torch.full((X,) + tuple(w["gate_up"].shape[1:]), float("nan"), dtype=w["gate_up"].dtype, device=DEV)
    pool_dn = torch.full((X,) + tuple(w["down"].shape[1:]), float("nan"), dtype=w["down"].dtype, device=DEV)
    initial = [1, 5, 9, 13, 17, 21, 25]
    ctx = _ctx(cfg)
    ctx.set_layer_weights(0, w["w_router"], w["router_bias"], None, None)
    ctx.set_slot_pool(0, pool_gu, pool_dn, host_gu, host_dn, initial)
    model = _LruModel(X, initial)
    full = torch.tensor(full_mask(E).view(np.int32), device=DEV)
    tot_hits = tot_misses = 0
    for blk in range(3):
        x = wl.hidden_states(cfg, 60 + blk, DEV)
        out, idx, wt, mask, stats = ctx.moe_verify(0, x, None, None, mask_override=full, want=True)
        assert ctx.device_status() == acm.OK
        ref = oracle.moe_verify(x, w["w_router"], w["router_bias"], w["gate_up"], w["down"], alpha.numpy(), cfg.top_k,
                                weighting=cfg.weighting, mask_override=full_mask(E))
        np.testing.assert_array_equal(idx.cpu().numpy(), ref["idx"])
        _ffn_check(out, ref["out"], f"waves block {blk}")
        activated = {int(e) for e in set(ref["idx"].ravel()) - {-1}}
        assert len(activated) > X
        hits, misses = model.block(activated)
        tot_hits += hits
        tot_misses += misses
    ps = ctx.pool_stats(0)
    assert (ps["hits"], ps["misses"]) == (tot_hits, tot_misses)
    assert ps["slot_expert"] == model.slot_expert
    ctx.close()


def _batch_reference(cfg, w, x, offsets, depths, params_kw):
    """The oracle knows single blocks only: a batch is, by definition, every block verified by itself."""
    p = wl.commitment_table(cfg)
    alphas, refs = [], []
    for b in range(len(offsets) - 1):
        lo, hi = offsets[b], offsets[b + 1]
        a = oracle.node_weights(depths[lo:hi].numpy(), p.numpy())
        refs.append(oracle.moe_verify(x[lo:hi], w["w_router"], w["router_bias"], w["gate_up"], w["down"], a,
                                      cfg.top_k, oracle.SelectParams(**params_kw), weighting=cfg.weighting,
                                      shared_gate_up=w["shared_gate_up"], shared_down=w["shared_down"],
                                      with_ffn=False))
        alphas.append(a)
    return np.concatenate(alphas), refs


@pytest.mark.parametrize("c,n_blocks,params_kw", [(3, 4, {}), (3, 7, {}), (3, 2, {"fixed_budget": 12}), (4, 3, {}),
                                                  (3, 12, {}), (2, 32, {}), (3, 1, {}), (3, 64, {})])
def test_multi_block_batch_equals_every_block_verified_alone(c, n_blocks, params_kw):
    """Several verification blocks in one call: each block's eligible set, routes and statistics are those of
    the oracle run on that block alone (ragged block sizes, 1 to 64 blocks, with and without the FFN
    kernel's early start, shared experts), the FFN output rows match the oracle's, and the activated mask is
    the union over the blocks."""
    cfg = wl.CONFIGS[c]
    ctx = _ctx(cfg)
    w = wl.layer_weights(cfg, 0, DEV)
    _set_weights(ctx, w, 0)
    x = wl.hidden_states(cfg, 0, DEV)
    offsets, depths = wl.batch_tree_depths(cfg, n_blocks)
    assert offsets[-1] == cfg.n_nodes and len(set(np.diff(offsets))) <= 2
    alpha_ref, refs = _batch_reference(cfg, w, x, offsets, depths, params_kw)
    p = wl.commitment_table(cfg)
    alpha = torch.cat([acm.node_weights(depths[offsets[b]:offsets[b + 1]], p) for b in range(n_blocks)])
    np.testing.assert_array_equal(alpha.numpy(), alpha_ref)
    for rep in range(2):                  # the second call runs on the workspace the first one left behind
        out, idx, wt, mask, act, stats = ctx.moe_verify_batch(0, x, offsets, alpha.to(DEV),
                                                              acm.SelectParams(**params_kw), want=True)
        assert ctx.device_status() == acm.OK
        union = set()
        for b, ref in enumerate(refs):
            lo, hi = offsets[b], offsets[b + 1]
            np.testing.assert_array_equal(_u32(mask[b]), ref["mask"])
            np.testing.assert_array_equal(idx[lo:hi].cpu().numpy(), ref["idx"])
            np.testing.assert_allclose(wt[lo:hi].cpu().numpy(), ref["w"], rtol=1e-5, atol=1e-7)
            st = acm.stats_dict(stats[b])
            assert st["n_eligible_pruned"] == ref["count"]
            for key in ("n_anchor", "n_er", "n_eligible", "n_natural_union", "displaced_aS"):
                assert st[key] == ref["stats"][key]
            mine = set(ref["idx"].ravel().tolist()) - {-1}
            assert st["n_activated"] == len(mine)
            union |= mine
        assert mask_to_set(_u32(act), cfg.n_experts) == union
        ref_idx = np.concatenate([r["idx"] for r in refs])
        ref_w = np.concatenate([r["w"] for r in refs])
        if rep == 0:
            ffn = oracle.expert_ffn(x, ref_idx, ref_w, w["gate_up"], w["down"], w["shared_gate_up"], w["shared_down"])
        _ffn_check(out, ffn, f"C{c} batch of {n_blocks}")
    ctx.close()


def test_multi_block_batch_rejects_bad_descriptions():
    cfg = wl.scaled(wl.CONFIGS[3], inter=128)
    ctx = _ctx(cfg)
    w = wl.layer_weights(cfg, 0, DEV)
    _set_weights(ctx, w, 0)
    x = wl.hidden_states(cfg, 0, DEV)
    alpha = torch.ones(cfg.n_nodes, device=DEV)
    for offs in ([0, 0, 64], [1, 64], [0, 40, 30, 64], [0, 65], [0]):
        with pytest.raises(acm.AcmError):
            ctx.moe_verify_batch(0, x[: max(1, min(offs[-1], 64))], offs, alpha)
    ctx.close()


def test_stage_times_come_from_device_stamps():
    cfg = wl.scaled(wl.CONFIGS[3], inter=256)
    ctx = _ctx(cfg, n_layers=2)
    with pytest.raises(acm.AcmError):
        ctx.stage_times()                       # stamps are off
    ctx.stage_timing(True)
    with pytest.raises(acm.AcmError):
        ctx.stage_times()                       # no call yet
    outs = []
    for layer in (0, 1):
        w, x, alpha = _block(cfg, layer)
        _set_weights(ctx, w, layer)
        outs.append((x, alpha.to(DEV)))
    for _ in range(3):
        for layer in (0, 1):
            out = ctx.moe_verify(layer, outs[layer][0], outs[layer][1])
    st = ctx.stage_times()
    assert ctx.device_status() == acm.OK
    assert all(v > 0.0 for v in st.values()), st
    assert st["whole"] >= st["ffn"] and st["whole"] >= st["router"] + st["select"]
    assert st["whole"] < 1000.0, st
    ref = ctx.moe_verify(1, outs[1][0], outs[1][1])
    ctx.stage_timing(False)
    again = ctx.moe_verify(1, outs[1][0], outs[1][1])
    np.testing.assert_allclose(again.cpu().numpy(), ref.cpu().numpy(), rtol=1e-3, atol=1e-4)    # same result with stamps on and off
    with pytest.raises(acm.AcmError):
        ctx.stage_times()
    ctx.close()


@pytest.mark.parametrize("T", [1, 2, 5, 17, 33, 63])
def test_fused_call_on_ragged_block_sizes(T):
    """Blocks of 1 to 63 nodes (padded accumulator columns, partial node tiles in the router kernel, trees
    shallower than the commitment table) through the fused call, every output row against the oracle."""
    cfg = wl.scaled(wl.CONFIGS[3], n_nodes=T, inter=256, n_layers=1)
    ctx = _ctx(cfg)
    st, rel = _verify_layer(cfg, 0, ctx, 0)
    assert st["n_activated"] >= min(cfg.top_k, cfg.n_experts)
    _verify_layer(cfg, 0, ctx, 0, natural=True)
    ctx.close()


def test_fused_call_on_every_block_size():
    """Every block size from 1 to 64 on one small layer shape: the selection kernel runs as a cluster of one, two or
    four CTAs with one warp per row, the last of them partly or wholly without rows; sets, routes and every output
    row against the oracle."""
    for T in range(1, 65):
        cfg = wl.scaled(wl.CONFIGS[3], n_nodes=T, hidden=256, inter=128, n_layers=1)
        ctx = _ctx(cfg)
        _verify_layer(cfg, 0, ctx, 0)
        ctx.close()


def _mx_layer(cfg, layer=0):
    """An MXFP4 layer: the config's bf16 draw quantised; returns the weights dict with the tiled device tensors and
    the dequantised bf16 tensors (what the layer means)."""
    w = wl.layer_weights_mxfp4(cfg, layer, DEV)
    w["gate_up_tiles"] = acm.pack_mxfp4_gate_up(w["gate_up_codes"], w["gate_up_scales"]).to(DEV)
    w["down_tiles"] = acm.pack_mxfp4_down(w["down_codes"], w["down_scales"]).to(DEV)
    gu = torch.tensor(oracle.dequantize_mxfp4(w["gate_up_codes"], w["gate_up_scales"]))
    dn = torch.tensor(oracle.dequantize_mxfp4(w["down_codes"], w["down_scales"]))
    assert torch.equal(gu.to(torch.bfloat16).double(), gu) and torch.equal(dn.to(torch.bfloat16).double(), dn)
    w["gate_up_deq"], w["down_deq"] = gu.to(torch.bfloat16).to(DEV), dn.to(torch.bfloat16).to(DEV)
    return w


@pytest.mark.parametrize("shape", [dict(inter=256, n_experts=32), dict(), dict(hidden=4096, inter=1536, n_nodes=33)])
def test_mxfp4_layer_equals_the_bf16_layer_with_the_dequantised_weights(shape):
    """Expert weights in MXFP4: sets and routes as always (the router is bf16); the FFN output against the oracle
    run on the dequantised weights, and against the library's own bf16 kernel on them, which does the same
    arithmetic in the same order."""
    cfg = wl.scaled(wl.CONFIGS[3], n_layers=1, **shape)
    ctx = _ctx(cfg, n_layers=2)
    w = _mx_layer(cfg)
    x = wl.hidden_states(cfg, 0, DEV)
    alpha = acm.node_weights(wl.tree_depths(cfg), wl.commitment_table(cfg))
    ctx.set_layer_weights_mxfp4(0, w["w_router"], w["router_bias"], w["gate_up_tiles"], w["down_tiles"])
    ctx.set_layer_weights(1, w["w_router"], w["router_bias"], w["gate_up_deq"], w["down_deq"])
    for natural in (False, True):
        kw = dict(mask_override=torch.tensor(full_mask(cfg.n_experts).view(np.int32), device=DEV)) if natural else {}
        a = None if natural else alpha.to(DEV)
        out, idx, wt, mask, stats = ctx.moe_verify(0, x, a, None if natural else acm.SelectParams(), want=True, **kw)
        ref_out, ref_idx, ref_wt, ref_mask, _ = ctx.moe_verify(1, x, a, None if natural else acm.SelectParams(), want=True, **kw)
        assert ctx.device_status() == acm.OK
        np.testing.assert_array_equal(idx.cpu().numpy(), ref_idx.cpu().numpy())
        np.testing.assert_array_equal(_u32(mask), _u32(ref_mask))
        ffn = oracle.expert_ffn(x, idx.cpu().numpy(), wt.cpu().numpy(), w["gate_up_deq"], w["down_deq"])
        _ffn_check(out, ffn, "MXFP4 layer")
        # same tiles, same MMAs, same order of additions inside a tile; split-K partial sums meet in L2 in any order
        rms = float(ref_out.double().pow(2).mean().sqrt())
        assert float((out - ref_out).abs().max()) <= 1e-3 * rms
    ctx.close()


def test_mxfp4_scale_bytes_up_to_the_limit_and_beyond():
    """E8M0 scale bytes up to 128 (block scale 2) are exact; a tensor with a larger one is refused when it is
    registered, on the device path and on the pool's host path, instead of computing something else."""
    cfg = wl.scaled(wl.CONFIGS[3], n_layers=1, inter=256, n_experts=32)
    w = wl.layer_weights_mxfp4(cfg, 0, DEV)
    rng = np.random.default_rng(3)
    x = wl.hidden_states(cfg, 0, DEV)
    alpha = acm.node_weights(wl.tree_depths(cfg), wl.commitment_table(cfg))
    ctx = _ctx(cfg, n_layers=2)
    for names in (("gate_up_scales",), ("gate_up_scales", "down_scales")):
        for name in names:                                  # a few hundred blocks at the largest supported scales
            sc = w[name].view(-1)
            pick = torch.tensor(rng.choice(sc.numel(), 300, replace=False), device=sc.device)
            sc[pick] = torch.tensor(rng.integers(126, 129, 300), dtype=torch.uint8, device=sc.device)
        w["gate_up_tiles"] = acm.pack_mxfp4_gate_up(w["gate_up_codes"], w["gate_up_scales"]).to(DEV)
        w["down_tiles"] = acm.pack_mxfp4_down(w["down_codes"], w["down_scales"]).to(DEV)
        gu = torch.tensor(oracle.dequantize_mxfp4(w["gate_up_codes"], w["gate_up_scales"])).to(torch.bfloat16)
        dn = torch.tensor(oracle.dequantize_mxfp4(w["down_codes"], w["down_scales"])).to(torch.bfloat16)
        assert float(gu.abs().max()) >= 4.0                  # (the large scales are really in there)
        ctx.set_layer_weights_mxfp4(0, w["w_router"], w["router_bias"], w["gate_up_tiles"], w["down_tiles"])
        ctx.set_layer_weights(1, w["w_router"], w["router_bias"], gu.to(DEV), dn.to(DEV))
        out, idx, wt, mask, stats = ctx.moe_verify(0, x, alpha.to(DEV), want=True)
        ref_out = ctx.moe_verify(1, x, alpha.to(DEV))
        assert ctx.device_status() == acm.OK
        # the expansion is exact: the bf16 kernel on the dequantised weights does the same arithmetic
        rms = float(ref_out.double().pow(2).mean().sqrt())
        assert float((out - ref_out).abs().max()) <= 1e-3 * rms
        if len(names) == 1:
            # against the oracle where the sum is well conditioned (with huge down weights too, terms of +-10^4 cancel
            # and the activations' rounding to bf16, which the tolerance allows for, is amplified)
            # ... and row by row: a few hundred weights are 256 times the others, so a row's size depends on which of
            # them its experts hold; each row within the tolerance of its own (or the layer's) RMS
            ffn = oracle.expert_ffn(x, idx.cpu().numpy(), wt.cpu().numpy(), gu, dn)
            got = out.double().cpu().numpy()
            row_rms = np.maximum(np.sqrt(np.mean(ffn ** 2, axis=1)), float(np.sqrt(np.mean(ffn ** 2))))
            assert (np.abs(got - ffn).max(axis=1) <= FFN_TOL * row_rms).all()
    # one byte beyond the limit
    bad = w["down_scales"].clone()
    bad.view(-1)[12345] = 129
    bad_tiles = acm.pack_mxfp4_down(w["down_codes"], bad).to(DEV)
    with pytest.raises(acm.AcmError) as e:
        ctx.set_layer_weights_mxfp4(0, w["w_router"], w["router_bias"], w["gate_up_tiles"], bad_tiles)
    assert e.value.code == acm.ERR_UNSUPPORTED
    ctx.set_layer_weights_mxfp4(0, w["w_router"], w["router_bias"], None, None)
    X = 8
    pool_gu = torch.zeros((X,) + tuple(w["gate_up_tiles"].shape[1:]), dtype=torch.uint8, device=DEV)
    pool_dn = torch.zeros((X,) + tuple(w["down_tiles"].shape[1:]), dtype=torch.uint8, device=DEV)
    with pytest.raises(acm.AcmError) as e:
        ctx.set_slot_pool(0, pool_gu, pool_dn, w["gate_up_tiles"].cpu().pin_memory(), bad_tiles.cpu().pin_memory(), [0, 1])
    assert e.value.code == acm.ERR_UNSUPPORTED
    ctx.close()


def test_multi_block_batch_on_an_mxfp4_layer():
    """The batch call on an MXFP4 layer: per-block sets and routes as on the bf16 layer with the dequantised
    weights, output rows within tolerance of the oracle."""
    cfg = wl.scaled(wl.CONFIGS[3], n_layers=1, inter=256, n_experts=64)
    ctx = _ctx(cfg, n_layers=2)
    w = _mx_layer(cfg)
    ctx.set_layer_weights_mxfp4(0, w["w_router"], w["router_bias"], w["gate_up_tiles"], w["down_tiles"])
    x = wl.hidden_states(cfg, 0, DEV)
    offsets, depths = wl.batch_tree_depths(cfg, 5)
    p = wl.commitment_table(cfg)
    alpha = torch.cat([acm.node_weights(depths[offsets[b]:offsets[b + 1]], p) for b in range(5)])
    wq = dict(w, gate_up=w["gate_up_deq"], down=w["down_deq"])
    _, refs = _batch_reference(cfg, wq, x, offsets, depths, {})
    out, idx, wt, mask, act, stats = ctx.moe_verify_batch(0, x, offsets, alpha.to(DEV), want=True)
    assert ctx.device_status() == acm.OK
    for b, ref in enumerate(refs):
        np.testing.assert_array_equal(_u32(mask[b]), ref["mask"])
        np.testing.assert_array_equal(idx[offsets[b]:offsets[b + 1]].cpu().numpy(), ref["idx"])
    ref_idx = np.concatenate([r["idx"] for r in refs])
    ref_w = np.concatenate([r["w"] for r in refs])
    ffn = oracle.expert_ffn(x, ref_idx, ref_w, w["gate_up_deq"], w["down_deq"])
    _ffn_check(out, ffn, "MXFP4 batch")
    ctx.close()


@pytest.mark.parametrize("params_kw", [dict(fixed_budget=4), dict(fixed_budget=9), dict(use_anchors=0),
                                       dict(use_anchors=0, fixed_budget=8), dict(demand=2, fixed_budget=30)])
def test_fused_call_when_the_eligible_set_is_little_more_than_the_anchors(params_kw):
    """The FFN kernel starts on the anchors before the eligible set is known: sets that hold nothing but the anchors
    (a budget below k), one expert more, no anchors at all (the kernel then starts on the eligible set), and a large
    fixed budget -- all rows against the oracle, on two layers back to back."""
    cfg = wl.scaled(wl.CONFIGS[3], n_layers=2, inter=256)
    ctx = _ctx(cfg, n_layers=2)
    for layer in (0, 1):
        st, _ = _verify_layer(cfg, layer, ctx, layer, params_kw=params_kw)
        if params_kw.get("fixed_budget") == 4:
            assert st["n_eligible_pruned"] == cfg.top_k == st["n_anchor"]
    ctx.close()


def test_fused_call_on_random_shapes_and_selector_settings():
    """A hundred seeded random layers -- hidden, experts, top-k, intermediate size, shared experts, nodes, weighting rule,
    selector mode, budget, anchors on or off -- twice each through the fused call (the second call runs on what the
    first left behind), everything against the oracle."""
    rng = np.random.default_rng(2026)
    for case in range(100):
        H = int(rng.choice([256, 512, 1024]))
        E = int(rng.integers(8, 129))
        k = int(rng.integers(1, min(8, E) + 1))
        I = int(rng.choice([64, 128, 192, 320]))
        ns = int(rng.choice([0, 0, 1, 2]))
        T = int(rng.integers(1, 65))
        D = int(min(rng.integers(1, 9), max(T - 1, 1)))
        cfg = wl.scaled(wl.CONFIGS[3], hidden=H, n_experts=E, top_k=k, inter=I, n_shared=ns, n_nodes=T, max_depth=D,
                        n_layers=1, weighting=int(rng.integers(0, 3)), zipf_bias=bool(rng.integers(0, 2)))
        kw = {}
        if rng.random() < 0.4:
            kw["fixed_budget"] = int(rng.integers(1, E + 1))
        if rng.random() < 0.25:
            kw["use_anchors"] = 0
        if rng.random() < 0.3:
            kw["demand"] = int(rng.integers(0, 3))
        ctx = _ctx(cfg)
        for rep in range(2):
            _verify_layer(cfg, 0, ctx, 0, params_kw=kw)
        ctx.close()


@pytest.mark.parametrize("sizes", [[33, 1, 16, 14], [17, 17, 17, 13], [16, 16, 16, 16], [1] * 10 + [22], [32, 32], [64]])
def test_batch_call_on_block_sizes_around_the_selection_clusters_steps(sizes):
    """Partitions whose widest block sits on either side of 16 and 32 rows (the selection kernel gives every block a
    cluster of one, two or four CTAs sized by the widest), with single-row blocks beside wide ones: every block
    against the oracle run on it alone, every output row."""
    rng = np.random.default_rng(len(sizes) * 1000 + sizes[0])
    offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(int).tolist()
    T = offsets[-1]
    cfg = wl.scaled(wl.CONFIGS[3], hidden=512, inter=128, n_nodes=T, max_depth=4, n_layers=1)
    w = wl.layer_weights(cfg, 0, DEV)
    x = wl.hidden_states(cfg, 0, DEV)
    depths = torch.cat([torch.sort(torch.cat([torch.zeros(1, dtype=torch.int32),
                                              torch.tensor(rng.integers(1, 5, size=n - 1), dtype=torch.int32)])).values
                        for n in sizes])
    alpha_ref, refs = _batch_reference(cfg, w, x, offsets, depths, {})
    ctx = _ctx(cfg)
    _set_weights(ctx, w, 0)
    for rep in range(2):
        out, idx, wt, mask, act, stats = ctx.moe_verify_batch(0, x, offsets, torch.tensor(alpha_ref, device=DEV),
                                                              acm.SelectParams(), want=True)
        assert ctx.device_status() == acm.OK
        for b, ref in enumerate(refs):
            np.testing.assert_array_equal(_u32(mask[b]), ref["mask"])
            np.testing.assert_array_equal(idx[offsets[b]:offsets[b + 1]].cpu().numpy(), ref["idx"])
        ref_idx = np.concatenate([r["idx"] for r in refs])
        ref_w = np.concatenate([r["w"] for r in refs])
        ffn = oracle.expert_ffn(x, ref_idx, ref_w, w["gate_up"], w["down"], w["shared_gate_up"], w["shared_down"])
        _ffn_check(out, ffn, f"sizes {sizes}")
    ctx.close()


def test_batch_call_on_random_block_partitions():
    """Forty seeded random batches: 1 to 10 blocks of random sizes over random layers, against every block verified
    alone by the oracle."""
    rng = np.random.default_rng(77)
    for case in range(40):
        E = int(rng.integers(16, 129))
        k = int(rng.integers(1, 9))
        T = int(rng.integers(1, 65))
        nb = int(rng.integers(1, min(T, 10) + 1))
        cuts = sorted(rng.choice(np.arange(1, T), size=nb - 1, replace=False).tolist()) if nb > 1 else []
        offsets = [0] + cuts + [T]
        cfg = wl.scaled(wl.CONFIGS[3], hidden=int(rng.choice([256, 512])), n_experts=E, top_k=k, inter=int(rng.choice([64, 128, 256])),
                        n_shared=int(rng.choice([0, 0, 1])), n_nodes=T, max_depth=4, n_layers=1, weighting=int(rng.integers(0, 3)))
        kw = {"fixed_budget": int(rng.integers(1, E + 1))} if rng.random() < 0.3 else {}
        w = wl.layer_weights(cfg, 0, DEV)
        x = wl.hidden_states(cfg, 0, DEV)
        depths = torch.cat([torch.sort(torch.cat([torch.zeros(1, dtype=torch.int32),
                                                  torch.tensor(rng.integers(1, 5, size=offsets[b + 1] - offsets[b] - 1), dtype=torch.int32)])).values
                            for b in range(nb)])
        alpha_ref, refs = _batch_reference(cfg, w, x, offsets, depths, kw)
        ctx = _ctx(cfg)
        _set_weights(ctx, w, 0)
        out, idx, wt, mask, act, stats = ctx.moe_verify_batch(0, x, offsets, torch.tensor(alpha_ref, device=DEV),
                                                              acm.SelectParams(**kw), want=True)
        assert ctx.device_status() == acm.OK
        for b, ref in enumerate(refs):
            np.testing.assert_array_equal(_u32(mask[b]), ref["mask"])
            np.testing.assert_array_equal(idx[offsets[b]:offsets[b + 1]].cpu().numpy(), ref["idx"])
        ref_idx = np.concatenate([r["idx"] for r in refs])
        ref_w = np.concatenate([r["w"] for r in refs])
        ffn = oracle.expert_ffn(x, ref_idx, ref_w, w["gate_up"], w["down"], w["shared_gate_up"], w["shared_down"])
        _ffn_check(out, ffn, f"random batch {case}")
        ctx.close()


@pytest.mark.parametrize("c,sizes", [(3, [64, 64]), (3, [64, 37]), (4, [48, 48, 20]), (2, [32, 32, 32, 32]), (3, [50, 30])])
def test_wide_batch_shares_one_pass_over_the_experts(c, sizes):
    """More than 64 nodes in one batch call (up to 128: two full 64-node blocks): the FFN kernel then runs with
    128-column accumulators, two 64 KB stages and an epilogue that takes the columns in two halves.  Every block's
    set and routes are those of the oracle on that block alone, every output row is within tolerance, and each
    activated expert is streamed once for all blocks.  Twice in a row on the same context."""
    cfg = wl.CONFIGS[c]
    ctx = _ctx(cfg)
    w = wl.layer_weights(cfg, 0, DEV)
    _set_weights(ctx, w, 0)
    offsets = [0] + list(np.cumsum(sizes))
    T = offsets[-1]
    rng = np.random.default_rng(sum(sizes))
    xs, depths = [], []
    for b, n in enumerate(sizes):
        xs.append(wl.hidden_states(wl.scaled(cfg, n_nodes=64), 70 + b, DEV)[:n])
        d = np.sort(rng.integers(1, cfg.max_depth + 1, size=n - 1))
        depths.append(torch.tensor(np.concatenate([[0], d]), dtype=torch.int32))
    x = torch.cat(xs).contiguous()
    alpha_ref, refs = _batch_reference(cfg, w, x, offsets, torch.cat(depths), {})
    alpha = torch.tensor(alpha_ref, device=DEV)
    ref_idx = np.concatenate([r["idx"] for r in refs])
    ref_w = np.concatenate([r["w"] for r in refs])
    ffn = oracle.expert_ffn(x, ref_idx, ref_w, w["gate_up"], w["down"], w["shared_gate_up"], w["shared_down"])
    for rep in range(2):
        out, idx, wt, mask, act, stats = ctx.moe_verify_batch(0, x, offsets, alpha, acm.SelectParams(), want=True)
        assert ctx.device_status() == acm.OK, ctx.wait_report()
        union = set()
        for b, ref in enumerate(refs):
            lo, hi = offsets[b], offsets[b + 1]
            np.testing.assert_array_equal(_u32(mask[b]), ref["mask"])
            np.testing.assert_array_equal(idx[lo:hi].cpu().numpy(), ref["idx"])
            np.testing.assert_allclose(wt[lo:hi].cpu().numpy(), ref["w"], rtol=1e-5, atol=1e-7)
            union |= set(ref["idx"].ravel().tolist()) - {-1}
        assert mask_to_set(_u32(act), cfg.n_experts) == union
        assert out.shape == (T, cfg.hidden)
        _ffn_check(out, ffn, f"C{c} wide batch {sizes}")
    # the limits: more than 128 rows in all, or a block beyond the context's own limit
    with pytest.raises(acm.AcmError):
        ctx.moe_verify_batch(0, torch.cat([x, x])[:130].contiguous(), [0, 64, 128, 130], torch.ones(130, device=DEV))
    with pytest.raises(acm.AcmError):
        ctx.moe_verify_batch(0, x[:70].contiguous(), [0, 70], torch.ones(70, device=DEV))
    ctx.close()
