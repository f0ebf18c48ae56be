"""Soak and failure-path tests of the fused calls on the GPU.

The kernels of a fused call hand data to one another through tagged words, counters and barriers, every wait
on which is bounded.  The soak test drives hundreds of fused and batch calls -- fresh and reused contexts,
1 to 32 blocks of ragged sizes, batches of up to 128 nodes, bursts without a host synchronisation, bf16 and MXFP4 layers -- and checks the
device status and the oracle's eligible sets and routes on every call.  The failure test makes one wait run
out on purpose (on the host side: a tag that nobody publishes) and checks that the library reports it,
returns promptly and is correct again afterwards."""
import time

import numpy as np
import pytest
import torch

import oracle
from paper_2608_02989_b200 import acm, workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
WAIT_LIMIT_NS = 50_000_000          # 50 ms: a call that gets stuck costs milliseconds, not a second per CTA


def _u32(t):
    return t.cpu().numpy().view(np.uint32)


def _host_bits(t):
    """A bf16 tensor as the uint16 array the oracle takes as is: copied to the host once, not on every call."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def _random_case(rng, cfg, many_blocks, wide=False):
    """A random batch: T nodes cut into nb blocks, per-block depths (root first), hidden states.  wide: more than 64
    nodes in all (the FFN kernel's 128-column form), no block above 64."""
    while True:
        if wide:
            T = int(rng.integers(65, 129))
            nb = int(rng.integers(2, 9))
        elif many_blocks:
            nb = int(rng.integers(9, 33))
            T = int(rng.integers(nb, 65))
        else:
            T = int(rng.integers(1, 65))
            nb = int(rng.integers(1, min(T, 8) + 1))
        cuts = sorted(rng.choice(np.arange(1, T), size=nb - 1, replace=False).tolist()) if nb > 1 else []
        offsets = [0] + cuts + [T]
        if max(np.diff(offsets)) <= 64:
            break
    depths = []
    for b in range(nb):
        n = offsets[b + 1] - offsets[b]
        d = np.sort(rng.integers(1, cfg.max_depth + 1, size=n - 1)) if n > 1 else np.zeros(0, dtype=np.int64)
        depths.append(np.concatenate([[0], d]).astype(np.int32))
    return T, nb, offsets, depths


def _reference(cfg, w, x, offsets, depths, p):
    refs, alphas = [], []
    for b in range(len(offsets) - 1):
        lo, hi = offsets[b], offsets[b + 1]
        a = oracle.node_weights(depths[b], p.numpy())
        refs.append(oracle.moe_verify(x[lo:hi], w["w_router"], w["router_bias"], w["gate_up"], w["down"], a, cfg.top_k,
                                      oracle.SelectParams(), weighting=cfg.weighting, with_ffn=False))
        alphas.append(a)
    return np.concatenate(alphas), refs


def _check_burst(ctx, cfg, w_ffn, pending, what):
    st = ctx.device_status()
    assert st == acm.OK, f"{what}: device status {st}, waits that gave up per CTA: {ctx.wait_report()}"
    for (single, x, offsets, refs, res) in pending:
        T = x.shape[0]
        if isinstance(res, tuple):            # the call returned sets and routes: compared bit for bit
            if single:
                out, idx, wt, mask, stats = res
                np.testing.assert_array_equal(_u32(mask)[: len(refs[0]["mask"])], refs[0]["mask"])
                np.testing.assert_array_equal(idx.cpu().numpy(), refs[0]["idx"])
            else:
                out, idx, wt, mask, act, stats = res
                for b, ref in enumerate(refs):
                    np.testing.assert_array_equal(_u32(mask[b]), ref["mask"])
                    np.testing.assert_array_equal(idx[offsets[b]:offsets[b + 1]].cpu().numpy(), ref["idx"])
        else:
            out = res
        # three output rows against the oracle's FFN on the oracle's routes (a wrong route shows here too)
        rows = sorted({0, T // 2, T - 1})
        ref_idx = np.concatenate([r["idx"] for r in refs])[rows]
        ref_w = np.concatenate([r["w"] for r in refs])[rows]
        sel = torch.as_tensor(rows, device=x.device)
        ffn = oracle.expert_ffn(x[sel], ref_idx, ref_w, w_ffn[0], w_ffn[1])
        got = out[sel].double().cpu().numpy()
        rms = float(np.sqrt(np.mean(ffn ** 2)))
        assert np.isfinite(got).all() and float(np.abs(got - ffn).max()) <= 2e-2 * rms, what


def _soak(cfg, layers, ffn_weights, set_weights, n_rounds, calls_per_round, seed, wide_ok=True):
    rng = np.random.default_rng(seed)
    p = wl.commitment_table(cfg)
    gen = torch.Generator(device=DEV).manual_seed(seed)
    done = 0
    for rnd in range(n_rounds):
        ctx = acm.Context.for_config(cfg, n_layers=len(layers))       # a fresh context: tags and counters start over
        ctx.set_wait_limit(WAIT_LIMIT_NS)
        for l in range(len(layers)):
            set_weights(ctx, l)
        i = 0
        while i < calls_per_round:
            burst, tight = min(int(rng.integers(1, 9)), calls_per_round - i), bool(rng.integers(0, 2))
            cases = []
            for j in range(burst):            # inputs and references of the whole burst first ...
                layer = int(rng.integers(0, len(layers)))
                T, nb, offsets, depths = _random_case(rng, cfg, many_blocks=((i + j) % 4 == 3),
                                                      wide=wide_ok and (i + j) % 4 == 1)
                x = torch.randn(T, cfg.hidden, generator=gen, device=DEV).to(torch.bfloat16)
                alpha, refs = _reference(cfg, layers[layer], x, offsets, depths, p)
                single = nb == 1 and bool(rng.integers(0, 2))
                cases.append((layer, single, x, offsets, refs, torch.tensor(alpha, device=DEV)))
            torch.cuda.synchronize()
            pending = []
            for layer, single, x, offsets, refs, alpha_dev in cases:      # ... then the calls, back to back
                # a tight burst asks for no optional output: nothing is enqueued between one call's last kernel and
                # the next call's first, so they overlap as in a serving loop
                if single:
                    res = ctx.moe_verify(layer, x, alpha_dev, acm.SelectParams(), want=not tight)
                else:
                    res = ctx.moe_verify_batch(layer, x, offsets, alpha_dev, acm.SelectParams(), want=not tight)
                pending.append((layer, (single, x, offsets, refs, res)))
            for layer, item in pending:
                _check_burst(ctx, cfg, ffn_weights[layer], [item], f"round {rnd} calls {i}..{i + burst - 1}")
            done += burst
            i += burst
        ctx.close()
    return done


def test_soak_fused_and_batch_calls_bf16():
    """300 calls on the Qwen3-30B-A3B-shaped layer (the full shape: 12 tiles per expert, leftover tiles cut over the
    CTAs, anchors of several roots), three fresh contexts."""
    cfg = wl.scaled(wl.CONFIGS[3], n_layers=2)
    layers = [wl.layer_weights(cfg, l, DEV) for l in range(2)]

    def set_weights(ctx, l):
        w = layers[l]
        ctx.set_layer_weights(l, w["w_router"], w["router_bias"], w["gate_up"], w["down"])

    ffn_weights = [(_host_bits(w["gate_up"]), _host_bits(w["down"])) for w in layers]
    host_layers = [dict(w_router=_host_bits(w["w_router"]), router_bias=w["router_bias"].cpu().numpy(), gate_up=None,
                        down=None) for w in layers]
    assert _soak(cfg, host_layers, ffn_weights, set_weights, n_rounds=3, calls_per_round=100, seed=11) == 300


def test_soak_fused_and_batch_calls_mxfp4():
    """The same on an MXFP4 layer (the second build of the FFN kernel), 100 calls."""
    cfg = wl.scaled(wl.CONFIGS[3], n_layers=1, inter=256, n_experts=64)
    w = wl.layer_weights_mxfp4(cfg, 0, DEV)
    gu_t = acm.pack_mxfp4_gate_up(w["gate_up_codes"], w["gate_up_scales"]).to(DEV)
    dn_t = acm.pack_mxfp4_down(w["down_codes"], w["down_scales"]).to(DEV)
    # what the layer means: the bf16 layer on the dequantised weights
    gu = torch.tensor(oracle.dequantize_mxfp4(w["gate_up_codes"], w["gate_up_scales"])).to(torch.bfloat16)
    dn = torch.tensor(oracle.dequantize_mxfp4(w["down_codes"], w["down_scales"])).to(torch.bfloat16)
    w["gate_up"] = w["down"] = None                     # (the reference routes need the router alone)

    def set_weights(ctx, l):
        ctx.set_layer_weights_mxfp4(l, w["w_router"], w["router_bias"], gu_t, dn_t)

    host_w = dict(w_router=_host_bits(w["w_router"]), router_bias=w["router_bias"].cpu().numpy(), gate_up=None, down=None)
    assert _soak(cfg, [host_w], [(_host_bits(gu), _host_bits(dn))], set_weights, n_rounds=1, calls_per_round=100,
                 seed=12, wide_ok=False) == 100


def test_wait_that_runs_out_is_reported_and_the_context_recovers():
    """A bounded wait that expires: the FFN kernel is launched waiting for an eligible set under a tag that no kernel
    publishes (the failure is made on the host; nothing faults or hangs).  With a 3 ms limit the call must come back
    at once with ACM_ERR_TIMEOUT, name the wait in every CTA, and leave a context whose next calls match the oracle."""
    cfg = wl.scaled(wl.CONFIGS[3], n_layers=1, inter=256)
    w = wl.layer_weights(cfg, 0, DEV)
    x = wl.hidden_states(cfg, 0, DEV)
    depth, p = wl.tree_depths(cfg), wl.commitment_table(cfg)
    alpha = acm.node_weights(depth, p)
    ref = oracle.moe_verify(x, w["w_router"], w["router_bias"], w["gate_up"], w["down"], alpha.numpy(), cfg.top_k,
                            oracle.SelectParams(), weighting=cfg.weighting)
    rms = float(np.sqrt(np.mean(ref["out"] ** 2)))

    def check_good_call():
        out, idx, wt, mask, stats = ctx.moe_verify(0, x, alpha.to(DEV), acm.SelectParams(), want=True)
        assert ctx.device_status() == acm.OK
        np.testing.assert_array_equal(_u32(mask), ref["mask"])
        np.testing.assert_array_equal(idx.cpu().numpy(), ref["idx"])
        assert float(np.abs(out.double().cpu().numpy() - ref["out"]).max()) <= 2e-2 * rms

    ctx = acm.Context.for_config(cfg, n_layers=1)
    ctx.set_layer_weights(0, w["w_router"], w["router_bias"], w["gate_up"], w["down"])
    with pytest.raises(acm.AcmError):
        ctx.set_wait_limit(10)                      # below a microsecond: refused
    check_good_call()
    ctx.set_wait_limit(3_000_000)
    for _ in range(2):                              # twice: the error path itself leaves nothing behind
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        ctx.inject_unpublished_wait(0, x)
        st = ctx.device_status()
        dt = time.perf_counter() - t0
        assert st == acm.ERR_TIMEOUT
        assert dt < 0.5, f"a 3 ms limit took {dt:.3f} s to come back"
        report = ctx.wait_report()
        assert len(report) == torch.cuda.get_device_properties(0).multi_processor_count
        assert set(report) == {2}, report           # every CTA gave up waiting for the eligible set's words
        assert ctx.device_status() == acm.OK        # sticky until read, then cleared
        check_good_call()
    ctx.set_wait_limit(1_000_000_000)
    check_good_call()
    assert set(ctx.wait_report()) == {0}
    ctx.close()


def test_sequence_tags_coming_round_do_not_revive_old_words():
    """The words the kernels publish for one another carry the call's sequence number in 16 bits.  A batch call
    writes words for eight blocks; 65534 single-block calls later the tags come round, and a second batch call,
    on other hidden states, gets the first one's tag again.  The old words of blocks 1..7 must not pass for
    current ones: sets, routes and every output row against the oracle."""
    import ctypes
    cfg = wl.scaled(wl.CONFIGS[3], hidden=256, inter=64, n_experts=16, top_k=2, n_nodes=16, max_depth=1, n_layers=1)
    w = wl.layer_weights(cfg, 0, DEV)
    p = wl.commitment_table(cfg)
    offsets = list(range(0, 17, 2))                       # eight blocks of two nodes
    depths = [np.array([0, 1], dtype=np.int32)] * 8
    ctx = acm.Context.for_config(cfg, n_layers=1)
    ctx.set_layer_weights(0, w["w_router"], w["router_bias"], w["gate_up"], w["down"])
    host_w = dict(w_router=_host_bits(w["w_router"]), router_bias=w["router_bias"].cpu().numpy(), gate_up=None, down=None)
    ffn_w = (_host_bits(w["gate_up"]), _host_bits(w["down"]))

    def batch_call(seed):
        x = wl.hidden_states(cfg, seed, DEV)
        alpha, refs = _reference(cfg, host_w, x, offsets, depths, p)
        res = ctx.moe_verify_batch(0, x, offsets, torch.tensor(alpha, device=DEV), acm.SelectParams(), want=True)
        assert ctx.device_status() == acm.OK
        out, idx, wt, mask, act, stats = res
        for b, ref in enumerate(refs):
            np.testing.assert_array_equal(_u32(mask[b]), ref["mask"])
            np.testing.assert_array_equal(idx[offsets[b]:offsets[b + 1]].cpu().numpy(), ref["idx"])
        ffn = oracle.expert_ffn(x, np.concatenate([r["idx"] for r in refs]), np.concatenate([r["w"] for r in refs]), *ffn_w)
        rms = float(np.sqrt(np.mean(ffn ** 2)))
        assert float(np.abs(out.double().cpu().numpy() - ffn).max()) <= 2e-2 * rms
        return [r["mask"].copy() for r in refs]

    first = batch_call(1)
    x1 = wl.hidden_states(cfg, 2, DEV)[:2].contiguous()
    alpha1 = torch.tensor(oracle.node_weights(depths[0], p.numpy()), device=DEV)
    out1 = torch.empty(2, cfg.hidden, dtype=torch.float32, device=DEV)
    params = acm.SelectParams()
    sp = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    args = (ctx.handle, 0, ctypes.c_void_p(x1.data_ptr()), 2, ctypes.c_void_p(alpha1.data_ptr()), ctypes.byref(params), None,
            ctypes.c_void_p(out1.data_ptr()), None, None, None, None, sp)
    for _ in range(65534):
        assert ctx.lib.acm_moe_verify(*args) == 0
    assert ctx.device_status() == acm.OK
    second = batch_call(3)
    assert any((a != b).any() for a, b in zip(first, second))       # (the two batches do have different sets)
    ctx.close()
