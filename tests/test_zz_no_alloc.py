"""The allocation-free fp32 expert FFN entry point against the context-based one and against the oracle.

Some callers cannot allocate device memory at the moment they call into this library (they run
inside someone else's memory pool, or an implicit synchronisation from cudaMalloc would stall
them), so one entry point keeps its scratch in a fixed array of the library image.  Called
through the C ABI twice in a row, it must give what acm_expert_ffn gives and what the CPU oracle
computes, leave the device's free memory as it found it, treat expert ids outside the layer as
empty slots, and refuse sizes beyond its fixed scratch.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_02989_b200 import acm, workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(seed):
    cfg = wl.CONFIGS[1]
    w = wl.layer_weights(cfg, seed, DEV)
    x = wl.hidden_states(cfg, seed, DEV)
    rng = np.random.default_rng(seed)
    idx = np.array([rng.permutation(cfg.n_experts)[:cfg.top_k] for _ in range(cfg.n_nodes)], dtype=np.int32)
    idx[2, 1] = -1
    wt = rng.uniform(0.1, 1.0, idx.shape).astype(np.float32)
    return cfg, w, x, torch.tensor(idx, device=DEV), torch.tensor(wt, device=DEV)


def test_noalloc_matches_context_entry_point_twice_in_a_row():
    for call in range(2):
        cfg, w, x, idx, wt = _inputs(call)
        ctx = acm.Context.for_config(cfg, n_layers=1)
        ctx.set_layer_weights(0, w["w_router"], None, w["gate_up"], w["down"])
        want = ctx.expert_ffn(0, x, idx, wt)
        out = torch.full_like(want, float("nan"))          # caller-owned output, allocated before the call
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        acm.expert_ffn_f32_noalloc(x, idx, wt, w["gate_up"], w["down"], out)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before                   # nothing was allocated (or freed) on the device
        rms = float(want.double().pow(2).mean().sqrt())
        err = float((out.double() - want.double()).abs().max())
        assert torch.isfinite(out).all()
        assert err <= 2e-2 * rms, (call, err, rms)
        # ... and against the CPU oracle (the two library entry points share their kernels)
        ref = oracle.expert_ffn(x, idx.cpu().numpy(), wt.double().cpu().numpy(), w["gate_up"], w["down"])
        rms_o = float(np.sqrt(np.mean(ref ** 2)))
        assert float(np.abs(out.double().cpu().numpy() - ref).max()) <= 1e-4 * rms_o      # fp32 against fp64
        ctx.close()


def test_noalloc_treats_expert_ids_outside_the_layer_as_empty_slots():
    """An id >= n_experts must read no weights: it contributes nothing, exactly like -1."""
    cfg, w, x, idx, wt = _inputs(5)
    bad = idx.clone()
    bad[0, 0] = cfg.n_experts            # first id past the layer
    bad[3, 1] = 10 ** 6
    hole = idx.clone()
    hole[0, 0] = -1
    hole[3, 1] = -1
    out_bad = torch.full((cfg.n_nodes, cfg.hidden), float("nan"), device=DEV)
    out_hole = torch.full_like(out_bad, float("nan"))
    acm.expert_ffn_f32_noalloc(x, bad, wt, w["gate_up"], w["down"], out_bad)
    acm.expert_ffn_f32_noalloc(x, hole, wt, w["gate_up"], w["down"], out_hole)
    torch.cuda.synchronize()
    assert torch.equal(out_bad, out_hole)
    ref = oracle.expert_ffn(x, hole.cpu().numpy(), wt.double().cpu().numpy(), w["gate_up"], w["down"])
    assert float(np.abs(out_bad.double().cpu().numpy() - ref).max()) <= 1e-4 * float(np.sqrt(np.mean(ref ** 2)))
    # the context-based call on an fp32 layer bounds the ids the same way
    ctx = acm.Context.for_config(cfg, n_layers=1)
    ctx.set_layer_weights(0, w["w_router"], None, w["gate_up"], w["down"])
    assert torch.equal(ctx.expert_ffn(0, x, bad, wt), out_hole)
    ctx.close()


def test_noalloc_wrapper_rejects_tensors_it_cannot_pass_on():
    cfg, w, x, idx, wt = _inputs(6)
    out = torch.empty(cfg.n_nodes, cfg.hidden, device=DEV)
    with pytest.raises(TypeError):
        acm.expert_ffn_f32_noalloc(x.double(), idx, wt, w["gate_up"], w["down"], out)
    with pytest.raises(TypeError):
        acm.expert_ffn_f32_noalloc(x, idx.long(), wt, w["gate_up"], w["down"], out)
    with pytest.raises(ValueError):
        acm.expert_ffn_f32_noalloc(x.t().contiguous().t(), idx, wt, w["gate_up"], w["down"], out)
    with pytest.raises(ValueError):
        acm.expert_ffn_f32_noalloc(x.cpu(), idx, wt, w["gate_up"], w["down"], out)


def test_noalloc_rejects_sizes_beyond_its_scratch():
    T, H, E, k = 64, 32, 8, 8
    I = acm.NOALLOC_MAX_FLOATS // (T * k) + 1            # one feature too many
    x = torch.zeros(T, H, device=DEV)
    idx = torch.zeros(T, k, dtype=torch.int32, device=DEV)
    wt = torch.zeros(T, k, device=DEV)
    gate_up = torch.zeros(1, device=DEV)                  # never read: the call must fail before any launch
    out = torch.full((T, H), 3.0, device=DEV)
    lib = acm.load_library()
    rc = lib.acm_expert_ffn_f32_noalloc(acm._p(x), T, H, I, E, k, acm._p(idx), acm._p(wt), acm._p(gate_up),
                                        acm._p(gate_up), acm._p(out), None)
    assert rc == acm.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert bool((out == 3.0).all())
    assert "limit" in acm.status_string(rc)
