"""The allocation-free fp32 expert FFN entry point against the context-based one.

Some callers cannot allocate device memory at the moment they call into this library (they run
inside someone else's memory pool, or an implicit synchronisation from cudaMalloc would stall
them), so one entry point keeps its scratch in a fixed array of the library image.  Called
through the C ABI twice in a row, it must give what acm_expert_ffn gives, and it must refuse
sizes beyond its fixed scratch.  Collected last on purpose."""
import numpy as np
import pytest
import torch

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
        acm.expert_ffn_f32_noalloc(x, idx, wt, w["gate_up"], w["down"], out)
        torch.cuda.synchronize()
        rms = float(want.double().pow(2).mean().sqrt())
        err = float((out.double() - want.double()).abs().max())
        assert torch.isfinite(out).all()
        assert err <= 2e-2 * rms, (call, err, rms)
        ctx.close()


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
