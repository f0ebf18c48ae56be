"""The input recipe: shapes, seeds, tree and table structure of the five configurations."""
import numpy as np
import torch

from paper_2608_02989_b200 import workloads as wl


def test_config_shapes_and_sizes():
    c3 = wl.CONFIGS[3]
    assert (c3.hidden, c3.n_experts, c3.top_k, c3.inter, c3.n_nodes, c3.n_layers) == (2048, 128, 8, 768, 64, 48)
    assert c3.expert_bytes == 3 * 2048 * 768 * 2 == 9_437_184
    assert wl.CONFIGS[5].expert_bytes == 37_748_736
    assert wl.CONFIGS[1].dtype == "f32" and wl.CONFIGS[1].seed(0) == 0
    assert wl.CONFIGS[4].n_shared == 2 and wl.CONFIGS[4].top_k == 6


def test_trees_and_tables():
    assert wl.tree_depths(wl.CONFIGS[1]).tolist() == [0, 1, 1, 2, 2, 3, 3, 3]
    np.testing.assert_allclose(wl.commitment_table(wl.CONFIGS[1]).numpy(), [1.0, 0.8, 0.64, 0.512], rtol=1e-6)
    np.testing.assert_allclose(wl.commitment_table(wl.CONFIGS[2]).numpy()[:2], [0.9, 0.675], rtol=1e-6)
    for c in (2, 3, 4, 5):
        cfg = wl.CONFIGS[c]
        d = wl.tree_depths(cfg).numpy()
        assert len(d) == cfg.n_nodes and d[0] == 0 and (d[1:] >= 1).all()
        assert np.all(np.diff(d) >= 0) and set(d) == set(range(cfg.max_depth + 1))
        assert len(wl.commitment_table(cfg)) == cfg.max_depth + 1
        assert torch.equal(wl.tree_depths(cfg), wl.tree_depths(cfg))


def test_weights_are_seeded_and_distributed_as_stated():
    cfg = wl.scaled(wl.CONFIGS[3], inter=64, n_experts=16)
    a = wl.layer_weights(cfg, 0)
    b = wl.layer_weights(cfg, 0)
    c = wl.layer_weights(cfg, 1)
    assert torch.equal(a["gate_up"], b["gate_up"]) and not torch.equal(a["gate_up"], c["gate_up"])
    assert a["gate_up"].shape == (16, 128, 2048) and a["down"].shape == (16, 2048, 64)
    assert a["gate_up"].dtype == torch.bfloat16
    assert abs(a["gate_up"].float().std().item() - 0.02) < 1e-3
    bias = a["router_bias"].double().numpy()
    np.testing.assert_allclose(np.sort(-bias / 1.1), np.log(np.arange(1, 17)), rtol=1e-6)
    x = wl.hidden_states(cfg, 0)
    assert x.shape == (64, 2048) and abs(x.float().std().item() - 1.0) < 0.02
    assert not torch.equal(x, wl.hidden_states(cfg, 1))
    assert wl.layer_weights(wl.CONFIGS[1], 0, experts=False)["router_bias"] is None


def test_resident_mask_fraction():
    cfg = wl.CONFIGS[5]
    m = wl.resident_mask(cfg, 3).numpy().view(np.uint32)
    assert sum(bin(int(v)).count("1") for v in m) == 51
    assert not np.array_equal(m, wl.resident_mask(cfg, 4).numpy().view(np.uint32))
    full = wl.resident_mask(wl.CONFIGS[3], 0).numpy().view(np.uint32)
    assert all(int(v) == 0xFFFFFFFF for v in full)
