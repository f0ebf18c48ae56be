#!/usr/bin/env python
"""Benchmark of the verifier-side MoE layer (one JSON line on stdout).

A step is one verification block through the whole hot path (router, selection, restricted
routing, expert FFN) of every layer of the configuration's stack, layers back to back with
distinct weights so that expert weights stream cold from HBM.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--layers L] [--impl reference]

metric  verify-blocks/s per MoE layer = (layers x steps) / time, summed over replicas.
N > 1   independent replicas (the path has no sharding and no collective): one rank per GPU
        under torchrun, barrier + max-over-ranks timing.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

DRAM_BYTES_PER_ACTIVATED_EXPERT = {3: (273758464 + 193700864 + 193257216) / 68.0}   # config -> bytes (ncu, profiles/)
METRIC = "verify_blocks_per_s_per_moe_layer"
UNIT = "layer-blocks/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps (default 100; 3 for config 5 as configured, whose steps are bound by host-to-device "
                         "copies; 20 for --impl reference)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=3, help="1..5; default 3 = Qwen3-30B-A3B-shaped stack")
    ap.add_argument("--layers", type=int, default=0, help="override the number of stacked layers (0 = the config's)")
    ap.add_argument("--impl", default="acm", choices=["acm", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-natural", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--selector", default="acceptmoe", choices=["acceptmoe", "acceptmoe-b", "count-b", "moe-spec"],
                    help="eligible-set policy of the restricted path: the paper's self-sizing selector (default), its "
                         "fixed-budget variant, or the fixed-budget baselines of Section 4.1 (votes / summed router mass)")
    ap.add_argument("--budget", type=int, default=22, help="B0 of the fixed-budget selectors")
    ap.add_argument("--mxfp4", action="store_true",
                    help="supplementary: the routed experts stored in MXFP4 (the configuration's weights quantised), "
                         "expanded to bf16 inside the FFN kernel")
    ap.add_argument("--zipf", action="store_true",
                    help="supplementary: give the configuration the Zipf(1.1) router bias that C3 has (skewed expert "
                         "popularity), e.g. --config 5 --zipf")
    ap.add_argument("--overlap", type=int, default=3, choices=[0, 1, 2, 3],
                    help="acm_set_overlap level: 0 plain stream order (cooperative FFN launch), 1 dependent launches, "
                         "2 + FFN start on the eligible set, 3 + FFN start on the anchors (default)")
    ap.add_argument("--bracket-every", type=int, default=47,
                    help="bracket every n-th FFN launch with events for the roofline figure (0: none, the pure pipeline)")
    ap.add_argument("--all-resident", action="store_true",
                    help="config 5 only: every expert on the GPU (no offloading) instead of the configured 40 % residency")
    ap.add_argument("--batch", type=int, default=0,
                    help="supplementary run: B > 1 verification blocks per call (they share the config's nodes and "
                         "one pass over the expert weights) against the same blocks verified one call each")
    ap.add_argument("--batch-nodes", type=int, default=0,
                    help="with --batch: nodes of all blocks together (default: the configuration's; up to 128, e.g. "
                         "--batch 2 --batch-nodes 128 = two full 64-node blocks per call)")
    ap.add_argument("--pool", type=int, default=0,
                    help="supplementary run: config-5-shaped layers (Zipf-biased routing) behind an LRU expert pool "
                         "of this many slots per layer; reports hit rate and host-to-device MiB per block")
    args = ap.parse_args()
    if args.steps is None:
        if args.impl == "reference":
            args.steps = 20           # (each step of the oracle is a bounded sample of about half a second)
        elif args.config == 5 and not args.all_resident and not args.pool:
            args.steps = 3
        else:
            args.steps = 100
    return args


def read_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.samples = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "10"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            f = [v.strip() for v in s.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                smax = float(f[1])
            except ValueError:
                continue
            for name, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        # the clock rises only under load: report the median of the upper half of the samples
        busy = sm[len(sm) // 2:] if sm else []
        med = busy[len(busy) // 2] if busy else None
        return {"sm_mhz": med, "sm_max_mhz": smax, "reasons": sorted(reasons), "samples": len(sm)}


def aggregate_over_ranks(local_ms: float, local_units: float, dist=None, device="cpu"):
    """Replicas only: every rank runs the same independent workload.  Returns (max time over ranks in ms,
    units summed over ranks); the job's throughput is their ratio."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms, local_units
    import torch
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t), float(u)


def dist_setup(args):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return world, rank, local


def relaunch_as_replicas(n_gpus: int, argv=None) -> int:
    """`bench.py --gpus N` started as one plain process: start the N replicas (one process per GPU) under
    torch.distributed.run on this node and pass their output through.  Returns the launcher's exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")            # the communicator's own log names its ranks
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), str(ROOT / "bench.py")] + list(argv if argv is not None else sys.argv[1:])
    return subprocess.run(cmd, env=env).returncode


# ------------------------------------------------------------------------------------------
def run_pool(args):
    """Offload variant (Section 3.4): every layer's experts live in an X-slot LRU pool on the GPU, the full
    weights in pinned host memory.  A 'step' is one verification block through the stacked layers; the blocks
    differ (new hidden states each step), so the pools see a changing demand."""
    import ctypes

    import numpy as np
    import torch

    from paper_2608_02989_b200 import acm, workloads as wl
    from paper_2608_02989_b200 import build as acm_build

    acm_build.build_library()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    cfg = wl.scaled(wl.CONFIGS[5], zipf_bias=True)
    L = args.layers or 4
    X = args.pool
    T, H, E = cfg.n_nodes, cfg.hidden, cfg.n_experts
    ctx = acm.Context.for_config(cfg, n_layers=L)
    keep = []
    for l in range(L):
        if args.mxfp4:
            w = wl.layer_weights_mxfp4(cfg, l, dev)
            gu = acm.pack_mxfp4_gate_up(w.pop("gate_up_codes"), w.pop("gate_up_scales"))
            dn = acm.pack_mxfp4_down(w.pop("down_codes"), w.pop("down_scales"))
            host_gu, host_dn = gu.cpu().pin_memory(), dn.cpu().pin_memory()
            pool_gu = torch.empty((X,) + tuple(gu.shape[1:]), dtype=torch.uint8, device=dev)
            pool_dn = torch.empty((X,) + tuple(dn.shape[1:]), dtype=torch.uint8, device=dev)
            del gu, dn
            ctx.set_layer_weights_mxfp4(l, w["w_router"], w["router_bias"], None, None)
        else:
            w = wl.layer_weights(cfg, l, dev)
            host_gu, host_dn = w["gate_up"].cpu().pin_memory(), w["down"].cpu().pin_memory()
            pool_gu = torch.empty((X,) + tuple(w["gate_up"].shape[1:]), dtype=w["gate_up"].dtype, device=dev)
            pool_dn = torch.empty((X,) + tuple(w["down"].shape[1:]), dtype=w["down"].dtype, device=dev)
            ctx.set_layer_weights(l, w["w_router"], w["router_bias"], None, None)
        ctx.set_slot_pool(l, pool_gu, pool_dn, host_gu, host_dn, list(range(X)))     # starts full: experts 0..X-1
        keep.append((w["w_router"], w["router_bias"], host_gu, host_dn, pool_gu, pool_dn))
        del w
        torch.cuda.empty_cache()
    n_blocks = max(args.steps, 8)
    xs = [[wl.hidden_states(cfg, 100 * b + l, dev) for l in range(L)] for b in range(n_blocks)]
    alpha = acm.node_weights(wl.tree_depths(cfg), wl.commitment_table(cfg)).to(dev)
    out = torch.zeros(T, H, dtype=torch.float32, device=dev)
    stats = torch.zeros(12, dtype=torch.int32, device=dev)
    full = torch.full((ctx.words,), -1, dtype=torch.int32, device=dev)
    res = {}
    for name, kw in (("restricted_eq7", dict(params=acm.SelectParams(residency=1))),
                     ("restricted_no_pruning", dict(params=acm.SelectParams(residency=0))),
                     ("natural", dict(params=None, mask_override=full))):
        for l in range(L):      # same starting pool for every policy
            ctx.set_slot_pool(l, keep[l][4], keep[l][5], keep[l][2], keep[l][3], list(range(X)))
        n_act = []
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        try:
            for b in range(n_blocks):
                for l in range(L):
                    ctx.moe_verify(l, xs[b][l], alpha if kw.get("params") is not None else None, kw.get("params"),
                                   mask_override=kw.get("mask_override"), out=out)
        except acm.AcmError as err:
            torch.cuda.synchronize()
            if err.code != acm.ERR_UNSUPPORTED:
                raise
            res[name] = {"unsupported": "a block activated more experts than the pool has slots: needs the paper's waves"}
            continue
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        ctx.check_device_status()
        hits = misses = h2d = 0
        for l in range(L):
            ps = ctx.pool_stats(l, reset=True)
            hits += ps["hits"]; misses += ps["misses"]; h2d += ps["h2d_bytes"]
        res[name] = {"layer_blocks_per_s": n_blocks * L / dt, "hit_rate": hits / max(hits + misses, 1),
                     "activated_per_layer_block": (hits + misses) / (n_blocks * L),
                     "h2d_mib_per_layer_block": h2d / 2 ** 20 / (n_blocks * L),
                     "h2d_gbs": h2d / dt / 1e9}      # host->device rate over the whole run (the bound of this variant)
    line = {"metric": METRIC, "value": res["restricted_eq7"]["layer_blocks_per_s"], "unit": UNIT, "n_gpus": 1,
            "steps": n_blocks, "warmup": 0, "higher_is_better": True, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": f"C5 {cfg.name}-shaped layers{' in MXFP4' if args.mxfp4 else ''} with Zipf-biased routing behind an LRU pool of {X} "
                                   f"expert slots per layer (offload variant); {L} layers, {n_blocks} distinct blocks",
                       "hidden": H, "n_experts": E, "top_k": cfg.top_k, "inter": cfg.inter, "n_nodes": T},
            "policies": res}
    print(json.dumps(line))


def run_reference(args, world, rank):
    """The CPU oracle as the reference arm: each step is a bounded sample of the workload.  With several ranks
    rank 0 alone does the work; the ranks only meet (gloo) so that the line can say how many there were."""
    ranks_seen = 1
    if world > 1:
        import torch
        import torch.distributed as dist
        dist.init_process_group("gloo")
        one = torch.ones(1)
        dist.all_reduce(one)
        ranks_seen = int(one.item())
        dist.destroy_process_group()
    if rank != 0:
        return
    import numpy as np
    import oracle
    from paper_2608_02989_b200 import workloads as wl

    cfg = wl.CONFIGS[args.config]
    blocks_per_step = 4                      # bounded sample: a step is 4 whole layer-blocks, not the whole stack
    depth, p = wl.tree_depths(cfg), wl.commitment_table(cfg)
    alpha = oracle.node_weights(depth.numpy(), p.numpy())
    layers = [(wl.layer_weights(cfg, l, "cpu"), wl.hidden_states(cfg, l, "cpu")) for l in range(min(2, cfg.n_layers))]
    cores = os.cpu_count() or 1

    def one_step():
        for i in range(blocks_per_step):
            w, x = layers[i % len(layers)]
            oracle.moe_verify(x, w["w_router"], w["router_bias"], w["gate_up"], w["down"], alpha, cfg.top_k,
                              weighting=cfg.weighting, shared_gate_up=w["shared_gate_up"],
                              shared_down=w["shared_down"])

    for _ in range(min(max(args.warmup, 1), 3)):
        one_step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_step()
    dt = time.perf_counter() - t0
    value = blocks_per_step * args.steps / dt
    sample = (f"each step = {blocks_per_step} whole layer-blocks of C{cfg.index} (all stages, all {cfg.n_nodes} nodes) "
              f"instead of the {cfg.n_layers}-layer stack")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "ranks_seen": ranks_seen,
        "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": f"C{cfg.index} {cfg.name}-shaped", "hidden": cfg.hidden, "n_experts": cfg.n_experts,
                   "top_k": cfg.top_k, "inter": cfg.inter, "n_nodes": cfg.n_nodes, "layers": blocks_per_step},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
def cpu_baseline(cfg, budget_s=15.0):
    """Times the oracle, as it stands, on the host cores for a bounded sample of the workload:
    whole layer-blocks (every stage, every node) over the first layers until the budget is spent."""
    import oracle
    from paper_2608_02989_b200 import workloads as wl

    depth, p = wl.tree_depths(cfg), wl.commitment_table(cfg)
    alpha = oracle.node_weights(depth.numpy(), p.numpy())
    layers = [(wl.layer_weights(cfg, l, "cpu"), wl.hidden_states(cfg, l, "cpu")) for l in range(min(2, cfg.n_layers))]
    t0 = time.perf_counter()
    done = 0
    while True:
        w, x = layers[done % len(layers)]
        oracle.moe_verify(x, w["w_router"], w["router_bias"], w["gate_up"], w["down"], alpha, cfg.top_k,
                          weighting=cfg.weighting, shared_gate_up=w["shared_gate_up"], shared_down=w["shared_down"])
        done += 1
        dt = time.perf_counter() - t0
        if dt > budget_s or done >= 400:
            break
    return {"value": done / dt, "unit": UNIT, "cores": os.cpu_count() or 1, "kind": "oracle",
            "sample": (f"{done} whole layer-blocks of C{cfg.index} (all stages, all {cfg.n_nodes} nodes) cycling over "
                       f"{len(layers)} layers; {dt:.1f} s wall")}


def run_acm(args, world, rank, local):
    import ctypes

    import numpy as np
    import torch

    from paper_2608_02989_b200 import acm, workloads as wl
    from paper_2608_02989_b200 import build as acm_build

    acm_build.build_library()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    cfg = wl.CONFIGS[args.config]
    if args.zipf and not cfg.zipf_bias:
        cfg = wl.scaled(cfg, zipf_bias=True)
    L = args.layers or cfg.n_layers
    resident = cfg.resident_frac > 0
    if resident:
        # the full stack does not fit in HBM: as many physical layers as fit, reused cyclically
        free, _ = torch.cuda.mem_get_info()
        L_phys = max(1, min(L, int(0.6 * free // wl.weight_bytes_per_layer(cfg))))
    else:
        L_phys = L
    T, H, E, k = cfg.n_nodes, cfg.hidden, cfg.n_experts, cfg.top_k

    ctx = acm.Context.for_config(cfg, n_layers=L_phys)
    ctx.set_overlap(args.overlap)
    keep = []
    for l in range(L_phys):
        if args.mxfp4:
            w = wl.layer_weights_mxfp4(cfg, l + 1000 * rank, dev)
            gu = acm.pack_mxfp4_gate_up(w.pop("gate_up_codes"), w.pop("gate_up_scales"))
            dn = acm.pack_mxfp4_down(w.pop("down_codes"), w.pop("down_scales"))
            ctx.set_layer_weights_mxfp4(l, w["w_router"], w["router_bias"], gu, dn)
            keep.append((w["w_router"], w["router_bias"], gu, dn))
            continue
        w = wl.layer_weights(cfg, l + 1000 * rank, dev)
        ctx.set_layer_weights(l, w["w_router"], w["router_bias"], w["gate_up"], w["down"], w["shared_gate_up"],
                              w["shared_down"])
        keep.append(w)
    xs = torch.stack([wl.hidden_states(cfg, l + 1000 * rank, dev) for l in range(L)])       # [L,T,H]
    depth, p = wl.tree_depths(cfg), wl.commitment_table(cfg)
    alpha = acm.node_weights(depth, p)
    if args.selector in ("count-b", "moe-spec"):
        alpha = torch.ones_like(alpha)           # the baselines weigh every node alike
    alpha_dev = alpha.to(dev)
    outs = torch.zeros(L, T, H, dtype=torch.float32, device=dev)
    stats = torch.zeros(L, 12, dtype=torch.int32, device=dev)
    full = torch.full((ctx.words,), -1, dtype=torch.int32, device=dev)
    params = {"acceptmoe": acm.SelectParams(),
              "acceptmoe-b": acm.SelectParams(fixed_budget=args.budget),
              "count-b": acm.SelectParams(demand=2, use_anchors=0, fixed_budget=args.budget),
              "moe-spec": acm.SelectParams(demand=1, use_anchors=0, fixed_budget=args.budget)}[args.selector]
    selector_name = {"acceptmoe": "restricted (AcceptMoE) routing",
                     "acceptmoe-b": f"restricted routing, AcceptMoE-B with B0={args.budget}",
                     "count-b": f"restricted routing, Count-B baseline with B0={args.budget}",
                     "moe-spec": f"restricted routing, MoE-Spec baseline with B0={args.budget}"}[args.selector]
    stream = torch.cuda.current_stream()
    sp = ctypes.c_void_p(stream.cuda_stream)
    lib, h = ctx.lib, ctx.handle

    def vp(t):
        return ctypes.c_void_p(t.data_ptr())

    # argument tuples prepared once: the timed loop is C calls only
    calls_sel = [(h, l % L_phys, vp(xs[l]), T, vp(alpha_dev), ctypes.byref(params), None, vp(outs[l]), None, None,
                  None, vp(stats[l]), sp) for l in range(L)]
    calls_nat = [(h, l % L_phys, vp(xs[l]), T, None, None, vp(full), vp(outs[l]), None, None, None, vp(stats[l]), sp)
                 for l in range(L)]

    def step(calls):
        for a in calls:
            rc = lib.acm_moe_verify(*a)
            if rc:
                raise acm.AcmError(rc, "acm_moe_verify")

    # Every `period`-th launch of the FFN kernel is bracketed by events (a bracketed launch cannot
    # overlap its set-up with the kernel before it, so bracketing all of them would slow the step it
    # measures).  The period is coprime with the layer count: over the steps every layer is sampled.
    period = 1
    if not resident:
        period = max(args.bracket_every, 1)
        while math.gcd(period, L) != 1:
            period += 1
    bracket = args.bracket_every > 0

    def sampled_layers(steps):
        return np.arange(0, steps * L, period) % L

    def timed(calls, steps, warmup, with_roofline):
        for _ in range(warmup):
            step(calls)
        barrier()
        if with_roofline and bracket:
            ctx.ffn_timing(period, steps * L * 2)
        n0 = ctx.launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            step(calls)
        e1.record(stream)
        barrier()
        ms = e0.elapsed_time(e1)
        launches = ctx.launch_count() - n0
        ffn_ms, ffn_n = (ctx.ffn_time_ms() if with_roofline and bracket else (0.0, 0))
        ctx.ffn_timing(False)
        if world > 1:
            ms, _ = aggregate_over_ranks(ms, float(L * steps), dist, dev)
        return ms, launches, ffn_ms, ffn_n

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms, launches, ffn_ms, ffn_n = timed(calls_sel, args.steps, max(args.warmup, 3), True)
    clocks = sampler.stop() if rank == 0 else None
    ctx.check_device_status()
    st = stats.cpu().numpy()
    n_act = st[:, 4].astype(float)
    # MXFP4: half a byte per weight plus one scale byte per 32
    expert_bytes = 3 * H * cfg.inter * (0.5 + 1.0 / 32.0) if args.mxfp4 else cfg.expert_bytes
    # algorithmic bytes of one FFN launch: the activated experts' weights (+ shared), x in, y out
    alg_bytes = (n_act + cfg.n_shared) * expert_bytes + T * H * 2 + T * H * 4
    alg_per_launch = float(alg_bytes[sampled_layers(args.steps)].mean()) if not resident else float(alg_bytes.mean())
    value = world * L * args.steps / (ms * 1e-3)

    nat = None
    if not args.no_natural:
        ms_n, _, ffn_ms_n, ffn_n_n = timed(calls_nat, args.steps, 3, True)
        st_n = stats.cpu().numpy()
        nat_bytes = (st_n[:, 4].astype(float) + cfg.n_shared) * expert_bytes + T * H * 6
        nat_bytes = float(nat_bytes[sampled_layers(args.steps)].mean()) if not resident else float(nat_bytes.mean())
        nat = {"value": world * L * args.steps / (ms_n * 1e-3), "unit": UNIT, "ms_per_step": ms_n / args.steps,
               "mean_activated_experts": float(st_n[:, 4].mean()),
               "ffn_us_per_launch": 1e3 * ffn_ms_n / max(ffn_n_n, 1),
               "ffn_gbs": nat_bytes / (1e6 * ffn_ms_n / max(ffn_n_n, 1)) if ffn_n_n else None}

    e2e = None
    if not args.no_e2e:
        # the same blocks through the library's host-buffer call: pinned x and alpha in, pinned y out, the
        # copies (the library's own, on its copy streams) inside the timed region
        xs_host = xs.cpu().pin_memory()
        alpha_host = alpha.pin_memory()
        outs_host = torch.zeros(L, T, H, dtype=torch.float32).pin_memory()
        calls_host = [(h, l % L_phys, vp(xs_host[l]), T, vp(alpha_host), ctypes.byref(params), vp(outs_host[l]), None, sp)
                      for l in range(L)]

        def e2e_step():
            for a in calls_host:
                rc = lib.acm_moe_verify_host(*a)
                if rc:
                    raise acm.AcmError(rc, "acm_moe_verify_host")
            ctx.host_synchronize()    # the step's result is on the host

        for _ in range(2):
            e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            e2e_step()
        barrier()
        dt = time.perf_counter() - t0
        if world > 1:
            dt, _ = aggregate_over_ranks(dt, float(L * args.steps), dist, dev)
        e2e = {"value": world * L * args.steps / dt, "unit": UNIT,
               "h2d_bytes_per_step": L * (T * H * cfg.elt_bytes + T * 4), "d2h_bytes_per_step": L * T * H * 4}

    # Per-stage device times (an instrumented pass after the timed ones): the kernels stamp a global clock,
    # the launch sequence and its overlaps stay as they are.  One sample per layer, each taken with that
    # layer as the last call of a pass over the whole stack (so it runs behind its usual predecessor).
    stage_us = pipeline_gbs = None
    if rank == 0 and not resident and cfg.dtype == "bf16":
        ctx.stage_timing(True)
        acc = {}
        n_samples = min(L, 16)
        for j in np.linspace(0, L - 1, n_samples).astype(int):
            order = list(range(j + 1, L)) + list(range(0, j + 1))
            for _ in range(2):
                for l in order:
                    rc = lib.acm_moe_verify(*calls_sel[l])
                    if rc:
                        raise acm.AcmError(rc, "acm_moe_verify")
            times = ctx.stage_times()
            for key, v in times.items():
                acc[key] = acc.get(key, 0.0) + v / n_samples
            # the FFN kernel's rate inside the live pipeline: this layer's algorithmic bytes over its stamped span
            n_act_j = float(n_act[j]) + cfg.n_shared
            acc["_gbs"] = acc.get("_gbs", 0.0) + (n_act_j * expert_bytes + T * H * 6) / (times["ffn"] * 1e3) / n_samples
        ctx.stage_timing(False)
        pipeline_gbs = acc.pop("_gbs")
        stage_us = {key: round(v, 2) for key, v in acc.items()}
        stage_us["note"] = ("in-kernel stamps, mean over %d layers: router = dependency release of the logits kernel to "
                            "the start of the selection kernel; select = softmax, natural top-k and selection; route; "
                            "ffn = first role start to last tile (it starts on the anchor experts while the selection "
                            "runs); whole = start of router to end of ffn" % n_samples)

    if rank != 0:
        return
    peak, peak_kind = read_peaks()
    ffn_us = 1e3 * ffn_ms / max(ffn_n, 1)
    achieved = alg_per_launch / (ffn_us * 1e-6) / 1e9 if ffn_n else None
    # DRAM bytes (read + write) of k_ffn_bf16 per activated expert, from the ncu capture summarised in
    # profiles/k_ffn_bf16_c3_layer.txt (4-layer case; traffic is proportional to the activated experts)
    per_expert = None if args.mxfp4 else DRAM_BYTES_PER_ACTIVATED_EXPERT.get(cfg.index)
    traffic = per_expert * (alg_per_launch - T * H * 6) / expert_bytes if per_expert else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": f"C{cfg.index} {cfg.name}-shaped stack{' with Zipf(1.1) router bias' if args.zipf else ''}{', MXFP4 expert weights' if args.mxfp4 else ''}, {selector_name}",
                   "hidden": H, "n_experts": E, "top_k": k, "inter": cfg.inter, "n_shared": cfg.n_shared,
                   "n_nodes": T, "layers": L, "physical_layers": L_phys,
                   "l2": f"inputs larger than L2: {L_phys} distinct layers, "
                         f"{alg_per_launch * L_phys / 1e9:.1f} GB of expert weights streamed per step",
                   "overlap": args.overlap,
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "us_per_layer": 1e3 * ms / (args.steps * L),
        "mean_eligible": float(st[:, 3].mean()), "mean_activated": float(n_act.mean()),
        "mean_natural_union": float(st[:, 5].mean()),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": (achieved / peak) if achieved else None, "traffic": traffic,
                     "traffic_kind": "scaled from the ncu capture in profiles/k_ffn_bf16_c3_layer.txt by this run's activated experts" if traffic else None,
                     "peak_kind": peak_kind,
                     "kernel": "k_ffn_mxfp4" if args.mxfp4 else "k_ffn_bf16", "us_per_launch": ffn_us, "launches_timed": ffn_n,
                     "timed_every": period if bracket else None,
                     "algorithmic_bytes_per_launch": alg_per_launch,
                     # context, not the headline: the same kernel inside the live pipeline (in-kernel stamps from its
                     # first role starting to its last tile; its set-up overlaps the kernels before it there)
                     "achieved_in_pipeline": pipeline_gbs,
                     "frac_in_pipeline": (pipeline_gbs / peak) if pipeline_gbs else None},
        "stage_us": stage_us,
        "natural_union_path": nat,
        "e2e": e2e,
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if not args.no_cpu_baseline and not args.mxfp4:      # (the oracle's MXFP4 layer is its bf16 layer on the dequantised weights)
        line["cpu_baseline"] = cpu_baseline(cfg)
    print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def run_offloaded(args):
    """Configuration 5 as stated: per layer a seeded 40 % of the experts is GPU-resident, the others exist only in
    pinned host memory (their device copies are NaN), eligibility is conditioned on residency, and an activated
    expert that is not resident is copied host-to-device inside the call and counted.  Headline: the strict
    resident-plus-anchors rule (residency = 2); beside it the budgeted pruning of Eq. 7 (residency = 1) and
    natural routing on the same offloaded layers."""
    import ctypes

    import numpy as np
    import torch

    from paper_2608_02989_b200 import acm, workloads as wl
    from paper_2608_02989_b200 import build as acm_build

    acm_build.build_library()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    cfg = wl.CONFIGS[args.config]
    if args.zipf and not cfg.zipf_bias:
        cfg = wl.scaled(cfg, zipf_bias=True)
    L = args.layers or cfg.n_layers
    T, H, E, k = cfg.n_nodes, cfg.hidden, cfg.n_experts, cfg.top_k
    # The stack (454 GB) fits neither the GPU nor a bounded pinned pool: L_phys physical layers carry the weights
    # (device tensors with the non-resident experts poisoned + full pinned host tensors), logical layer l uses
    # physical layer l mod L_phys with its own hidden states.  Pinned host memory is bounded at 32 GB.
    layer_bytes = E * cfg.expert_bytes
    pinned_budget = 32 * 10 ** 9
    L_phys = max(1, min(L, pinned_budget // layer_bytes))
    ctx = acm.Context.for_config(cfg, n_layers=L_phys)
    keep, masks = [], []
    for l in range(L_phys):
        w = wl.layer_weights(cfg, l, dev)
        rmask = wl.resident_mask(cfg, l)
        words = rmask.numpy().view(np.uint32)
        host_gu, host_dn = w["gate_up"].cpu().pin_memory(), w["down"].cpu().pin_memory()
        for e in range(E):
            if not (int(words[e >> 5]) >> (e & 31)) & 1:
                w["gate_up"][e] = float("nan")          # never read: a non-resident expert comes from the host
                w["down"][e] = float("nan")
        ctx.set_layer_weights(l, w["w_router"], w["router_bias"], w["gate_up"], w["down"])
        ctx.set_resident(l, rmask, host_gu, host_dn)
        keep.append((w, host_gu, host_dn))
        masks.append(words)
    xs = torch.stack([wl.hidden_states(cfg, l, dev) for l in range(L)])
    alpha = acm.node_weights(wl.tree_depths(cfg), wl.commitment_table(cfg)).to(dev)
    outs = torch.zeros(L, T, H, dtype=torch.float32, device=dev)
    stats = torch.zeros(L, 12, dtype=torch.int32, device=dev)
    full = torch.full((ctx.words,), -1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    sp = ctypes.c_void_p(stream.cuda_stream)
    lib, h = ctx.lib, ctx.handle

    def vp(t):
        return ctypes.c_void_p(t.data_ptr())

    def run_policy(params, override, steps, warmup):
        pp = ctypes.byref(params) if params is not None else None
        calls = [(h, l % L_phys, vp(xs[l]), T, vp(alpha) if params is not None else None, pp,
                  vp(full) if override else None, vp(outs[l]), None, None, None, vp(stats[l]), sp) for l in range(L)]

        def step():
            for a in calls:
                rc = lib.acm_moe_verify(*a)
                if rc:
                    raise acm.AcmError(rc, "acm_moe_verify")

        for _ in range(warmup):
            step()
        torch.cuda.synchronize()
        ctx.h2d_bytes(reset=True)
        ctx.offload_timing(True, steps * L)
        n0 = ctx.launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        ot = ctx.offload_times()
        ctx.offload_timing(False)
        ctx.check_device_status()
        st = stats.cpu().numpy()
        n = steps * L
        h2d = ctx.h2d_bytes()
        # HBM bytes of the expert FFN per layer-block: every activated expert's weights once, wherever they came from
        ffn_bytes = float(st[:, 4].mean()) * cfg.expert_bytes
        return {"layer_blocks_per_s": n / (ms * 1e-3), "us_per_layer": 1e3 * ms / n, "steps": steps,
                "mean_eligible_before_pruning": float(st[:, 2].mean()), "mean_eligible": float(st[:, 3].mean()),
                "mean_activated": float(st[:, 4].mean()), "mean_loaded": float(st[:, 8].mean()),
                "h2d_mib_per_layer_block": h2d / 2 ** 20 / n, "h2d_bytes_per_step": h2d / steps,
                "h2d_gbs_while_copying": (h2d / 1e9) / (ot["copy_ms"] * 1e-3) if ot["copy_ms"] > 0 else None,
                "us_per_layer_device": 1e3 * ot["whole_ms"] / max(ot["calls"], 1),
                "us_per_layer_resident_part": 1e3 * ot["resident_ms"] / max(ot["calls"], 1),
                "us_per_layer_h2d_copies": 1e3 * ot["copy_ms"] / max(ot["calls"], 1),
                "us_per_layer_h2d_stall": 1e3 * ot["stall_ms"] / max(ot["calls"], 1),
                "us_per_layer_without_h2d_wait": 1e3 * (ot["whole_ms"] - ot["stall_ms"]) / max(ot["calls"], 1),
                "expert_weight_mb_per_layer_block": ffn_bytes / 1e6,
                "launches": int(ctx.launch_count() - n0)}

    sampler = ClockSampler(0)
    sampler.start()
    head = run_policy(acm.SelectParams(residency=2), False, args.steps, max(args.warmup, 1))
    clocks = sampler.stop()
    res = {"residency_2_resident_plus_anchors": head}
    res["residency_1_eq7_pruning"] = run_policy(acm.SelectParams(residency=1), False, max(1, min(args.steps, 2)), 1)
    if not args.no_natural:
        res["natural_routing_offloaded"] = run_policy(None, True, 1, 1)
    peak, peak_kind = read_peaks()
    line = {
        "metric": METRIC, "value": head["layer_blocks_per_s"], "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 1), "ms_per_step": head["us_per_layer"] * L * 1e-3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": f"C{cfg.index} {cfg.name}-shaped stack as configured: {round(100 * cfg.resident_frac)} % of the "
                               f"experts GPU-resident per layer (seeded), eligibility = (S and resident) plus root anchors, "
                               f"non-resident activated experts copied from pinned host memory inside the call"
                               f"{', Zipf(1.1) router bias' if args.zipf else ''}",
                   "hidden": H, "n_experts": E, "top_k": k, "inter": cfg.inter, "n_nodes": T, "layers": L,
                   "physical_layers": L_phys, "pinned_host_gb": L_phys * layer_bytes / 1e9,
                   "l2": f"inputs larger than L2: every layer-block streams {head['expert_weight_mb_per_layer_block']:.0f} MB "
                         f"of expert weights, {L_phys} distinct physical layers"},
        "us_per_layer": head["us_per_layer"],
        "h2d_bytes_per_step": head["h2d_bytes_per_step"],
        "roofline": {"bound": "hbm", "unit": "GB/s", "peak": peak, "peak_kind": peak_kind,
                     "achieved": head["expert_weight_mb_per_layer_block"] * 1e6 / (head["us_per_layer_without_h2d_wait"] * 1e-6) / 1e9,
                     "frac": head["expert_weight_mb_per_layer_block"] * 1e6 / (head["us_per_layer_without_h2d_wait"] * 1e-6) / 1e9 / peak,
                     "traffic": None,
                     "note": "whole layer-block without its host-to-device stall (all four stages, two FFN launches), "
                             "activated experts' weight bytes over that time; the kernel-level figure is the default run's"},
        "policies": res, "gpu_launches": head["launches"], "clocks": clocks,
    }
    print(json.dumps(line), flush=True)
    ctx.close()


def run_batch(args):
    """Multi-block batches: the configuration's T nodes are B verification blocks (trees of their own).  One
    call per layer verifies them together -- every activated expert is streamed once for all blocks -- and is
    compared with the same blocks verified one call each.  A 'step' is the B blocks through the stacked
    layers; the metric counts blocks, so one batch call of B blocks is B layer-blocks."""
    import ctypes

    import torch

    from paper_2608_02989_b200 import acm, workloads as wl
    from paper_2608_02989_b200 import build as acm_build

    acm_build.build_library()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    cfg = wl.CONFIGS[args.config]
    L, B = args.layers or cfg.n_layers, args.batch
    if args.batch_nodes:
        cfg = wl.scaled(cfg, n_nodes=args.batch_nodes)        # the blocks' nodes together (each block at most 64)
    T, H, E, k = cfg.n_nodes, cfg.hidden, cfg.n_experts, cfg.top_k
    ctx = acm.Context.for_config(cfg, n_layers=L)
    ctx.set_overlap(args.overlap)
    keep = []
    for l in range(L):
        w = wl.layer_weights(cfg, l, dev)
        ctx.set_layer_weights(l, w["w_router"], w["router_bias"], w["gate_up"], w["down"], w["shared_gate_up"],
                              w["shared_down"])
        keep.append(w)
    xs = torch.stack([wl.hidden_states(cfg, l, dev) for l in range(L)])
    offsets, depths = wl.batch_tree_depths(cfg, B)
    p = wl.commitment_table(cfg)
    alpha = torch.cat([acm.node_weights(depths[offsets[b]:offsets[b + 1]], p) for b in range(B)]).to(dev)
    outs = torch.zeros(L, T, H, dtype=torch.float32, device=dev)
    stats = torch.zeros(L, B, 12, dtype=torch.int32, device=dev)
    act = torch.zeros(L, ctx.words, dtype=torch.int32, device=dev)
    params = acm.SelectParams()
    sp = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    lib, h = ctx.lib, ctx.handle
    offs_c = (ctypes.c_int32 * (B + 1))(*offsets)

    def vp(t):
        return ctypes.c_void_p(t.data_ptr())

    calls_batch = [(h, l, vp(xs[l]), B, offs_c, vp(alpha), ctypes.byref(params), vp(outs[l]), None, None, None,
                    vp(act[l]), vp(stats[l]), sp) for l in range(L)]
    calls_single = [(h, l, vp(xs[l][offsets[b]:]), offsets[b + 1] - offsets[b], vp(alpha[offsets[b]:]),
                     ctypes.byref(params), None, vp(outs[l][offsets[b]:]), None, None, None, vp(stats[l][b]), sp)
                    for l in range(L) for b in range(B)]

    def run(fn, calls, name):
        for a in calls:
            rc = fn(*a)
            if rc:
                raise acm.AcmError(rc, name)

    res = {}
    for name, fn, calls in (("batched", lib.acm_moe_verify_batch, calls_batch),
                            ("one_call_per_block", lib.acm_moe_verify, calls_single)):
        for _ in range(max(args.warmup, 3)):
            run(fn, calls, name)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            run(fn, calls, name)
        e1.record()
        torch.cuda.synchronize()
        ctx.check_device_status()
        ms = e0.elapsed_time(e1) / args.steps
        streamed = float(stats[:, :, 4].sum().item()) if name == "one_call_per_block" else \
            float(sum(bin(int(v) & 0xffffffff).count("1") for v in act.flatten().tolist()))
        res[name] = {"layer_blocks_per_s": B * L / (ms * 1e-3), "ms_per_step": ms,
                     "us_per_layer": ms * 1e3 / L, "experts_streamed_per_layer": streamed / L,
                     "expert_weight_mb_per_block_per_layer": streamed / L * cfg.expert_bytes / 1e6 / B}
    line = {"metric": METRIC, "value": res["batched"]["layer_blocks_per_s"], "unit": UNIT, "n_gpus": 1,
            "steps": args.steps, "warmup": max(args.warmup, 3), "higher_is_better": True, "dtype": cfg.dtype,
            "data": "synthetic",
            "config": {"workload": f"C{cfg.index} {cfg.name}-shaped stack, {B} verification blocks per call "
                                   f"({T} nodes in all, block sizes {offsets[1]}..{offsets[-1] - offsets[-2]})",
                       "hidden": H, "n_experts": E, "top_k": k, "inter": cfg.inter, "n_nodes": T, "blocks": B,
                       "layers": L, "l2": "inputs larger than L2: distinct layers streamed per step"},
            "variants": res}
    print(json.dumps(line))


def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(relaunch_as_replicas(args.gpus))
    world, rank, local = dist_setup(args)
    if args.pool and args.impl == "acm":
        if rank == 0:
            run_pool(args)
        return
    if args.batch > 1 and args.impl == "acm":
        if rank == 0:
            run_batch(args)
        return
    if args.impl == "acm" and args.config == 5 and not args.all_resident:
        if rank == 0:
            run_offloaded(args)
        return
    if args.impl == "reference":
        run_reference(args, world, rank)
        return
    run_acm(args, world, rank, local)


if __name__ == "__main__":
    main()
