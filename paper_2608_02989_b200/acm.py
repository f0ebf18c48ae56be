"""Python binding of libacm.so (the C ABI in include/acm.h): argument marshalling only.

Every step of the path runs in the library's CUDA kernels; torch supplies device memory and
streams.  There is no CPU fallback: importing works without a GPU (so that the exported
symbols can be checked), but creating a context needs a B200 and a built library.
"""
from __future__ import annotations

import ctypes
from ctypes import POINTER, byref, c_float, c_int, c_int32, c_uint64, c_void_p
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libacm.so"

OK, ERR_INVALID, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT, ERR_NOMEM, ERR_NONFINITE = range(7)
F32, BF16 = 0, 1
W_RENORM_TOPK, W_SOFTMAX_RAW, W_SOFTMAX_MASKED = 0, 1, 2
OVERLAP_NONE, OVERLAP_DEPENDENT, OVERLAP_ELIGIBLE, OVERLAP_ANCHORS = 0, 1, 2, 3
DEMAND_TOPK_MASS, DEMAND_FULL_MASS, DEMAND_VOTES = 0, 1, 2

EXPORTS = [
    "acm_default_select_params", "acm_create", "acm_destroy", "acm_set_layer_weights", "acm_set_layer_weights_mxfp4",
    "acm_node_weights", "acm_router", "acm_select_eligible", "acm_route_restricted",
    "acm_expert_ffn", "acm_moe_verify", "acm_moe_verify_batch", "acm_moe_verify_host", "acm_host_synchronize", "acm_set_resident",
    "acm_set_slot_pool", "acm_pool_stats", "acm_pool_plan",
    "acm_h2d_bytes", "acm_ffn_timing", "acm_ffn_time_ms", "acm_stage_timing", "acm_stage_times", "acm_launch_count", "acm_device_status", "acm_status_string",
    "acm_set_overlap", "acm_set_wait_limit", "acm_wait_report", "acm_inject_unpublished_wait",
    "acm_offload_timing", "acm_offload_times", "acm_ffn_plan",
    "acm_expert_ffn_f32_noalloc",
]
NOALLOC_MAX_FLOATS = 1 << 20


class ModelDesc(ctypes.Structure):
    _fields_ = [("hidden", c_int32), ("n_experts", c_int32), ("top_k", c_int32), ("inter", c_int32),
                ("n_shared", c_int32), ("max_nodes", c_int32), ("n_layers", c_int32), ("dtype", c_int32),
                ("weighting", c_int32), ("routed_scale", c_float)]


class SelectParams(ctypes.Structure):
    """acm_select_params; the defaults are the paper's (Eq. 4-6, anchors on, no residency)."""
    _fields_ = [("demand", c_int32), ("use_anchors", c_int32), ("fixed_budget", c_int32),
                ("ceil_guard", c_float), ("residency", c_int32), ("max_remove", c_int32)]

    def __init__(self, demand=0, use_anchors=1, fixed_budget=0, ceil_guard=2.0 ** -10, residency=0,
                 max_remove=128):
        super().__init__(demand, use_anchors, fixed_budget, ceil_guard, residency, max_remove)


class BlockStats(ctypes.Structure):
    _fields_ = [("n_anchor", c_int32), ("n_er", c_int32), ("n_eligible", c_int32),
                ("n_eligible_pruned", c_int32), ("n_activated", c_int32), ("n_natural_union", c_int32),
                ("displaced_aS", c_int32), ("pruned_m", c_int32), ("n_staged", c_int32),
                ("n_streamed", c_int32), ("reserved", c_int32 * 2)]
    NAMES = ["n_anchor", "n_er", "n_eligible", "n_eligible_pruned", "n_activated", "n_natural_union",
             "displaced_aS", "pruned_m", "n_staged", "n_streamed"]


class AcmError(RuntimeError):
    def __init__(self, code, where):
        self.code = int(code)
        super().__init__(f"{where}: {status_string(code)} (acm_status {int(code)})")


_lib = None


def load_library():
    """dlopen libacm.so (built in-tree by ``paper_2608_02989_b200.build``); fails loudly if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2608_02989_b200.build` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(str(LIB_PATH))
    lib.acm_status_string.restype = ctypes.c_char_p
    lib.acm_status_string.argtypes = [c_int]
    lib.acm_create.argtypes = [POINTER(ModelDesc), POINTER(c_void_p)]
    lib.acm_destroy.argtypes = [c_void_p]
    lib.acm_set_layer_weights.argtypes = [c_void_p, c_int] + [c_void_p] * 6
    lib.acm_set_layer_weights_mxfp4.argtypes = [c_void_p, c_int] + [c_void_p] * 4
    lib.acm_node_weights.argtypes = [c_void_p, c_int, c_void_p, c_int, c_float, c_int, c_void_p]
    lib.acm_router.argtypes = [c_void_p, c_int, c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.acm_select_eligible.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_int,
                                        POINTER(SelectParams), c_void_p, c_void_p, c_void_p, c_void_p,
                                        c_void_p, c_void_p, c_void_p]
    lib.acm_route_restricted.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p]
    lib.acm_expert_ffn.argtypes = [c_void_p, c_int, c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.acm_moe_verify.argtypes = [c_void_p, c_int, c_void_p, c_int, c_void_p, POINTER(SelectParams),
                                   c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.acm_moe_verify_batch.argtypes = [c_void_p, c_int, c_void_p, c_int, c_void_p, c_void_p, POINTER(SelectParams),
                                         c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.acm_moe_verify_host.argtypes = [c_void_p, c_int, c_void_p, c_int, c_void_p, POINTER(SelectParams),
                                        c_void_p, c_void_p, c_void_p]
    lib.acm_host_synchronize.argtypes = [c_void_p]
    lib.acm_set_resident.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p]
    lib.acm_set_slot_pool.argtypes = [c_void_p, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int]
    lib.acm_pool_stats.argtypes = [c_void_p, c_int, POINTER(c_uint64), POINTER(c_uint64), POINTER(c_uint64),
                                   c_void_p, c_int]
    lib.acm_pool_plan.argtypes = [c_int, c_int, c_void_p, c_void_p, POINTER(c_uint64), c_void_p, c_void_p, c_void_p,
                                  c_void_p, POINTER(c_int32), POINTER(c_int32)]
    lib.acm_h2d_bytes.argtypes = [c_void_p, POINTER(c_uint64), c_int]
    lib.acm_ffn_timing.argtypes = [c_void_p, c_int, c_int]
    lib.acm_stage_timing.argtypes = [c_void_p, c_int]
    lib.acm_stage_times.argtypes = [c_void_p, POINTER(ctypes.c_double)]
    lib.acm_ffn_time_ms.argtypes = [c_void_p, POINTER(c_float), POINTER(c_int32)]
    lib.acm_launch_count.argtypes = [c_void_p, POINTER(c_uint64)]
    lib.acm_device_status.argtypes = [c_void_p, c_void_p]
    lib.acm_set_overlap.argtypes = [c_void_p, c_int]
    lib.acm_ffn_plan.argtypes = [c_int] * 5 + [c_void_p, c_int, POINTER(c_int32), POINTER(c_int32)]
    lib.acm_offload_timing.argtypes = [c_void_p, c_int, c_int]
    lib.acm_offload_times.argtypes = [c_void_p, POINTER(ctypes.c_double), POINTER(c_int32)]
    lib.acm_set_wait_limit.argtypes = [c_void_p, c_uint64]
    lib.acm_wait_report.argtypes = [c_void_p, c_void_p, c_int, POINTER(c_int32)]
    lib.acm_inject_unpublished_wait.argtypes = [c_void_p, c_int, c_void_p, c_int, c_void_p, c_void_p]
    lib.acm_default_select_params.argtypes = [POINTER(SelectParams)]
    lib.acm_expert_ffn_f32_noalloc.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_void_p, c_void_p,
                                               c_void_p, c_void_p, c_void_p, c_void_p]
    _lib = lib
    return lib


def status_string(code) -> str:
    return load_library().acm_status_string(int(code)).decode()


def _check(code, where):
    if code != OK:
        raise AcmError(code, where)


def _p(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return c_void_p(stream.cuda_stream)


def node_weights(depth, p_table, beta=0.5, width_norm=True) -> torch.Tensor:
    """acm_node_weights (Eq. 3) on host tensors -> alpha [T] float32 (host)."""
    depth = depth.to(torch.int32).contiguous().cpu()
    p_table = p_table.to(torch.float32).contiguous().cpu()
    alpha = torch.empty(depth.numel(), dtype=torch.float32)
    _check(load_library().acm_node_weights(_p(depth), depth.numel(), _p(p_table), p_table.numel(),
                                           float(beta), int(bool(width_norm)), _p(alpha)), "acm_node_weights")
    return alpha


def ffn_plan(n_experts_streamed, hidden, inter, grid, n_anchor_first=0):
    """acm_ffn_plan on the host -> (pieces [n, 8] int32 numpy array, number of segments); see include/acm.h."""
    import numpy as np
    cap = 1 << 16
    while True:
        buf = np.zeros((cap, 8), dtype=np.int32)
        n, nseg = c_int32(0), c_int32(0)
        rc = load_library().acm_ffn_plan(n_experts_streamed, n_anchor_first, hidden, inter, grid,
                                         buf.ctypes.data_as(c_void_p), cap, byref(n), byref(nseg))
        if rc == ERR_NOMEM:
            cap = n.value
            continue
        _check(rc, "acm_ffn_plan")
        return buf[: n.value], nseg.value


def pool_plan(n_experts, slot_expert, last_use, tick, activated):
    """acm_pool_plan on host data: slot_expert / last_use are lists (updated copies are returned), `activated`
    a set of expert ids.  Returns (slot_expert, last_use, tick, loads [(expert, slot, wave)], n_hits)."""
    import numpy as np
    n_slots = len(slot_expert)
    se = np.asarray(slot_expert, dtype=np.int32).copy()
    lu = np.asarray(last_use, dtype=np.uint64).copy()
    words = (n_experts + 31) // 32
    mask = np.zeros(words, dtype=np.uint32)
    for e in activated:
        mask[e // 32] |= np.uint32(1 << (e % 32))
    le, ls, lw = (np.zeros(n_experts, dtype=np.int32) for _ in range(3))
    t, n_loads, n_hits = c_uint64(int(tick)), c_int32(0), c_int32(0)
    vp = lambda a: a.ctypes.data_as(c_void_p)
    _check(load_library().acm_pool_plan(n_experts, n_slots, vp(se), vp(lu), byref(t), vp(mask), vp(le), vp(ls), vp(lw),
                                        byref(n_loads), byref(n_hits)), "acm_pool_plan")
    n = n_loads.value
    return se.tolist(), lu.tolist(), t.value, list(zip(le[:n].tolist(), ls[:n].tolist(), lw[:n].tolist())), n_hits.value


# ---- MXFP4 expert weights: the library's tiled layout ------------------------------------------------
# The FFN kernel fetches one pipeline stage of an MXFP4 weight tile -- 128 rows x 128 K -- with a single
# contiguous copy, so the weights are stored tile by tile: per (expert, tile, stage) 8704 bytes =
#   128 rows x 64 bytes of codes, then 128 rows x 4 scale bytes (one E8M0 byte per 32 K).
# Inside each group of 8 consecutive K elements the codes sit in one 32-bit word with the even elements in
# the low half and the odd ones in the high half (nibble j = element 2j, nibble 4+j = element 2j+1), which
# is the order the kernel's expansion to bf16 pairs wants; the four 16-byte pieces of a row (32 K each) are
# stored rotated by the row number (piece p of row r at position p ^ ((r >> 1) & 3)).  These functions only
# permute bytes.
MX_STAGE_BYTES = 128 * 64 + 128 * 4


def _mx_words(codes):
    """codes [..., rows, 128] (4-bit values in uint8) -> [..., rows, 64] bytes in the word order above."""
    c = codes.to(torch.int32).reshape(*codes.shape[:-1], 16, 4, 2)        # [group of 8][pair j][even, odd]
    even, odd = c[..., 0], c[..., 1]                                           # [..., 16, 4]
    lo = even[..., 0] | (even[..., 1] << 4) | (even[..., 2] << 8) | (even[..., 3] << 12)
    hi = odd[..., 0] | (odd[..., 1] << 4) | (odd[..., 2] << 8) | (odd[..., 3] << 12)
    b = torch.stack([lo & 0xff, lo >> 8, hi & 0xff, hi >> 8], dim=-1)          # little-endian bytes of the word
    b = b.to(torch.uint8).reshape(*codes.shape[:-1], 4, 16)                    # the row's four 16-byte pieces (32 K each)
    # piece p of row r is stored at position p ^ ((r >> 1) & 3): a warp reading one piece per row then touches
    # every shared-memory bank once
    rows = codes.shape[-2]
    pos = torch.arange(4, device=codes.device)[None, :] ^ ((torch.arange(rows, device=codes.device)[:, None] >> 1) & 3)
    out = torch.empty_like(b)
    out.scatter_(-2, pos[..., None].expand(*b.shape[:-3], rows, 4, 16).contiguous(), b)
    return out.reshape(*codes.shape[:-1], 64)


def pack_mxfp4_gate_up(codes, scales):
    """codes [E, 2I, H], scales [E, 2I, H/32] (uint8; rows 0..I-1 gate, I..2I-1 up) ->
    uint8 [E, I/64, H/128, 8704]: tile t = gate rows 64t..64t+63 followed by the matching up rows."""
    E, R, H = codes.shape
    I = R // 2
    if I % 64 or H % 128:
        raise ValueError("MXFP4 layers need inter % 64 == 0 and hidden % 128 == 0")
    c = codes.reshape(E, 2, I // 64, 64, H // 128, 128).permute(0, 2, 4, 1, 3, 5)      # [E, tile, stage, g|u, 64, 128]
    c = _mx_words(c.reshape(E, I // 64, H // 128, 128, 128)).reshape(E, I // 64, H // 128, 128 * 64)
    s = scales.reshape(E, 2, I // 64, 64, H // 128, 4).permute(0, 2, 4, 1, 3, 5).reshape(E, I // 64, H // 128, 512)
    return torch.cat([c, s], dim=-1).contiguous()


def pack_mxfp4_down(codes, scales):
    """codes [E, H, I], scales [E, H, I/32] (uint8) -> uint8 [E, H/128, I/128, 8704]."""
    E, H, I = codes.shape
    if H % 128 or I % 128:
        raise ValueError("MXFP4 layers need hidden % 128 == 0 and inter % 128 == 0")
    c = codes.reshape(E, H // 128, 128, I // 128, 128).permute(0, 1, 3, 2, 4)          # [E, tile, stage, 128 rows, 128]
    c = _mx_words(c).reshape(E, H // 128, I // 128, 128 * 64)
    s = scales.reshape(E, H // 128, 128, I // 128, 4).permute(0, 1, 3, 2, 4).reshape(E, H // 128, I // 128, 512)
    return torch.cat([c, s], dim=-1).contiguous()


def expert_ffn_f32_noalloc(x, idx, w, gate_up, down, out, stream=None):
    """acm_expert_ffn_f32_noalloc: the fp32 expert FFN for callers that may not allocate device memory at
    call time.  Every tensor, `out` included, is the caller's; nothing is allocated here or in the library
    (its scratch is a fixed array in the library image, shared by all calls: do not overlap calls)."""
    for name, t, dt in (("x", x, torch.float32), ("idx", idx, torch.int32), ("w", w, torch.float32),
                        ("gate_up", gate_up, torch.float32), ("down", down, torch.float32), ("out", out, torch.float32)):
        if t.dtype != dt:
            raise TypeError(f"{name} must be {dt}, got {t.dtype}")
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous CUDA tensor")
    T, H = x.shape
    E, _, I = down.shape
    k = idx.shape[1]
    if tuple(gate_up.shape) != (E, 2 * I, H) or tuple(idx.shape) != (T, k) or tuple(w.shape) != (T, k) or \
            tuple(out.shape) != (T, H):
        raise ValueError("shapes: x [T,H], idx/w [T,k], gate_up [E,2I,H], down [E,H,I], out [T,H]")
    _check(load_library().acm_expert_ffn_f32_noalloc(_p(x), T, H, I, E, k, _p(idx), _p(w), _p(gate_up), _p(down),
                                                     _p(out), _stream(stream)), "acm_expert_ffn_f32_noalloc")
    return out


class Context:
    """Owns one acm_ctx.  Methods mirror the C entry points and take torch CUDA tensors."""

    def __init__(self, hidden, n_experts, top_k, inter, n_shared=0, max_nodes=64, n_layers=1, dtype=BF16,
                 weighting=W_RENORM_TOPK, routed_scale=1.0):
        self.lib = load_library()
        self.desc = ModelDesc(hidden, n_experts, top_k, inter, n_shared, max_nodes, n_layers, dtype, weighting,
                              routed_scale)
        self.handle = c_void_p()
        _check(self.lib.acm_create(byref(self.desc), byref(self.handle)), "acm_create")
        self._keep = {}
        self.E, self.k, self.H, self.I = n_experts, top_k, hidden, inter
        self.words = (n_experts + 31) // 32

    @classmethod
    def for_config(cls, cfg, n_layers=None, max_nodes=64):
        return cls(cfg.hidden, cfg.n_experts, cfg.top_k, cfg.inter, cfg.n_shared, max_nodes,
                   n_layers or cfg.n_layers, F32 if cfg.dtype == "f32" else BF16, cfg.weighting, 1.0)

    def close(self):
        if self.handle:
            self.lib.acm_destroy(self.handle)
            self.handle = c_void_p()
            self._keep.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ set-up
    def set_layer_weights(self, layer, w_router, router_bias, gate_up, down, shared_gate_up=None, shared_down=None):
        self._keep[("w", layer)] = (w_router, router_bias, gate_up, down, shared_gate_up, shared_down)
        _check(self.lib.acm_set_layer_weights(self.handle, layer, _p(w_router), _p(router_bias), _p(gate_up),
                                              _p(down), _p(shared_gate_up), _p(shared_down)),
               "acm_set_layer_weights")

    def set_layer_weights_mxfp4(self, layer, w_router, router_bias, gate_up_tiles, down_tiles):
        """Routed experts in MXFP4, in the library's tiled layout (pack_mxfp4_gate_up / pack_mxfp4_down), on the device."""
        self._keep[("w", layer)] = (w_router, router_bias, gate_up_tiles, down_tiles)
        _check(self.lib.acm_set_layer_weights_mxfp4(self.handle, layer, _p(w_router), _p(router_bias), _p(gate_up_tiles),
                                                    _p(down_tiles)), "acm_set_layer_weights_mxfp4")

    def set_resident(self, layer, resident_mask, host_gate_up, host_down):
        """resident_mask: host int32/uint32 words (or None to clear); host_*: pinned host tensors."""
        if resident_mask is None:
            _check(self.lib.acm_set_resident(self.handle, layer, None, None, None), "acm_set_resident")
            self._keep.pop(("r", layer), None)
            return
        m = resident_mask.contiguous().cpu()
        self._keep[("r", layer)] = (m, host_gate_up, host_down)
        _check(self.lib.acm_set_resident(self.handle, layer, _p(m), _p(host_gate_up), _p(host_down)),
               "acm_set_resident")

    def set_slot_pool(self, layer, pool_gate_up, pool_down, host_gate_up, host_down, initial_experts=()):
        """LRU expert pool: pool_* device tensors [n_slots, ...], host_* pinned tensors [E, ...]."""
        init = torch.tensor(list(initial_experts), dtype=torch.int32)
        self._keep[("p", layer)] = (pool_gate_up, pool_down, host_gate_up, host_down)
        _check(self.lib.acm_set_slot_pool(self.handle, layer, pool_gate_up.shape[0], _p(pool_gate_up), _p(pool_down),
                                          _p(host_gate_up), _p(host_down), _p(init) if init.numel() else None,
                                          init.numel()), "acm_set_slot_pool")

    def pool_stats(self, layer, reset=False):
        """-> dict(hits, misses, h2d_bytes, slot_expert [n_slots] list)."""
        h, m, b = c_uint64(0), c_uint64(0), c_uint64(0)
        n_slots = self._keep[("p", layer)][0].shape[0]
        slots = torch.full((n_slots,), -2, dtype=torch.int32)
        _check(self.lib.acm_pool_stats(self.handle, layer, byref(h), byref(m), byref(b), _p(slots), int(reset)),
               "acm_pool_stats")
        return {"hits": h.value, "misses": m.value, "h2d_bytes": b.value, "slot_expert": slots.tolist()}

    # ------------------------------------------------------------------ stages
    def router(self, layer, x, stream=None, want_probs=True, want_topk=True):
        T = x.shape[0]
        dev = x.device
        logits = torch.empty(T, self.E, dtype=torch.float32, device=dev)
        probs = torch.empty(T, self.E, dtype=torch.float32, device=dev) if want_probs else None
        nat = torch.empty(T, self.k, dtype=torch.int32, device=dev) if want_topk else None
        _check(self.lib.acm_router(self.handle, layer, _p(x), T, _p(logits), _p(probs), _p(nat), _stream(stream)),
               "acm_router")
        return logits, probs, nat

    def select_eligible(self, probs, nat_idx, alpha, params=None, anchor_nodes=None, resident_mask=None,
                        stream=None):
        T = probs.shape[0]
        dev = probs.device
        params = params or SelectParams()
        mask = torch.zeros(self.words, dtype=torch.int32, device=dev)
        unpruned = torch.zeros(self.words, dtype=torch.int32, device=dev)
        count = torch.zeros(1, dtype=torch.int32, device=dev)
        demand = torch.zeros(self.E, dtype=torch.float32, device=dev)
        stats = torch.zeros(12, dtype=torch.int32, device=dev)
        n_anchor = 0 if anchor_nodes is None else anchor_nodes.numel()
        _check(self.lib.acm_select_eligible(self.handle, _p(probs), _p(nat_idx), T, _p(alpha), _p(anchor_nodes),
                                            n_anchor, byref(params), _p(resident_mask), _p(mask), _p(count),
                                            _p(demand), _p(unpruned), _p(stats), _stream(stream)),
               "acm_select_eligible")
        return {"mask": mask, "unpruned_mask": unpruned, "count": count, "demand": demand, "stats": stats}

    def route_restricted(self, logits, mask, stream=None):
        T = logits.shape[0]
        idx = torch.empty(T, self.k, dtype=torch.int32, device=logits.device)
        w = torch.empty(T, self.k, dtype=torch.float32, device=logits.device)
        _check(self.lib.acm_route_restricted(self.handle, _p(logits), _p(mask), T, _p(idx), _p(w), _stream(stream)),
               "acm_route_restricted")
        return idx, w

    def expert_ffn(self, layer, x, idx, w, out=None, stream=None):
        T = x.shape[0]
        if out is None:
            out = torch.empty(T, self.H, dtype=torch.float32, device=x.device)
        _check(self.lib.acm_expert_ffn(self.handle, layer, _p(x), T, _p(idx), _p(w), _p(out), _stream(stream)),
               "acm_expert_ffn")
        return out

    def moe_verify(self, layer, x, alpha, params=None, mask_override=None, out=None, want=False, stream=None):
        """Stages 1-4.  want=True also returns idx, w, mask and stats (device tensors)."""
        T = x.shape[0]
        dev = x.device
        if out is None:
            out = torch.empty(T, self.H, dtype=torch.float32, device=dev)
        if params is None and mask_override is None:
            params = SelectParams()
        idx = w = mask = stats = None
        if want:
            idx = torch.empty(T, self.k, dtype=torch.int32, device=dev)
            w = torch.empty(T, self.k, dtype=torch.float32, device=dev)
            mask = torch.zeros(self.words, dtype=torch.int32, device=dev)
            stats = torch.zeros(12, dtype=torch.int32, device=dev)
        _check(self.lib.acm_moe_verify(self.handle, layer, _p(x), T, _p(alpha),
                                       byref(params) if params is not None else None, _p(mask_override), _p(out),
                                       _p(idx), _p(w), _p(mask), _p(stats), _stream(stream)), "acm_moe_verify")
        if want:
            return out, idx, w, mask, stats
        return out

    def moe_verify_batch(self, layer, x, block_offsets, alpha, params=None, out=None, want=False, stream=None):
        """Stages 1-4 for several blocks stacked along the node axis (block b = rows block_offsets[b] ..
        block_offsets[b+1]-1).  want=True also returns idx, w, the blocks' masks [n_blocks, words], the
        union of activated experts [words] and the blocks' stats [n_blocks, 12]."""
        T = x.shape[0]
        dev = x.device
        offs = (c_int32 * len(block_offsets))(*[int(v) for v in block_offsets])
        nb = len(block_offsets) - 1
        if out is None:
            out = torch.empty(T, self.H, dtype=torch.float32, device=dev)
        params = params or SelectParams()
        idx = w = mask = act = stats = None
        if want:
            idx = torch.empty(T, self.k, dtype=torch.int32, device=dev)
            w = torch.empty(T, self.k, dtype=torch.float32, device=dev)
            mask = torch.zeros(max(nb, 1), self.words, dtype=torch.int32, device=dev)
            act = torch.zeros(self.words, dtype=torch.int32, device=dev)
            stats = torch.zeros(max(nb, 1), 12, dtype=torch.int32, device=dev)
        _check(self.lib.acm_moe_verify_batch(self.handle, layer, _p(x), nb, offs, _p(alpha), byref(params), _p(out),
                                             _p(idx), _p(w), _p(mask), _p(act), _p(stats), _stream(stream)),
               "acm_moe_verify_batch")
        if want:
            return out, idx, w, mask, act, stats
        return out

    def moe_verify_host(self, layer, x_host, alpha_host, out_host, params=None, stats_host=None, stream=None):
        """Stages 1-4 on PINNED host tensors (x, alpha in; out, optional stats [12] int32 out).  Asynchronous:
        call host_synchronize() before reading out_host."""
        for t in (x_host, alpha_host, out_host):
            if t.is_cuda or not t.is_pinned():
                raise ValueError("moe_verify_host takes pinned host tensors")
        params = params or SelectParams()
        _check(self.lib.acm_moe_verify_host(self.handle, layer, _p(x_host), x_host.shape[0], _p(alpha_host),
                                            byref(params), _p(out_host), _p(stats_host), _stream(stream)),
               "acm_moe_verify_host")

    def host_synchronize(self):
        _check(self.lib.acm_host_synchronize(self.handle), "acm_host_synchronize")

    # ------------------------------------------------------------------ bookkeeping
    def h2d_bytes(self, reset=False) -> int:
        v = c_uint64(0)
        _check(self.lib.acm_h2d_bytes(self.handle, byref(v), int(reset)), "acm_h2d_bytes")
        return v.value

    def ffn_timing(self, enable, capacity=0):
        _check(self.lib.acm_ffn_timing(self.handle, int(enable), int(capacity)), "acm_ffn_timing")

    def ffn_time_ms(self):
        ms, n = c_float(0), c_int32(0)
        _check(self.lib.acm_ffn_time_ms(self.handle, byref(ms), byref(n)), "acm_ffn_time_ms")
        return ms.value, n.value

    def offload_timing(self, enable, capacity=0):
        _check(self.lib.acm_offload_timing(self.handle, int(bool(enable)), int(capacity)), "acm_offload_timing")

    def offload_times(self) -> dict:
        """Sums over the recorded calls (ms): whole, resident part, copies, stall; and the number of calls."""
        ms = (ctypes.c_double * 4)()
        n = c_int32(0)
        _check(self.lib.acm_offload_times(self.handle, ms, byref(n)), "acm_offload_times")
        return {"whole_ms": ms[0], "resident_ms": ms[1], "copy_ms": ms[2], "stall_ms": ms[3], "calls": n.value}

    def stage_timing(self, enable):
        _check(self.lib.acm_stage_timing(self.handle, int(bool(enable))), "acm_stage_timing")

    def stage_times(self) -> dict:
        """Device microseconds of the last fused call's stages (they overlap; see acm_stage_times)."""
        us = (ctypes.c_double * 5)()
        _check(self.lib.acm_stage_times(self.handle, us), "acm_stage_times")
        return dict(zip(("router", "select", "route", "ffn", "whole"), [float(v) for v in us]))

    def launch_count(self) -> int:
        v = c_uint64(0)
        _check(self.lib.acm_launch_count(self.handle, byref(v)), "acm_launch_count")
        return v.value

    def set_overlap(self, level):
        """acm_set_overlap: OVERLAP_NONE (safe on a shared GPU) .. OVERLAP_ANCHORS (default)."""
        _check(self.lib.acm_set_overlap(self.handle, int(level)), "acm_set_overlap")

    def set_wait_limit(self, nanoseconds):
        _check(self.lib.acm_set_wait_limit(self.handle, int(nanoseconds)), "acm_set_wait_limit")

    def wait_report(self) -> list:
        """Per CTA of the last expert-FFN launch: 0 = no wait ran out, -1 = never started, else the wait site."""
        buf = (c_int32 * 256)()
        n = c_int32(0)
        _check(self.lib.acm_wait_report(self.handle, buf, 256, byref(n)), "acm_wait_report")
        return [int(buf[i]) for i in range(min(n.value, 256))]

    def inject_unpublished_wait(self, layer, x, out=None, stream=None):
        """acm_inject_unpublished_wait: the FFN kernel waits for an eligible set nobody publishes (error-path tests)."""
        T = x.shape[0]
        if out is None:
            out = torch.empty(T, self.H, dtype=torch.float32, device=x.device)
        _check(self.lib.acm_inject_unpublished_wait(self.handle, layer, _p(x), T, _p(out), _stream(stream)),
               "acm_inject_unpublished_wait")
        return out

    def device_status(self, stream=None) -> int:
        return int(self.lib.acm_device_status(self.handle, _stream(stream)))

    def check_device_status(self, stream=None):
        _check(self.device_status(stream), "device status")


def stats_dict(stats_tensor) -> dict:
    v = stats_tensor.cpu().tolist()
    return dict(zip(BlockStats.NAMES, v))
