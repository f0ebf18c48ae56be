"""ctypes/numpy wrapper of the C++ oracle (test infrastructure; see acm_oracle.cpp).

Matrices are numpy arrays: float32 for the fp32 configuration, uint16 holding
bfloat16 bit patterns for the bf16 ones (torch CPU tensors are converted).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "acm_oracle.cpp"
_LIB = _HERE / "liboracle_acm.so"
_lib = None

CXXFLAGS = ["-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-mfma", "-fopenmp",
            "-shared", "-fPIC"]


class SelectParams(ctypes.Structure):
    """Selector switches; defaults are the paper's (Eq. 4-6, no residency)."""
    _fields_ = [("demand", ctypes.c_int32), ("use_anchors", ctypes.c_int32),
                ("fixed_budget", ctypes.c_int32), ("ceil_guard", ctypes.c_float),
                ("residency", ctypes.c_int32), ("max_remove", ctypes.c_int32)]

    def __init__(self, demand=0, use_anchors=1, fixed_budget=0, ceil_guard=2.0 ** -10,
                 residency=0, max_remove=128):
        super().__init__(demand, use_anchors, fixed_budget, ceil_guard, residency, max_remove)


class SelectStats(ctypes.Structure):
    _fields_ = [("n_anchor", ctypes.c_int32), ("n_er", ctypes.c_int32),
                ("n_eligible", ctypes.c_int32), ("n_eligible_pruned", ctypes.c_int32),
                ("n_natural_union", ctypes.c_int32), ("displaced_aS", ctypes.c_int32),
                ("pruned_m", ctypes.c_int32), ("residual_mass", ctypes.c_float),
                ("entropy", ctypes.c_float), ("perplexity", ctypes.c_float)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


def build(force: bool = False) -> Path:
    """Compile the oracle shared library with g++ (no-op when up to date)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(["g++", *CXXFLAGS, str(_SRC), "-o", str(tmp)], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _lib.orc_expf.restype = ctypes.c_float
        _lib.orc_expf.argtypes = [ctypes.c_float]
        _lib.orc_logf.restype = ctypes.c_float
        _lib.orc_logf.argtypes = [ctypes.c_float]
        _lib.orc_tree_sum.restype = ctypes.c_float
        _lib.orc_route_restricted.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                              ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                              ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p]
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _matrix(a):
    """-> (contiguous numpy array, dtype code).  Accepts numpy f32/u16 or torch f32/bf16 CPU tensors."""
    if a is None:
        return None, None
    if not isinstance(a, np.ndarray):
        import torch
        a = a.detach().cpu().contiguous()
        a = a.view(torch.int16).numpy().view(np.uint16) if a.dtype == torch.bfloat16 else a.numpy()
    a = np.ascontiguousarray(a)
    if a.dtype == np.float32:
        return a, 0
    if a.dtype == np.uint16:
        return a, 1
    raise TypeError(f"oracle matrices are float32 or bf16 bits (uint16), got {a.dtype}")


def _np(a):
    if hasattr(a, "detach"):
        return a.detach().cpu().numpy()
    return np.asarray(a)


def _f32(a):
    if a is None:
        return None
    return np.ascontiguousarray(_np(a), dtype=np.float32)


def _i32(a):
    if a is None:
        return None
    return np.ascontiguousarray(_np(a), dtype=np.int32)


def _u32(a):
    if a is None:
        return None
    a = _np(a)
    return np.ascontiguousarray(a).view(np.uint32) if a.dtype == np.int32 else np.ascontiguousarray(a, dtype=np.uint32)


def expf(x):
    x = _f32(np.atleast_1d(x))
    y = np.empty_like(x)
    _load().orc_expf_array(_ptr(x), _ptr(y), ctypes.c_int64(x.size))
    return y


def logf(x):
    x = _f32(np.atleast_1d(x))
    y = np.empty_like(x)
    _load().orc_logf_array(_ptr(x), _ptr(y), ctypes.c_int64(x.size))
    return y


def tree_sum(v):
    v = _f32(v)
    return float(_load().orc_tree_sum(_ptr(v), ctypes.c_int(v.size)))


def node_weights(depth, p_table, beta=0.5, width_norm=True):
    """Eq. 3 -> alpha [T] float32."""
    depth = _i32(depth)
    p_table = _f32(p_table)
    alpha = np.empty(depth.size, dtype=np.float32)
    rc = _load().orc_node_weights(_ptr(depth), depth.size, _ptr(p_table), p_table.size,
                                  ctypes.c_float(beta), int(bool(width_norm)), _ptr(alpha))
    if rc:
        raise ValueError("depth outside the commitment table")
    return alpha


def router(x, w_router, bias, k):
    """-> logits [T,E] f32, probs [T,E] f32, nat_idx [T,k] i32."""
    x, dt = _matrix(x)
    w_router, dt2 = _matrix(w_router)
    assert dt == dt2
    T, H = x.shape
    E = w_router.shape[0]
    bias = _f32(bias)
    logits = np.empty((T, E), dtype=np.float32)
    probs = np.empty((T, E), dtype=np.float32)
    nat = np.empty((T, k), dtype=np.int32)
    rc = _load().orc_router(_ptr(x), _ptr(w_router), _ptr(bias), T, H, E, k, dt, _ptr(logits),
                            _ptr(probs), _ptr(nat))
    if rc:
        raise ValueError("orc_router: bad arguments")
    return logits, probs, nat


def select_eligible(probs, nat_idx, alpha, params: SelectParams | None = None, anchor_nodes=None,
                    resident_mask=None):
    """-> dict(mask u32[ceil(E/32)], unpruned_mask, count, demand f32[E], stats)."""
    probs = _f32(probs)
    nat_idx = _i32(nat_idx)
    alpha = _f32(alpha)
    T, E = probs.shape
    k = nat_idx.shape[1]
    params = params or SelectParams()
    anchor_nodes = _i32(anchor_nodes)
    resident_mask = _u32(resident_mask)
    words = (E + 31) // 32
    mask = np.zeros(words, dtype=np.uint32)
    unpruned = np.zeros(words, dtype=np.uint32)
    count = ctypes.c_int32(0)
    demand = np.empty(E, dtype=np.float32)
    stats = SelectStats()
    rc = _load().orc_select_eligible(_ptr(probs), _ptr(nat_idx), T, E, k, _ptr(alpha),
                                     _ptr(anchor_nodes), 0 if anchor_nodes is None else anchor_nodes.size,
                                     ctypes.byref(params), _ptr(resident_mask), _ptr(mask), _ptr(unpruned),
                                     ctypes.byref(count), _ptr(demand), ctypes.byref(stats))
    if rc:
        raise ValueError("orc_select_eligible: bad arguments")
    return {"mask": mask, "unpruned_mask": unpruned, "count": count.value, "demand": demand,
            "stats": stats.as_dict()}


def route_restricted(logits, mask, k, weighting=0, routed_scale=1.0):
    """Eq. 2 -> idx [T,k] i32 (-1 = empty slot), w [T,k] f64."""
    logits = _f32(logits)
    mask = _u32(mask)
    T, E = logits.shape
    idx = np.empty((T, k), dtype=np.int32)
    w = np.empty((T, k), dtype=np.float64)
    rc = _load().orc_route_restricted(_ptr(logits), _ptr(mask), T, E, k, int(weighting),
                                      float(routed_scale), _ptr(idx), _ptr(w))
    if rc:
        raise ValueError("orc_route_restricted: bad arguments")
    return idx, w


def expert_ffn(x, idx, w, gate_up, down, shared_gate_up=None, shared_down=None):
    """SwiGLU experts + weighted combine -> out [T,H] f64."""
    x, dt = _matrix(x)
    gate_up, dt2 = _matrix(gate_up)
    down, dt3 = _matrix(down)
    assert dt == dt2 == dt3
    sgu, _ = _matrix(shared_gate_up)
    sdn, _ = _matrix(shared_down)
    T, H = x.shape
    E, I = down.shape[0], down.shape[2]
    assert gate_up.shape == (E, 2 * I, H) and down.shape == (E, H, I)
    n_shared = 0 if sgu is None else sgu.shape[0]
    idx = _i32(idx)
    k = idx.shape[1]
    w = np.ascontiguousarray(w, dtype=np.float64)
    out = np.empty((T, H), dtype=np.float64)
    rc = _load().orc_expert_ffn(_ptr(x), T, H, I, E, k, dt, _ptr(idx), _ptr(w), _ptr(gate_up),
                                _ptr(down), n_shared, _ptr(sgu), _ptr(sdn), _ptr(out))
    if rc:
        raise ValueError("orc_expert_ffn: bad arguments")
    return out


def moe_verify(x, w_router, bias, gate_up, down, alpha, k, params: SelectParams | None = None,
               weighting=0, routed_scale=1.0, shared_gate_up=None, shared_down=None,
               resident_mask=None, mask_override=None, anchor_nodes=None, with_ffn=True):
    """The whole path for one block and layer, stage by stage (Sections 3.1-3.4)."""
    logits, probs, nat = router(x, w_router, bias, k)
    E = logits.shape[1]
    if mask_override is not None:
        mask = _u32(mask_override).copy()
        sel = {"mask": mask, "unpruned_mask": mask.copy(),
               "count": int(sum(bin(int(v)).count("1") for v in mask)),
               "demand": None, "stats": None}
    else:
        sel = select_eligible(probs, nat, alpha, params, anchor_nodes, resident_mask)
    idx, w = route_restricted(logits, sel["mask"], k, weighting, routed_scale)
    out = None
    if with_ffn:
        out = expert_ffn(x, idx, w, gate_up, down, shared_gate_up, shared_down)
    return {"logits": logits, "probs": probs, "nat_idx": nat, "mask": sel["mask"],
            "unpruned_mask": sel["unpruned_mask"], "count": sel["count"], "demand": sel["demand"],
            "stats": sel["stats"], "idx": idx, "w": w, "out": out, "n_experts": E}


# E2M1 code -> value (sign bit 3, exponent bits 2:1 with bias 1, mantissa bit 0; exponent 0 is subnormal)
_E2M1 = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0], dtype=np.float64)


def dequantize_mxfp4(codes, scales):
    """MXFP4 -> float64: codes [..., K] uint8 (4-bit E2M1 codes), scales [..., K/32] uint8 (E8M0: 2^(s-127));
    value = (-1)^sign * e2m1(code & 7) * 2^(s - 127).  Every result is exactly representable in bfloat16 as
    long as it is in range, so an MXFP4 layer is the bf16 layer with these weights."""
    codes = _np(codes).astype(np.int64)
    scales = _np(scales).astype(np.int64)
    mag = _E2M1[codes & 7]
    sign = np.where(codes & 8, -1.0, 1.0)
    factor = np.ldexp(1.0, scales - 127)
    return sign * mag * np.repeat(factor, 32, axis=-1)
