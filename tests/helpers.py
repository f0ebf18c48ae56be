"""Shared helpers for the tests (no method arithmetic)."""
import numpy as np


def mask_to_set(mask, E):
    mask = np.asarray(mask).view(np.uint32)
    return {e for e in range(E) if (int(mask[e // 32]) >> (e % 32)) & 1}


def set_to_mask(s, E):
    m = np.zeros((E + 31) // 32, dtype=np.uint32)
    for e in s:
        m[e // 32] |= np.uint32(1 << (e % 32))
    return m


def full_mask(E):
    return set_to_mask(range(E), E)


def topk_brute(z, k, allowed=None):
    """indices of the k largest entries, ties to the lower index."""
    cand = list(range(len(z))) if allowed is None else sorted(allowed)
    cand.sort(key=lambda e: (-float(z[e]), e))
    return cand[:k]
