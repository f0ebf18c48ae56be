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


class LruModel:
    """The pool policy restated for the test: free slots first (lowest index), else the least recently used
    slot among those the current block does not use; ties to the lower slot index."""

    def __init__(self, n_slots, initial):
        self.slot_expert = [-1] * n_slots
        self.last_use = [0] * n_slots
        self.tick = 0
        for i, e in enumerate(initial):
            self.slot_expert[i] = e

    def resident(self):
        return {e for e in self.slot_expert if e >= 0}

    def block(self, activated):
        """One block: hits are touched; misses are loaded in ascending id order, in waves -- the first wave may
        only replace slots this block does not use, every later wave any slot it has not just filled."""
        self.tick += 1
        n = len(self.slot_expert)
        hits = misses = 0
        for s, e in enumerate(self.slot_expert):
            if e in activated:
                self.last_use[s] = self.tick
                hits += 1
        todo = sorted(activated - self.resident())
        wave, wave_of = 0, [-1] * n
        while todo:
            while todo:
                cand = [s for s in range(n) if wave_of[s] != wave and not (wave == 0 and self.last_use[s] == self.tick)]
                if not cand:
                    break
                victim = min(cand, key=lambda s: (self.last_use[s], s))
                self.slot_expert[victim] = todo.pop(0)
                self.last_use[victim] = self.tick
                wave_of[victim] = wave
                misses += 1
            wave += 1
        return hits, misses
