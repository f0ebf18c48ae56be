"""The expert-FFN kernel's work plan, checked on the host: every weight stage of every activated expert is
streamed exactly once, cut tiles meet in the CTA that holds their first chunk, the CTAs' loads are balanced, and a
launch that started on the anchors hands the rest of its tiles to the CTAs that were idle first."""
import numpy as np
import pytest

from paper_2608_02989_b200 import acm

SHAPES = [(2048, 768), (2048, 1024), (2048, 1408), (4096, 1536), (512, 256), (256, 64), (1024, 320)]


def _check(n_act, H, I, G, n_pre=0):
    tpe, kc1, h_tiles = I // 64, H // 128, H // 128
    kpe = (tpe + 1) // 2
    pieces, n_seg = acm.ffn_plan(n_act, H, I, G, n_pre)
    assert 1 <= n_seg <= 5
    gu = np.zeros((n_act * tpe, kc1), dtype=np.int32)           # gate/up stage (tile, chunk) -> times streamed
    dn = np.zeros((h_tiles, n_act * kpe), dtype=np.int32)       # down stage (output tile, expert slot * kpe + chunk)
    load = np.zeros(G, dtype=np.int64)
    last_seg = np.full(G, -1)
    heads, parts = {}, {}
    seen_down = np.zeros(G, dtype=bool)
    for cta, si, phase, flag, tile, k0, k1, aux in pieces.tolist():
        assert 0 <= cta < G and k0 < k1 and si >= last_seg[cta]          # each CTA walks its segments in order
        last_seg[cta] = si
        load[cta] += k1 - k0
        if phase == 1:
            assert not seen_down[cta]                                     # all gate/up work before any down work
            assert 0 <= tile < n_act * tpe and k1 <= kc1
            gu[tile, k0:k1] += 1
            if flag == 1:
                assert (k0, k1) == (0, kc1)                               # a whole tile
            elif k0 == 0 and k1 < kc1:
                heads[(si, tile)] = cta
            elif k0 > 0:
                parts.setdefault((si, tile), []).append(cta)
        else:
            seen_down[cta] = True
            assert 0 <= tile < h_tiles
            dn[tile, aux * kpe + k0: aux * kpe + k1] += 1
    assert (gu == 1).all(), "a gate/up stage is streamed twice or never"
    assert (dn == 1).all(), "a down stage is streamed twice or never"
    for key, ctas in parts.items():                                       # partial sums go to the CTA with the tile's head
        assert key in heads and all(c > heads[key] for c in ctas)
    assert set(heads) <= set(parts)
    if n_pre:                                                             # segment 0: the anchors' tiles, one per CTA
        first = pieces[pieces[:, 1] == 0]
        assert sorted(first[:, 4].tolist()) == list(range(n_pre * tpe)) and (first[:, 0] == first[:, 4]).all()
    return load, pieces


@pytest.mark.parametrize("H,I", SHAPES)
def test_every_stage_is_streamed_exactly_once(H, I):
    tpe = I // 64
    for G in (148, 144, 141, 132, 7):
        for n_act in list(range(1, 34)) + [45, 64, 100, 132]:
            _check(n_act, H, I, G)
            for n_pre in {1, min(n_act, G // tpe), min(n_act, 8)}:
                if 0 < n_pre <= n_act and n_pre * tpe <= G:
                    _check(n_act, H, I, G, n_pre)


def test_qwen3_30b_sized_launch_is_balanced_to_the_stage():
    # 20 activated experts, 148 CTAs: 240 tiles = 92 cut over all CTAs + one whole round
    load, pieces = _check(20, 2048, 768, 148)
    gu = pieces[pieces[:, 2] == 1]
    assert (gu[:, 3] == 1).sum() == 148 and len({int(t) for t in gu[gu[:, 3] == 0][:, 4]}) == 92
    ideal = (20 * 12 * 16 + 20 * 16 * 6) / 148
    assert load.max() <= ideal + 3 and load.min() >= ideal - 3


def test_anchor_start_deals_whole_tiles_to_the_idle_ctas_first():
    # 8 anchors on 144 CTAs (96 tiles, CTAs 0..95), 19 experts in all: the 132 rest tiles are fewer than the CTAs and
    # are dealt whole -- to the 48 idle CTAs first, then to CTAs 0..83; nothing is cut, nothing is exchanged
    load, pieces = _check(19, 2048, 768, 144, n_pre=8)
    gu = pieces[(pieces[:, 2] == 1) & (pieces[:, 1] > 0)]
    assert (gu[:, 3] == 1).all() and len(gu) == 132
    owner = dict(zip(gu[:, 4].tolist(), gu[:, 0].tolist()))
    assert [owner[96 + i] for i in range(48)] == list(range(96, 144)) and owner[96 + 48] == 0 and owner[96 + 131] == 83
    # the anchors' experts come first in the down phase
    dn = pieces[pieces[:, 2] == 2]
    assert set(dn[dn[:, 1] == dn[:, 1].min()][:, 7].tolist()) == {0} and set(dn[:, 7].tolist()) == {0, 8}


def test_anchor_start_with_more_rest_tiles_than_ctas_cuts_the_leftover_first():
    # 21 experts on 144 CTAs behind 8 anchors: 156 rest tiles = 12 leftover (cut over all CTAs) + one whole round;
    # down: the anchors' experts and the leftover tiles' expert, then the whole round's experts
    load, pieces = _check(21, 2048, 768, 144, n_pre=8)
    seg_kind = {}
    for cta, si, phase, whole, tile, k0, k1, aux in pieces.tolist():
        seg_kind.setdefault(si, (phase, whole, aux if phase == 2 else None))
    assert [seg_kind[i] for i in sorted(seg_kind)] == [(1, 1, None), (1, 0, None), (1, 1, None), (2, 0, 0), (2, 0, 9)]
    assert load.max() - load.min() <= 16 + 3            # the anchor CTAs carry their anchor tile on top


def test_leftover_tiles_are_cut_and_few_tiles_are_cut_in_two_halves():
    # 150 tiles on 148 CTAs: the two that do not fill a round are cut over all CTAs
    load, pieces = _check(75, 2048, 128, 148)
    assert (pieces[pieces[:, 2] == 1][:, 3] == 0).any()
    assert load.max() - load.min() <= 2
    # fewer tiles than CTAs: everything cut, in two halves
    load, pieces = _check(5, 2048, 768, 148)
    assert (pieces[pieces[:, 2] == 1][:, 3] == 0).all()
    assert load.max() - load.min() <= 4                  # four segments, each cut to within a stage


def test_full_rounds_and_large_launches():
    for n_act, H, I in ((37, 2048, 256), (110, 4096, 1536), (56, 2048, 1024)):
        load, pieces = _check(n_act, H, I, 148)
        tpe, kc1 = I // 64, H // 128
        ideal = (n_act * tpe * kc1 + n_act * (H // 128) * ((tpe + 1) // 2)) / 148
        assert load.max() <= ideal + kc1            # never more than a tile above the balanced load
