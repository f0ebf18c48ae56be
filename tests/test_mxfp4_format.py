"""MXFP4 storage (E2M1 codes, one E8M0 scale per 32 elements): the oracle's dequantiser against the format's
definition, the input quantiser against it, and the library's tiled layout as a pure permutation."""
import numpy as np
import torch

import oracle
from paper_2608_02989_b200 import acm, workloads as wl


def test_dequantiser_reproduces_the_code_table_and_the_scale_rule():
    codes = np.tile(np.arange(16, dtype=np.uint8), 2)[None, :]           # one block holding every code twice
    want = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, -0.0, -.5, -1, -1.5, -2, -3, -4, -6] * 2)
    for s, factor in ((127, 1.0), (126, 0.5), (120, 2.0 ** -7), (130, 8.0), (0, 2.0 ** -127)):
        got = oracle.dequantize_mxfp4(codes, np.array([[s]], dtype=np.uint8))
        np.testing.assert_array_equal(got[0], want * factor)
    # E2M1 is sign | 2 exponent bits (bias 1) | 1 mantissa bit, exponent 0 subnormal: the table follows from that
    for code in range(8):
        e, m = code >> 1, code & 1
        assert wl.E2M1_VALUES[code] == (m * 0.5 if e == 0 else (1 + m / 2) * 2.0 ** (e - 1))


def test_every_dequantised_value_is_a_bfloat16():
    rng = np.random.default_rng(0)
    codes = rng.integers(0, 16, (64, 256), dtype=np.uint8)
    scales = rng.integers(90, 135, (64, 8), dtype=np.uint8)
    v = torch.tensor(oracle.dequantize_mxfp4(codes, scales))
    assert torch.equal(v.to(torch.bfloat16).double(), v)


def test_quantiser_is_the_nearest_representable_value_under_the_block_scale():
    g = torch.Generator().manual_seed(3)
    w = torch.randn(40, 256, generator=g) * 0.02
    w[0, :32] = 0.0                                     # a block of zeros
    w[1, 0] = 6.0 * 2.0 ** -6                           # exactly representable at its block's scale
    w[2, 32:64] = torch.tensor([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 7.0] * 4) * 2.0 ** -5     # midpoints and overflow
    codes, scales = wl.quantize_mxfp4(w)
    deq = oracle.dequantize_mxfp4(codes, scales)
    wd = w.double().numpy()
    blocks = wd.reshape(40, 8, 32)
    amax = np.abs(blocks).max(-1)
    sc = np.ldexp(1.0, scales.numpy().astype(int) - 127)
    nz = amax > 0
    # the block scale puts the largest magnitude into [4, 8): 2^(floor(log2 amax) - 2)
    assert np.all((amax[nz] / sc[nz] >= 4.0) & (amax[nz] / sc[nz] < 8.0))
    assert np.all(deq.reshape(40, 8, 32)[~nz] == 0.0)
    # every element is the closest grid point (saturating at 6), so no other grid point is closer
    grid = np.array(wl.E2M1_VALUES)
    scaled = np.abs(blocks) / sc[..., None]
    err = np.abs(np.abs(deq.reshape(40, 8, 32)) / sc[..., None] - np.minimum(scaled, 6.0))
    best = np.abs(np.minimum(scaled, 6.0)[..., None] - grid).min(-1)
    np.testing.assert_allclose(err, best, atol=1e-12)
    assert np.all(np.sign(deq) * np.sign(wd) >= 0)
    assert deq[1, 0] == wd[1, 0]
    # midpoints go to the even code: 0.25 -> 0, 0.75 -> 1, 1.25 -> 1, 1.75 -> 2, 2.5 -> 2, 3.5 -> 4, 5 -> 4; 7 saturates
    np.testing.assert_array_equal(deq[2, 32:40] * 2.0 ** 5, [0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 4.0, 6.0])
    # relative error of the synthetic weights as a whole: what 1 mantissa bit gives
    rel = np.linalg.norm(deq - wd) / np.linalg.norm(wd)
    assert 0.05 < rel < 0.2


def _unpack_words(tile_bytes):
    """Inverse of the word order: [rows, 64] bytes -> [rows, 128] codes."""
    rows = tile_bytes.shape[0]
    pieces = tile_bytes.reshape(rows, 4, 16)
    unrot = np.empty_like(pieces)
    for r in range(rows):
        for piece in range(4):
            unrot[r, piece] = pieces[r, piece ^ ((r >> 1) & 3)]
    b = unrot.astype(np.uint32).reshape(-1, 16, 4)
    word = b[..., 0] | (b[..., 1] << 8) | (b[..., 2] << 16) | (b[..., 3] << 24)
    out = np.zeros(word.shape + (8,), dtype=np.uint8)
    for j in range(4):
        out[..., 2 * j] = (word >> (4 * j)) & 0xF
        out[..., 2 * j + 1] = (word >> (16 + 4 * j)) & 0xF
    return out.reshape(-1, 128)


def test_tiled_layout_is_a_permutation_of_the_plain_one():
    rng = np.random.default_rng(1)
    E, I, H = 3, 128, 256
    codes = torch.tensor(rng.integers(0, 16, (E, 2 * I, H), dtype=np.uint8))
    scales = torch.tensor(rng.integers(100, 130, (E, 2 * I, H // 32), dtype=np.uint8))
    t = acm.pack_mxfp4_gate_up(codes, scales).numpy()
    assert t.shape == (E, I // 64, H // 128, acm.MX_STAGE_BYTES)
    for e, tile, stage in ((0, 0, 0), (2, 1, 1), (1, 1, 0)):
        blk = t[e, tile, stage]
        got = _unpack_words(blk[: 128 * 64].reshape(128, 64))
        rows = list(range(64 * tile, 64 * tile + 64)) + list(range(I + 64 * tile, I + 64 * tile + 64))
        np.testing.assert_array_equal(got, codes.numpy()[e][rows, 128 * stage: 128 * stage + 128])
        np.testing.assert_array_equal(blk[128 * 64:].reshape(128, 4), scales.numpy()[e][rows, 4 * stage: 4 * stage + 4])
    dc = torch.tensor(rng.integers(0, 16, (E, H, I), dtype=np.uint8))
    ds = torch.tensor(rng.integers(100, 130, (E, H, I // 32), dtype=np.uint8))
    t = acm.pack_mxfp4_down(dc, ds).numpy()
    assert t.shape == (E, H // 128, I // 128, acm.MX_STAGE_BYTES)
    blk = t[1, 1, 0]
    np.testing.assert_array_equal(_unpack_words(blk[: 128 * 64].reshape(128, 64)), dc.numpy()[1][128:256, 0:128])
    np.testing.assert_array_equal(blk[128 * 64:].reshape(128, 4), ds.numpy()[1][128:256, 0:4])
