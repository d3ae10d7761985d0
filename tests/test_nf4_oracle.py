"""Pins for the NF4 oracle (oracle/nf4_oracle.py): the level table, the quantiser's decisions, the storage format and
the dequantised values are each fixed against something other than the oracle itself."""
import os

import numpy as np
import pytest

from oracle import lora_oracle, nf4_oracle as nf4
from tests.test_oracle import _read_golden

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "nf4_block_example.txt")


def test_levels_match_the_quantile_construction():
    """QLoRA builds NF4 from normal quantiles: 8 positive and 7 negative quantile points plus an exact zero, scaled to
    [-1, 1], with the outermost probability (1 - 1/30 + 1 - 1/32) / 2.  scipy's normal quantile function rebuilds the
    table independently of the typed literals."""
    from scipy.stats import norm
    offset = 0.5 * ((1 - 1 / (2 * 15)) + (1 - 1 / (2 * 16)))
    pos = norm.ppf(np.linspace(offset, 0.5, 9))[:-1]
    neg = -norm.ppf(np.linspace(offset, 0.5, 8))[:-1]
    built = np.sort(np.concatenate([pos, [0.0], neg]))
    built /= np.max(np.abs(built))
    assert nf4.LEVELS.dtype == np.float32 and nf4.LEVELS.shape == (16,)
    assert np.max(np.abs(built - nf4.LEVELS.astype(np.float64))) <= 1e-6
    assert np.all(np.diff(nf4.LEVELS) > 0)
    assert nf4.LEVELS[0] == -1.0 and nf4.LEVELS[7] == 0.0 and nf4.LEVELS[15] == 1.0


def test_hand_worked_block():
    g = _read_golden(GOLDEN)
    W = np.zeros((1, 64), dtype=np.float32)
    W[0, :8] = g["w8"][0]
    codes, absmax = nf4.quantize(W)
    assert codes.shape == (1, 32) and absmax.shape == (1, 1)
    assert absmax[0, 0] == g["absmax"][0, 0]
    assert np.array_equal(nf4.unpack(codes)[0, :8], g["code8"][0].astype(np.uint8))
    assert np.all(nf4.unpack(codes)[0, 8:] == 7)
    assert np.array_equal(codes[0, :5], g["bytes5"][0].astype(np.uint8)) and np.all(codes[0, 4:] == 119)
    what = nf4.dequantize(codes, absmax)
    assert np.array_equal(what[0, :8], g["what8"][0])
    assert np.all(what[0, 8:] == 0.0)


def test_quantiser_picks_the_nearest_level_brute_force():
    rng = np.random.default_rng(0)
    W = (rng.standard_normal((24, 256)) * rng.uniform(0.01, 3.0, size=(24, 1))).astype(np.float32)
    codes, absmax = nf4.quantize(W)
    code = nf4.unpack(codes).astype(np.int64)
    scale = np.repeat(absmax.T.astype(np.float64), 64, axis=1)
    x = W.astype(np.float64) / scale
    L = nf4.LEVELS.astype(np.float64)
    dist = np.abs(x[:, :, None] - L[None, None, :])                # brute force over the 16 levels, float64
    best = dist.min(axis=2)
    chosen = np.take_along_axis(dist, code[:, :, None], axis=2)[:, :, 0]
    assert np.all(chosen <= best + 2e-7)                          # equal up to float32 rounding of x near a midpoint
    assert np.mean(code == dist.argmin(axis=2)) > 0.999
    # every block holds its own extreme: code 0 or 15 appears in every block
    blocks = code.reshape(24, 4, 64)
    assert np.all(((blocks == 0) | (blocks == 15)).any(axis=2))
    assert np.array_equal(absmax.T, np.abs(W).reshape(24, 4, 64).max(axis=2))


def test_round_trip_error_bound_and_exact_levels():
    rng = np.random.default_rng(1)
    W = rng.standard_normal((16, 128)).astype(np.float32)
    codes, absmax = nf4.quantize(W)
    what = nf4.dequantize(codes, absmax)
    scale = np.repeat(absmax.T.astype(np.float64), 64, axis=1)
    half_gap = float(np.max(np.diff(nf4.LEVELS.astype(np.float64)))) / 2
    assert np.all(np.abs(W - what) <= scale * (half_gap + 2.0 ** -8) + 1e-12)
    # values that sit exactly on a level come back as bf16(level * absmax) with that level's code
    Wl = np.zeros((1, 64), dtype=np.float32)
    Wl[0, :16] = nf4.LEVELS * np.float32(2.0)
    c2, a2 = nf4.quantize(Wl)
    assert a2[0, 0] == 2.0
    assert np.array_equal(nf4.unpack(c2)[0, :16], np.arange(16, dtype=np.uint8))
    got = nf4.dequantize(c2, a2)[0, :16]
    import torch
    want = (torch.tensor(nf4.LEVELS) * 2.0).to(torch.bfloat16).double().numpy()     # library's RNE bf16 rounding
    assert np.array_equal(got, want)
    # all-zero block: absmax 0, level-0 codes, zeros back
    cz, az = nf4.quantize(np.zeros((2, 64), dtype=np.float32))
    assert np.all(az == 0) and np.all(cz == 119) and np.all(nf4.dequantize(cz, az) == 0)


def test_midpoint_tie_goes_to_the_lower_code_and_packing_order():
    mids = nf4.midpoints()
    W = np.zeros((1, 64), dtype=np.float32)
    W[0, 0] = 1.0                                    # absmax 1: x = w
    W[0, 1] = mids[12]                               # exactly on the midpoint between codes 12 and 13
    W[0, 2] = np.nextafter(mids[12], np.float32(2.0))
    codes, _ = nf4.quantize(W)
    c = nf4.unpack(codes)[0]
    assert c[0] == 15 and c[1] == 12 and c[2] == 13
    assert codes[0, 0] == (15 | (12 << 4)) and codes[0, 1] == (13 | (7 << 4))     # even element in the low nibble
    with pytest.raises(ValueError):
        nf4.quantize(np.zeros((2, 32), dtype=np.float32))


def test_layer_with_nf4_weight_is_the_lora_layer_on_the_dequantised_weight():
    rng = np.random.default_rng(2)
    X, W = rng.standard_normal((5, 64)), rng.standard_normal((8, 64)).astype(np.float32)
    A, B, dY = rng.standard_normal((2, 64)), rng.standard_normal((8, 2)), rng.standard_normal((5, 8))
    codes, absmax = nf4.quantize(W)
    what = nf4.dequantize(codes, absmax)
    Y = nf4.forward(X, codes, absmax, A, B, 2.0)
    dX, dA, dB = nf4.backward(dY, X, codes, absmax, A, B, 2.0)
    # merged-weight identity written without the oracle's own matmul path
    Wm = what + 2.0 * np.einsum("or,ri->oi", B, A)
    np.testing.assert_allclose(Y, np.einsum("ti,oi->to", X, Wm), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dX, np.einsum("to,oi->ti", dY, Wm), rtol=1e-12, atol=1e-12)
    dA0, dB0 = lora_oracle.backward_adapter_grads(dY, X, A, B, 2.0)
    assert np.array_equal(dA, dA0) and np.array_equal(dB, dB0)          # W does not enter the adapter gradients
