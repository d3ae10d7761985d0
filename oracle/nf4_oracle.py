"""CPU oracle for the 4-bit NormalFloat (NF4) frozen weight of the quantised-LoRA regime.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this file; it shares no
code, table or constant generator with the CUDA library.

Section 4.5 ("Quantised LoRA", Q+LoRA) trains the same LoRA layer with the frozen W held in
NF4 (Dettmers et al. 2023, QLoRA: 4-bit NormalFloat with block-wise absmax scaling).  The
paper fixes no storage format, so this library defines one (the kernels follow the same
written rules, in code of their own):

  * W [d_out, d_in] is cut into blocks of 64 consecutive elements along d_in (d_in % 64 == 0).
  * absmax[b, o] = max |W[o, 64 b : 64 b + 64]| as float32, stored block-major: [d_in / 64, d_out].
  * each element is coded by the nearest of the 16 NF4 levels to  x = w / absmax  (float32
    division; a block of zeros has absmax 0 and codes 7, the level 0.0).  "Nearest" is decided
    by counting the float32 midpoints between neighbouring levels that lie strictly below x,
    so a value exactly on a midpoint takes the lower code.
  * codes [d_out, d_in / 2] uint8: byte k of a row holds element 2k in its LOW nibble and
    element 2k + 1 in its HIGH nibble.
  * dequantisation:  w_hat = bf16( float32(level[code]) * absmax )  - one float32 product, one
    round-to-nearest-even to bf16 (the compute dtype of the GEMMs).

The layer itself is unchanged: forward and backward are lora_oracle's with W replaced by w_hat.

The 16 levels are the published NF4 code book (QLoRA, Appendix E), typed here as float32
literals.  Pins (tests/test_nf4_oracle.py): the quantile construction of the QLoRA paper
evaluated with scipy reproduces the table to 1e-6; the table is strictly increasing with
-1, 0, +1 at codes 0, 7, 15; a hand-worked block under tests/golden/; brute-force nearest
search in float64; the round-trip error bound |w - w_hat| <= absmax * (largest half gap +
bf16 rounding); exact round trip of values that sit on a level; packing order.
"""
from __future__ import annotations

import numpy as np

BLOCK = 64

# NF4 levels (QLoRA, Appendix E), float32
LEVELS = np.array([
    -1.0, -0.6961928009986877, -0.5250730514526367, -0.39491748809814453,
    -0.28444138169288635, -0.18477343022823334, -0.09105003625154495, 0.0,
    0.07958029955625534, 0.16093020141124725, 0.24611230194568634, 0.33791524171829224,
    0.44070982933044434, 0.5626170039176941, 0.7229568362236023, 1.0], dtype=np.float32)


def midpoints() -> np.ndarray:
    """float32 midpoints between neighbouring levels: (L[k] + L[k+1]) / 2 evaluated in float32."""
    return ((LEVELS[:-1] + LEVELS[1:]) * np.float32(0.5)).astype(np.float32)


def _bf16_rne(x32: np.ndarray) -> np.ndarray:
    """float32 -> nearest bf16 (ties to even), returned as float32 values."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def quantize(W) -> tuple[np.ndarray, np.ndarray]:
    """W [d_out, d_in] (any float type, used as float32) -> (codes uint8 [d_out, d_in/2], absmax float32 [d_in/64, d_out])."""
    W = np.asarray(W, dtype=np.float32)
    d_out, d_in = W.shape
    if d_in % BLOCK != 0:
        raise ValueError("d_in must be a multiple of 64")
    blocks = W.reshape(d_out, d_in // BLOCK, BLOCK)
    absmax = np.max(np.abs(blocks), axis=2).astype(np.float32)              # [d_out, n_blocks]
    safe = np.where(absmax > 0, absmax, np.float32(1.0)).astype(np.float32)
    x = (blocks / safe[:, :, None]).astype(np.float32)                      # float32 division
    mids = midpoints()
    code = np.zeros(x.shape, dtype=np.uint8)
    for m in mids:                                                          # count the midpoints strictly below x
        code += (x > m).astype(np.uint8)
    code = np.where(absmax[:, :, None] > 0, code, np.uint8(7)).astype(np.uint8)
    code = code.reshape(d_out, d_in)
    packed = (code[:, 0::2] | (code[:, 1::2] << np.uint8(4))).astype(np.uint8)
    return packed, np.ascontiguousarray(absmax.T)


def unpack(codes: np.ndarray) -> np.ndarray:
    """codes [d_out, d_in/2] -> one 4-bit code per element, [d_out, d_in]."""
    codes = np.asarray(codes, dtype=np.uint8)
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & np.uint8(0x0F)
    out[:, 1::2] = codes >> np.uint8(4)
    return out


def dequantize(codes, absmax) -> np.ndarray:
    """(codes, absmax) -> w_hat [d_out, d_in] as float64 holding bf16 values: bf16(float32(level) * absmax)."""
    code = unpack(codes)
    d_out, d_in = code.shape
    absmax = np.asarray(absmax, dtype=np.float32)
    if absmax.shape != (d_in // BLOCK, d_out):
        raise ValueError("absmax must be [d_in/64, d_out]")
    scale = np.repeat(absmax.T, BLOCK, axis=1)                              # [d_out, d_in]
    prod = (LEVELS[code] * scale).astype(np.float32)                        # one float32 product
    return _bf16_rne(prod).astype(np.float64)


def forward(X, codes, absmax, A, B, s: float) -> np.ndarray:
    """Y = X w_hat^T + s (X A^T) B^T with the NF4 weight (Section 4.5, Q+LoRA)."""
    from oracle import lora_oracle
    return lora_oracle.forward(X, dequantize(codes, absmax), A, B, s)


def backward(dY, X, codes, absmax, A, B, s: float):
    """(dX, dA, dB) with the NF4 weight: dX = dY w_hat + s (dY B) A; dA, dB do not involve W."""
    from oracle import lora_oracle
    return lora_oracle.backward(dY, X, dequantize(codes, absmax), A, B, s)
