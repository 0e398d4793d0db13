"""Weight-only quantised storage formats for the frozen linear weights (encoders only).

The paper stores the frozen weights in INT8 or NF4 "building on Q-LoRA" and dequantises them during the
forward pass; it does not restate the formats.  This build's reading:

* INT8: symmetric, one float32 scale per output row, scale = max|w| / 127, code = round(w / scale).
* NF4: the 4-bit NormalFloat codebook of the Q-LoRA paper, blocks of 64 consecutive elements along the
  input dimension, one float32 absmax per block (no double quantisation), code = nearest level of
  w / absmax; two codes per byte, the even element in the high nibble.

These functions only produce stored bytes for the synthetic checkpoints; the decoders are written
separately in the oracle and in the CUDA library.
"""
import numpy as np

NF4_BLOCK = 64
# 4-bit NormalFloat levels (Dettmers et al., "QLoRA", 2023): 7 negative and 8 positive normal
# quantiles plus zero, normalised to [-1, 1].
_NF4 = np.array([-1.0, -0.6961928009986877, -0.5250730514526367, -0.39491748809814453,
                 -0.28444138169288635, -0.18477343022823334, -0.09105003625154495, 0.0,
                 0.07958029955625534, 0.16093020141124725, 0.24611230194568634, 0.33791524171829224,
                 0.44070982933044434, 0.5626170039176941, 0.7229568362236023, 1.0], np.float32)


def quantize_int8(w: np.ndarray):
    """w [rows, K] float32 -> (codes int8 [rows, K], scale float32 [rows])."""
    w = np.asarray(w, np.float32)
    scale = (np.abs(w).max(axis=1) / 127.0).astype(np.float32)
    scale = np.where(scale > 0, scale, np.float32(1.0))
    codes = np.clip(np.rint(w / scale[:, None]), -127, 127).astype(np.int8)
    return codes, scale


def quantize_nf4(w: np.ndarray):
    """w [rows, K] float32, K % 64 == 0 -> (packed uint8 [rows, K/2], absmax float32 [rows, K/64])."""
    w = np.asarray(w, np.float32)
    rows, K = w.shape
    assert K % NF4_BLOCK == 0
    blk = w.reshape(rows, K // NF4_BLOCK, NF4_BLOCK)
    absmax = np.abs(blk).max(axis=2).astype(np.float32)
    safe = np.where(absmax > 0, absmax, np.float32(1.0))
    x = blk / safe[:, :, None]
    mid = (_NF4[:-1] + _NF4[1:]) * np.float32(0.5)           # nearest level; a tie goes to the lower one
    codes = np.searchsorted(mid, x.reshape(-1), side="left").astype(np.uint8).reshape(rows, K)
    packed = ((codes[:, 0::2] << 4) | codes[:, 1::2]).astype(np.uint8)
    return packed, safe


def quantize_layer(L: dict, fmt: str) -> dict:
    """Replace the four linear weights of a decoder block by {'fmt', 'codes', 'scale'} records."""
    out = dict(L)
    for name in ("w_qkv", "w_o", "w_fc1", "w_fc2"):
        if fmt == "int8":
            c, s = quantize_int8(L[name])
        elif fmt == "nf4":
            c, s = quantize_nf4(L[name])
        else:
            raise ValueError(fmt)
        out[name] = {"fmt": fmt, "codes": c, "scale": s, "shape": L[name].shape}
    return out
