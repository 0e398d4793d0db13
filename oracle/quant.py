"""Decoders of the weight-only quantised formats (test infrastructure).

The paper keeps the frozen weights in INT8 or NF4 (Q-LoRA style) and dequantises them to the 16-bit
compute type during the forward pass (appendix "MobiZO with weight-only quantization"); with MP-LoRA
this happens once per step for all 2q paths.  Formats as read by this build: INT8 = code * per-row
scale; NF4 = level[code] * per-block absmax, blocks of 64 along the input dimension, two codes per
byte with the even element in the high nibble.  The dequantised value is rounded to the storage type
the GEMM consumes (bfloat16, or kept in float32).
"""
import numpy as np

# 4-bit NormalFloat levels as published with Q-LoRA; pinned in the tests against their construction
# from normal quantiles.
NF4_LEVELS = np.array([-1.0, -0.6961928009986877, -0.5250730514526367, -0.39491748809814453,
                       -0.28444138169288635, -0.18477343022823334, -0.09105003625154495, 0.0,
                       0.07958029955625534, 0.16093020141124725, 0.24611230194568634,
                       0.33791524171829224, 0.44070982933044434, 0.5626170039176941,
                       0.7229568362236023, 1.0], np.float32)


def _round_bf16(x32: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x32, np.float32).view(np.uint32)
    r = ((u + (((u >> 16) & 1) + np.uint32(0x7FFF))) >> 16).astype(np.uint32) << 16
    return r.view(np.float32)


def dequant_int8(codes, scale, bf16: bool):
    w = codes.astype(np.float32) * np.asarray(scale, np.float32)[:, None]     # one fp32 product
    return (_round_bf16(w) if bf16 else w).astype(np.float64)


def dequant_nf4(packed, absmax, bf16: bool):
    rows, half = packed.shape
    codes = np.empty((rows, 2 * half), np.uint8)
    codes[:, 0::2] = packed >> 4
    codes[:, 1::2] = packed & 0xF
    lv = NF4_LEVELS[codes].reshape(rows, -1, 64)
    w = (lv * np.asarray(absmax, np.float32)[:, :, None]).reshape(rows, 2 * half)  # one fp32 product
    return (_round_bf16(w) if bf16 else w).astype(np.float64)


def weight(x, bf16: bool):
    """A frozen weight as float64: a plain array, or a quantised record {'fmt','codes','scale'}."""
    if isinstance(x, dict):
        if x["fmt"] == "int8":
            return dequant_int8(x["codes"], x["scale"], bf16)
        return dequant_nf4(x["codes"], x["scale"], bf16)
    return np.asarray(x, np.float64)
