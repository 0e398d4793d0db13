"""Pins for the oracle's weight-only dequantisers (CPU only)."""
import numpy as np
from scipy.stats import norm

import oracle
from oracle import quant as oq
from workloads import ModelSpec, make_decoder_problem, quantize_int8, quantize_layer, quantize_nf4
from workloads.spec import ARCH_LLAMA


def test_nf4_levels_are_the_published_normal_quantile_construction():
    """NormalFloat-4: 8 positive quantiles of N(0,1) from p = 0.9677083 down to (not including) 0.5,
    zero, 7 negative ones, normalised by the largest."""
    off = 0.9677083
    pos = norm.ppf(np.linspace(off, 0.5, 9)[:-1])
    neg = -norm.ppf(np.linspace(off, 0.5, 8)[:-1])
    v = np.sort(np.concatenate([pos, [0.0], neg]))
    v /= v.max()
    assert oq.NF4_LEVELS.shape == (16,)
    assert np.abs(v - oq.NF4_LEVELS).max() < 2e-7
    assert oq.NF4_LEVELS[7] == 0.0 and oq.NF4_LEVELS[0] == -1.0 and oq.NF4_LEVELS[15] == 1.0
    assert np.all(np.diff(oq.NF4_LEVELS) > 0)


def test_nf4_nibble_order_block_scaling_and_error_bound():
    # hand-built: row of 64 elements, absmax 2.0, codes 0..15 repeated; even element in the high nibble
    codes = np.arange(64, dtype=np.uint8) % 16
    packed = ((codes[0::2] << 4) | codes[1::2])[None, :]
    w = oq.dequant_nf4(packed, np.array([[2.0]], np.float32), bf16=False)
    assert np.array_equal(w[0], (oq.NF4_LEVELS[codes] * np.float32(2.0)).astype(np.float64))
    assert w[0, 0] == -2.0 and w[0, 1] == np.float64(np.float32(-0.6961928009986877) * np.float32(2.0))
    # two blocks scale independently; round trip within half the widest level gap times absmax
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 128)).astype(np.float32) * np.array([[1.0] * 64 + [10.0] * 64], np.float32)
    p, a = quantize_nf4(x)
    assert p.shape == (5, 64) and a.shape == (5, 2)
    y = oq.dequant_nf4(p, a, bf16=False)
    gap = np.diff(oq.NF4_LEVELS).max() / 2
    err = np.abs(y - x).reshape(5, 2, 64).max(axis=2)
    assert np.all(err <= gap * a * (1 + 1e-6))
    # the element holding the block's absmax is reproduced exactly (levels +-1)
    blk = np.abs(x).reshape(5, 2, 64)
    yb = np.abs(y).reshape(5, 2, 64)
    assert np.array_equal(yb.max(axis=2), blk.max(axis=2).astype(np.float64))


def test_int8_round_trip_and_exact_grid():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((7, 40)).astype(np.float32)
    c, s = quantize_int8(x)
    y = oq.dequant_int8(c, s, bf16=False)
    assert np.all(np.abs(y - x) <= s[:, None] / 2 * (1 + 1e-6))
    grid = (np.arange(-127, 128, dtype=np.float32)[None, :] * np.float32(0.25))
    c, s = quantize_int8(grid)
    assert np.array_equal(oq.dequant_int8(c, s, bf16=False)[0], grid[0].astype(np.float64))
    # bf16 storage: values are bf16-representable and within half a bf16 ulp of the fp32 product
    yb = oq.dequant_int8(*quantize_int8(x), bf16=True)
    assert np.all((yb.astype(np.float32).view(np.uint32) & 0xFFFF) == 0)
    assert np.all(np.abs(yb - y) <= np.abs(y) * 2.0 ** -8)


def test_forward_with_quantised_record_equals_forward_with_its_dequantised_weights():
    spec = ModelSpec(arch=ARCH_LLAMA, n_layers=2, d_model=64, n_heads=4, d_ffn=128, vocab=53, max_seq=8,
                     lora_rank=2, E=2, S=8, n_labelled=3, bf16=True)
    p = make_decoder_problem(spec, seed=3, b_std=0.05)
    Bs = [np.asarray(L["B"], np.float64)[None] for L in p["layers"]]
    for fmt in ("int8", "nf4"):
        pq = dict(p, layers=[quantize_layer(L, fmt) for L in p["layers"]])
        pd = dict(p, layers=[{k: (oq.weight(v, True) if isinstance(v, dict) else v) for k, v in L.items()}
                             for L in pq["layers"]])
        a = oracle.replica_losses(spec, pq, Bs, p["tokens"], p["labels"])
        b = oracle.replica_losses(spec, pd, Bs, p["tokens"], p["labels"])
        c = oracle.replica_losses(spec, p, Bs, p["tokens"], p["labels"])
        assert np.array_equal(a, b)
        assert a[0] != c[0] and abs(a[0] - c[0]) < 0.2 * c[0]      # quantisation moves the loss a little
