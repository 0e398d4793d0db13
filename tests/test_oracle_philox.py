"""Pins for the oracle's perturbation stream (CPU only)."""
import os

import numpy as np

from oracle import philox

GOLD = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(t, 16) for t in line.split()]
        yield w[:4], w[4:6], w[6:]


def test_philox_known_answers():
    n = 0
    for ctr, key, out in _kat():
        got = philox.philox4x32_10(np.array(ctr, np.uint32), key)
        assert [int(x) for x in got] == out
        n += 1
    assert n == 3


def test_philox_scalar_python_integers_agree():
    """Bit-level cross-check on random counters with unbounded Python ints
    (guards the uint64 vectorisation: masks, shifts, key schedule)."""
    rng = np.random.default_rng(0)
    ctrs = rng.integers(0, 2 ** 32, size=(64, 4), dtype=np.uint64).astype(np.uint32)
    key = (0x9ABCDEF0, 0x12345678)
    got = philox.philox4x32_10(ctrs, key)
    for c, g in zip(ctrs, got):
        c0, c1, c2, c3 = (int(v) for v in c)
        k0, k1 = key
        for r in range(10):
            p0, p1 = 0xD2511F53 * c0, 0xCD9E8D57 * c2
            c0, c1, c2, c3 = (p1 >> 32) ^ c1 ^ k0, p1 & 0xFFFFFFFF, (p0 >> 32) ^ c3 ^ k1, p0 & 0xFFFFFFFF
            k0, k1 = (k0 + 0x9E3779B9) & 0xFFFFFFFF, (k1 + 0xBB67AE85) & 0xFFFFFFFF
        assert [int(v) for v in g] == [c0, c1, c2, c3]


def test_counter_layout_and_lane_mapping():
    seed = 0x0123456789ABCDEF
    w = philox.perturbation_u32(seed, tensor_id=7, query=3, n_elems=37)
    assert w.shape == (37,)
    for e in (0, 1, 5, 18, 36):
        blk = philox.philox4x32_10(np.array([e >> 2, 7, 3, 0], np.uint32),
                                   (0x89ABCDEF, 0x01234567))
        assert int(w[e]) == int(blk[e & 3])
    # different tensor / query / seed give different streams
    assert not np.array_equal(w, philox.perturbation_u32(seed, 8, 3, 37))
    assert not np.array_equal(w, philox.perturbation_u32(seed, 7, 2, 37))
    assert not np.array_equal(w, philox.perturbation_u32(seed + 1, 7, 3, 37))


def test_uniform_map_is_open_interval_and_exact():
    u = philox.uniforms_from_u32(np.array([0, 0x1FF, 0x200, 0xFFFFFFFF], np.uint32))
    assert u[0] == 2.0 ** -24 and u[1] == 2.0 ** -24      # low 9 bits are dropped
    assert u[2] == 1.5 * 2.0 ** -23
    assert u[3] == 1.0 - 2.0 ** -24
    assert np.all(u.astype(np.float32).astype(np.float64) == u)   # exact in fp32


def test_box_muller_closed_form_points():
    a, b = philox.box_muller(np.exp(-0.5), 0.0)           # rho = 1, phi = 0
    assert abs(a - 1.0) < 1e-15 and abs(b) < 1e-15
    a, b = philox.box_muller(np.exp(-2.0), 0.25)          # rho = 2, phi = pi/2
    assert abs(a) < 1e-15 and abs(b - 2.0) < 1e-15
    a, b = philox.box_muller(np.exp(-0.5), 0.5)
    assert abs(a + 1.0) < 1e-15


def test_perturbation_is_standard_normal():
    z = philox.perturbation(42, 0, 0, (64, 4096)).reshape(-1)
    n = z.size
    assert abs(z.mean()) < 5 / np.sqrt(n)
    assert abs(z.var() - 1.0) < 5 * np.sqrt(2.0 / n)
    assert abs((z ** 3).mean()) < 5 * np.sqrt(15.0 / n)
    assert abs((z ** 4).mean() - 3.0) < 5 * np.sqrt(96.0 / n)
    # pairs from one block are uncorrelated, and so are neighbouring blocks
    zz = z.reshape(-1, 4)
    for i, j in ((0, 1), (2, 3), (0, 2), (1, 3)):
        assert abs((zz[:, i] * zz[:, j]).mean()) < 5 / np.sqrt(n / 4)
    assert abs((zz[:-1, 0] * zz[1:, 0]).mean()) < 5 / np.sqrt(n / 4)
    # tail mass: P(|z| > 3) = 0.0026998
    assert abs((np.abs(z) > 3).mean() - 0.0026998) < 5 * np.sqrt(0.0027 / n)
    # values are fp32
    assert np.all(z.astype(np.float32).astype(np.float64) == z)


def test_perturbation_shape_and_prefix_property():
    a = philox.perturbation(5, 3, 1, (8, 12))
    b = philox.perturbation(5, 3, 1, (96,))
    assert np.array_equal(a.reshape(-1), b)
    c = philox.perturbation(5, 3, 1, (10,))               # ragged: not a multiple of 4
    assert np.array_equal(c, b[:10])
