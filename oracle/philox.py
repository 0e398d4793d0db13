"""Perturbation stream z_i ~ N(0, I) regenerated from a seed (test infrastructure).

The paper draws z_i "using s_i" (Algorithm 1) and relies on the MeZO seed
trick (Background, "ZO LLM Fine-Tuning") without fixing a generator.  This
build fixes one so that the result is unique:

* Philox4x32-10 exactly as published (Salmon, Moraes, Dror, Shaw, SC'11):
  10 rounds; per round (hi0,lo0) = M0*c0, (hi1,lo1) = M1*c2,
  c <- (hi1^c1^k0, lo1, hi0^c3^k1, lo0); the key is bumped by (W0, W1)
  between rounds.
* key = (seed low word, seed high word); counter = (e >> 2, tensor_id,
  query index i, 0) with e the row-major element index inside the LoRA B
  tensor; the element takes output word e & 3.
* word x -> uniform u = ((x >> 9) + 0.5) * 2^-23 in (0,1);
  words (0,1) and (2,3) form Box-Muller pairs:
  rho = sqrt(-2 ln u_a), phi = 2 pi u_b -> (rho cos phi, rho sin phi).
  Evaluated in fp64 here and rounded once to fp32.
"""
import numpy as np

_M0, _M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
_W0, _W1 = np.uint64(0x9E3779B9), np.uint64(0xBB67AE85)
_MASK = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(counter, key):
    """counter: uint32 array [..., 4]; key: two uint32 -> uint32 array [..., 4]."""
    c = np.asarray(counter).astype(np.uint64)
    c0, c1, c2, c3 = c[..., 0], c[..., 1], c[..., 2], c[..., 3]
    k0, k1 = np.uint64(int(key[0]) & 0xFFFFFFFF), np.uint64(int(key[1]) & 0xFFFFFFFF)
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _W0) & _MASK
            k1 = (k1 + _W1) & _MASK
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _S32, p0 & _MASK
        hi1, lo1 = p1 >> _S32, p1 & _MASK
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def perturbation_u32(seed, tensor_id, query, n_elems):
    """The raw 32-bit words behind the first n_elems elements of z for
    (tensor_id, query): element e reads word e&3 of block e>>2."""
    nblk = (n_elems + 3) // 4
    ctr = np.zeros((nblk, 4), np.uint32)
    ctr[:, 0] = np.arange(nblk, dtype=np.uint32)
    ctr[:, 1] = np.uint32(tensor_id)
    ctr[:, 2] = np.uint32(query)
    key = (int(seed) & 0xFFFFFFFF, (int(seed) >> 32) & 0xFFFFFFFF)
    return philox4x32_10(ctr, key).reshape(-1)[:n_elems]


def uniforms_from_u32(x):
    return ((np.asarray(x, np.uint32) >> np.uint32(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def box_muller(u_a, u_b):
    rho = np.sqrt(-2.0 * np.log(u_a))
    phi = 2.0 * np.pi * u_b
    return rho * np.cos(phi), rho * np.sin(phi)


def perturbation(seed, tensor_id, query, shape):
    """z for one LoRA B tensor and one query: fp32 values (as float64 array)."""
    n = int(np.prod(shape))
    nblk = (n + 3) // 4
    w = perturbation_u32(seed, tensor_id, query, nblk * 4).reshape(nblk, 4)
    u = uniforms_from_u32(w)
    z = np.empty((nblk, 4), np.float64)
    z[:, 0], z[:, 1] = box_muller(u[:, 0], u[:, 1])
    z[:, 2], z[:, 3] = box_muller(u[:, 2], u[:, 3])
    z = z.astype(np.float32).astype(np.float64)
    return z.reshape(-1)[:n].reshape(shape)
