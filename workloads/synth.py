"""Seeded synthetic tensors standing in for pretrained checkpoints and
tokenised task prompts (neither is available offline).

Recipe: frozen weights, embeddings and LoRA A ~ N(0, 0.02); biases ~ N(0, 0.02);
norm gains ~ 1 + N(0, 0.02); LoRA B = 0 (the LoRA initialisation stated in the
paper's Background section) or N(0, b_std) for a "mid-training" state; token
ids uniform in [0, V); MSE targets N(0, 1).  Everything is float32 on the host;
with ``spec.bf16`` the frozen tensors hold bf16-representable values so that a
16-bit device copy is exact.
"""
from __future__ import annotations

import numpy as np

from .spec import (ARCH_LINEAR, ARCH_OPT, ARCH_LLAMA, LOSS_CE_LABEL_WORDS, ModelSpec)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + bias) >> 16).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def bf16_round(x: np.ndarray) -> np.ndarray:
    return from_bf16_bits(to_bf16_bits(x))


def _rng(seed: int, *ids: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), *[int(i) for i in ids]])


def _normal(rng, shape, std, bf16, mean=0.0):
    x = rng.standard_normal(shape, dtype=np.float32)
    x *= np.float32(std)
    if mean:
        x += np.float32(mean)
    return bf16_round(x) if bf16 else x


def make_linear_problem(spec: ModelSpec, seed: int = 1234, b_std: float = 0.0):
    """Single MP-LoRA linear with an MSE loss.  X [T,k_in], target [T,k_out],
    W [k_out,k_in], A [r,k_in], B [r,k_out] (B always float32)."""
    assert spec.arch == ARCH_LINEAR
    T, ki, ko, r = spec.E * spec.S, spec.d_model, spec.d_out, spec.lora_rank
    h = spec.bf16
    p = {
        "W": _normal(_rng(seed, 1), (ko, ki), 0.02, h),
        "bias": _normal(_rng(seed, 2), (ko,), 0.02, h),
        "A": _normal(_rng(seed, 3), (r, ki), 0.02, h),
        "B": (_normal(_rng(seed, 4), (r, ko), b_std, False) if b_std > 0
              else np.zeros((r, ko), np.float32)),
        "X": _normal(_rng(seed, 5), (T, ki), 1.0, h),
        "target": _normal(_rng(seed, 6), (T, ko), 1.0, False),
    }
    return p


def make_decoder_globals(spec: ModelSpec, seed: int = 1234):
    """Embeddings, final norm, LM head, tokens and labels of a random-init decoder."""
    d, V = spec.d_model, spec.vocab
    h = spec.bf16
    opt = spec.arch == ARCH_OPT
    p = {"tok_emb": _normal(_rng(seed, 10), (V, d), 0.02, h),
         "final_norm_g": _normal(_rng(seed, 12), (d,), 0.02, h, mean=1.0)}
    if opt:
        p["pos_emb"] = _normal(_rng(seed, 11), (spec.max_seq, d), 0.02, h)
        p["final_norm_b"] = _normal(_rng(seed, 13), (d,), 0.02, h)
    if not spec.tie_lm_head:
        p["lm_head"] = _normal(_rng(seed, 14), (V, d), 0.02, h)
    p["tokens"] = _rng(seed, 20).integers(0, V, size=(spec.E, spec.S), dtype=np.int32)
    if spec.loss_kind == LOSS_CE_LABEL_WORDS:
        p["labels"] = label_word_labels(spec, seed)
    else:
        p["labels"] = next_token_labels(p["tokens"], spec.n_labelled)
    return p


def make_decoder_layer(spec: ModelSpec, seed: int, l: int, b_std: float = 0.0):
    """Frozen tensors and LoRA A/B of decoder block ``l``: norm1, fused q|k|v projection
    [3d,d], output projection, norm2, MLP (OPT: fc1 [ffn,d], fc2 [d,ffn]; Llama: fc1 = gate
    rows then up rows [2ffn,d], fc2 [d,ffn]), LoRA A [n_targets*r, d], B [n_targets, r, d]."""
    d, f, r, nt = spec.d_model, spec.d_ffn, spec.lora_rank, spec.n_targets
    h = spec.bf16
    opt = spec.arch == ARCH_OPT
    f1 = f if opt else 2 * f
    L = {
        "norm1_g": _normal(_rng(seed, 100, l, 0), (d,), 0.02, h, mean=1.0),
        "w_qkv": _normal(_rng(seed, 100, l, 2), (3 * d, d), 0.02, h),
        "w_o": _normal(_rng(seed, 100, l, 4), (d, d), 0.02, h),
        "norm2_g": _normal(_rng(seed, 100, l, 6), (d,), 0.02, h, mean=1.0),
        "w_fc1": _normal(_rng(seed, 100, l, 8), (f1, d), 0.02, h),
        "w_fc2": _normal(_rng(seed, 100, l, 10), (d, f), 0.02, h),
        "A": _normal(_rng(seed, 100, l, 12), (nt * r, d), 0.02, h),
        "B": (_normal(_rng(seed, 100, l, 13), (nt, r, d), b_std, False) if b_std > 0
              else np.zeros((nt, r, d), np.float32)),
    }
    if opt:
        L.update({
            "norm1_b": _normal(_rng(seed, 100, l, 1), (d,), 0.02, h),
            "b_qkv": _normal(_rng(seed, 100, l, 3), (3 * d,), 0.02, h),
            "b_o": _normal(_rng(seed, 100, l, 5), (d,), 0.02, h),
            "norm2_b": _normal(_rng(seed, 100, l, 7), (d,), 0.02, h),
            "b_fc1": _normal(_rng(seed, 100, l, 9), (f1,), 0.02, h),
            "b_fc2": _normal(_rng(seed, 100, l, 11), (d,), 0.02, h),
        })
    return L


def make_decoder_problem(spec: ModelSpec, seed: int = 1234, b_std: float = 0.0, layers=None):
    """Random-init decoder of the given family (globals + every block, or the blocks whose
    indices are listed in ``layers``)."""
    assert spec.arch in (ARCH_OPT, ARCH_LLAMA)
    p = make_decoder_globals(spec, seed)
    p["layers"] = [make_decoder_layer(spec, seed, l, b_std)
                   for l in (range(spec.n_layers) if layers is None else layers)]
    return p


def next_token_labels(tokens: np.ndarray, n_labelled: int) -> np.ndarray:
    """labels[b,t] = tokens[b,t+1] on the last ``n_labelled`` predicting
    positions t in [S-1-n_labelled, S-2]; -1 (ignored) elsewhere."""
    E, S = tokens.shape
    lab = np.full((E, S), -1, np.int32)
    lo = max(0, S - 1 - n_labelled)
    lab[:, lo:S - 1] = tokens[:, lo + 1:S]
    return lab


def label_word_labels(spec: ModelSpec, seed: int) -> np.ndarray:
    """Bernoulli(0.5) class ids at the final position, -1 elsewhere."""
    lab = np.full((spec.E, spec.S), -1, np.int32)
    lab[:, spec.S - 1] = _rng(seed, 21).integers(0, 2, size=spec.E, dtype=np.int32)
    return lab


def make_ragged_batch(spec: ModelSpec, seed: int = 1234, min_frac: float = 0.25):
    """Variable-length stand-in for tokenised task prompts: E sequences with lengths uniform in
    [max(2, min_frac*S), S], uniform random token ids; labels as for the fixed-length batches (the last
    `n_labelled` predicting positions of each sequence, or the class id at its final position).
    Returns (list of int32 token arrays, list of int32 label arrays)."""
    rng = _rng(seed, 30)
    lo = max(2, int(min_frac * spec.S))
    lens = rng.integers(lo, spec.S + 1, size=spec.E)
    toks, labs = [], []
    for b, n in enumerate(lens):
        t = rng.integers(0, spec.vocab, size=int(n), dtype=np.int32)
        if spec.loss_kind == LOSS_CE_LABEL_WORDS:
            l = np.full(int(n), -1, np.int32)
            l[-1] = rng.integers(0, 2)
        else:
            l = next_token_labels(t[None], min(spec.n_labelled, int(n) - 1))[0]
        toks.append(t)
        labs.append(l)
    return toks, labs
