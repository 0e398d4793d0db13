"""GPU parity: the CUDA library through its C ABI against the CPU oracle, element by element,
on the same seeded inputs.  Tolerances: perturbation words bit-exact; fp32 mode losses 1e-4
relative, projected gradients 1e-2 relative, updated B 1e-3 relative to the update; bf16 mode
losses 2e-2 relative."""
import numpy as np
import pytest

import oracle
from oracle.philox import perturbation, perturbation_u32
from workloads import ModelSpec, config
from workloads.spec import (ARCH_LLAMA, ARCH_OPT, LOSS_CE_FULL, LOSS_CE_LABEL_WORDS, TARGET_K,
                            TARGET_Q, TARGET_V)

from gpu_util import make_problem, old_B, run_gpu, run_oracle, update_rel_err

pytestmark = pytest.mark.gpu

SIMT = 1  # ZO_FLAG_SIMT_GEMM
PAIR = 2  # ZO_FLAG_GEMM_PAIR
SINGLE = 8  # ZO_FLAG_GEMM_SINGLE
LORA_EPI = 4  # ZO_FLAG_LORA_EPILOGUE


def test_perturbation_words_bit_exact_and_normals_close():
    import paper_2409_15520_b200 as zo
    for seed, tensor, query, n in [(1, 0, 0, 4096), (0xDEADBEEFCAFEF00D, 63, 15, 1003), (7, 5, 2, 1)]:
        u, z = zo.perturbation(seed, tensor, query, n)
        assert np.array_equal(u, perturbation_u32(seed, tensor, query, n))
        ref = perturbation(seed, tensor, query, (n,))
        assert np.max(np.abs(z - ref)) <= 4e-7 * max(1.0, np.max(np.abs(ref)))


def _check_fp32(spec, seed, b_std, q=None, eps=None, lr=None, tol_g=1e-2, **kw):
    p, tok, lab = make_problem(spec, b_std=b_std)
    ref = run_oracle(spec, p, tok, lab, seed, q, eps, lr)
    got = run_gpu(spec, p, seed, q, eps, lr, **kw)
    assert np.allclose(got["losses"], ref["losses"], rtol=1e-4, atol=0), (got["losses"], ref["losses"])
    scale = np.max(np.abs(ref["g"]))
    assert np.all(np.abs(got["g"] - ref["g"]) <= tol_g * scale), (got["g"], ref["g"])
    assert update_rel_err(spec, p, got["B"], ref["B"]) < 1e-3
    return got, ref


def test_linear_fp32_config():
    """The single MP-LoRA linear + MSE configuration, B = 0 and mid-training B."""
    spec = config("linear_fp32")
    _check_fp32(spec, seed=1, b_std=0.0)
    _check_fp32(spec, seed=2, b_std=0.02)
    _check_fp32(spec, seed=3, b_std=0.02, host=True)


def test_linear_fp32_ragged_shapes_and_scale():
    spec = config("linear_fp32", d_model=40, d_out=20, lora_rank=3, E=1, S=37, q=5, lora_scale=2.0)
    _check_fp32(spec, seed=5, b_std=0.05)
    spec = config("linear_fp32", d_model=8, d_out=4, lora_rank=1, E=1, S=1, q=1)
    _check_fp32(spec, seed=6, b_std=0.05)


TINY = dict(n_layers=2, d_model=64, n_heads=4, d_ffn=96, vocab=131, max_seq=24, lora_rank=4,
            E=3, S=24, q=3, n_labelled=5, eps=1e-2, lr=1e-2)


@pytest.mark.parametrize("arch,targets,loss", [
    (ARCH_OPT, TARGET_Q | TARGET_V, LOSS_CE_FULL),
    (ARCH_LLAMA, TARGET_Q | TARGET_V, LOSS_CE_FULL),
    (ARCH_LLAMA, TARGET_Q | TARGET_K | TARGET_V, LOSS_CE_FULL),
    (ARCH_OPT, TARGET_V, LOSS_CE_LABEL_WORDS),
])
def test_decoder_fp32(arch, targets, loss):
    spec = ModelSpec(arch=arch, lora_targets=targets, loss_kind=loss, label_words=(7, 90),
                     tie_lm_head=(arch == ARCH_OPT), bf16=False, lora_scale=2.0,
                     **{**TINY, "n_labelled": 1 if loss == LOSS_CE_LABEL_WORDS else 5})
    got, ref = _check_fp32(spec, seed=11, b_std=0.05)
    # per labelled-row losses as well
    p, tok, lab = make_problem(spec, b_std=0.05)
    z = [oracle.zo.draw_z(spec, p, 11, i) for i in range(spec.q)]
    Bn = [np.stack([np.asarray(L["B"], np.float64) + (1 if n % 2 == 0 else -1) * spec.eps * z[n // 2][l]
                    for n in range(2 * spec.q)]) for l, L in enumerate(p["layers"])]
    _, rows = oracle.replica_losses(spec, p, Bn, tok, lab, return_rows=True)
    assert np.allclose(got["rows"].reshape(rows.shape), rows, rtol=2e-4)


def test_decoder_fp32_head_dims_and_ragged_sequence():
    for dh, S, E in [(32, 7, 2), (64, 70, 1), (128, 65, 1)]:
        spec = ModelSpec(arch=ARCH_LLAMA, bf16=False, **{**TINY, "d_model": 2 * dh, "n_heads": 2,
                                                         "S": S, "E": E, "max_seq": S,
                                                         "n_layers": 1, "q": 2})
        _check_fp32(spec, seed=4, b_std=0.05)


@pytest.mark.parametrize("flags", [SIMT, 0, PAIR])
@pytest.mark.parametrize("arch", [ARCH_OPT, ARCH_LLAMA])
def test_decoder_bf16(arch, flags):
    """bf16 storage; flags=SIMT runs the validation GEMM, 0 the tensor-core path.
    T = 3*40 = 120 (< one 128-row tile) and d = 64 (< one 256-column tile)."""
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=True,
                     **{**TINY, "S": 40, "max_seq": 40})
    p, tok, lab = make_problem(spec, b_std=0.05)
    ref = run_oracle(spec, p, tok, lab, 21)
    got = run_gpu(spec, p, 21, flags=flags)
    assert np.allclose(got["losses"], ref["losses"], rtol=2e-2, atol=0), (got["losses"], ref["losses"])


@pytest.mark.parametrize("arch", [ARCH_OPT, ARCH_LLAMA])
def test_decoder_bf16_tensor_core_multi_tile(arch):
    """Several row tiles per replica and several column tiles with ragged tails:
    T = 2*160 = 320 -> padded 384 rows per replica, d = 320, ffn = 328, vocab = 1003."""
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=True,
                     **{**TINY, "d_model": 320, "n_heads": 5, "d_ffn": 328, "vocab": 1003,
                        "S": 160, "E": 2, "max_seq": 160, "q": 2, "lora_rank": 8, "n_labelled": 7})
    p, tok, lab = make_problem(spec, b_std=0.05)
    ref = run_oracle(spec, p, tok, lab, 31)
    got = run_gpu(spec, p, 31)
    simt = run_gpu(spec, p, 31, flags=SIMT)
    pair = run_gpu(spec, p, 31, flags=PAIR)
    assert np.allclose(got["losses"], ref["losses"], rtol=2e-2, atol=0), (got["losses"], ref["losses"])
    # CTA-pair and single-CTA tensor-core kernels accumulate in the same order: bit-identical
    assert np.array_equal(got["losses"], pair["losses"]) and np.array_equal(got["rows"], pair["rows"])
    # the two bf16 GEMM implementations agree far more closely with each other
    assert np.allclose(got["losses"], simt["losses"], rtol=2e-3, atol=0), (got["losses"], simt["losses"])
    assert np.allclose(got["rows"], simt["rows"], rtol=0, atol=0.05)


@pytest.mark.parametrize("vocab", [5000, 4100, 64])
def test_full_vocab_loss_vector_path(vocab):
    """Vocabularies that are a multiple of 4 take the 16-byte-load form of the log-softmax reduction:
    5000 runs the four-loads-in-flight body once plus single chunks, 4100 the body and a one-chunk
    tail in a few lanes only, 64 leaves most lanes of the block without any element.  fp32 mode, so
    the 1e-4 loss tolerance applies; per-row losses are checked too."""
    spec = ModelSpec(arch=ARCH_LLAMA, bf16=False, **{**TINY, "vocab": vocab, "q": 2})
    p, tok, lab = make_problem(spec, b_std=0.05)
    ref = run_oracle(spec, p, tok, lab, 23)
    got = run_gpu(spec, p, 23)
    assert np.allclose(got["losses"], ref["losses"], rtol=1e-4, atol=0), (got["losses"], ref["losses"])
    assert np.all(np.abs(got["g"] - ref["g"]) <= 1e-2 * np.abs(ref["g"]).max())
    assert update_rel_err(spec, p, got["B"], ref["B"]) < 1e-3
    seq = run_gpu(spec, p, 23, schedule="sequential")
    assert np.array_equal(seq["losses"], got["losses"]) and np.array_equal(seq["rows"], got["rows"])


@pytest.mark.parametrize("arch,bf16,d,heads", [(ARCH_OPT, True, 768, 12), (ARCH_OPT, False, 384, 6),
                                               (ARCH_LLAMA, False, 384, 3), (ARCH_LLAMA, True, 1536, 12),
                                               (ARCH_LLAMA, True, 5120, 40)])
def test_decoder_wide_rows_block_norm(arch, bf16, d, heads):
    """Rows wider than one warp's 64 vectors: the one-block-per-row norm (LayerNorm with bias and
    RMSNorm, both precisions, two and three vectors per thread) instead of the warp-per-row kernel."""
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=bf16,
                     **{**TINY, "d_model": d, "n_heads": heads, "d_ffn": 256, "vocab": 211, "S": 24,
                        "E": 2, "max_seq": 24, "q": 2, "n_layers": 1 if d > 2048 else 2, "lora_rank": 4})
    if not bf16:
        _check_fp32(spec, seed=19, b_std=0.05)
        return
    p, tok, lab = make_problem(spec, b_std=0.05)
    ref = run_oracle(spec, p, tok, lab, 19)
    got = run_gpu(spec, p, 19)
    assert np.allclose(got["losses"], ref["losses"], rtol=2e-2, atol=0), (got["losses"], ref["losses"])


@pytest.mark.parametrize("arch,q", [(ARCH_LLAMA, 1), (ARCH_OPT, 1)])
def test_decoder_bf16_small_batch_split_k(arch, q):
    """One short sequence and one query (256 rows per pass) with k_in = 512 and 1024: too few tiles
    for the SMs, so the tensor-core GEMMs cut K into units of work that store fp32 parts, and a second
    launch sums the parts in K order and runs the fused epilogue (bias, residual, rotary embedding;
    the LoRA k-block rides with the first part).  Checked against the oracle and the CUDA-core GEMM,
    and for run-to-run bit-identity."""
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=True,
                     **{**TINY, "d_model": 512, "n_heads": 4, "d_ffn": 1024, "vocab": 517, "S": 40,
                        "E": 1, "max_seq": 40, "q": q, "n_layers": 2, "lora_rank": 8})
    p, tok, lab = make_problem(spec, b_std=0.05)
    ref = run_oracle(spec, p, tok, lab, 47)
    got = run_gpu(spec, p, 47)
    again = run_gpu(spec, p, 47)
    simt = run_gpu(spec, p, 47, flags=SIMT)
    assert np.allclose(got["losses"], ref["losses"], rtol=2e-2, atol=0), (got["losses"], ref["losses"])
    assert np.allclose(got["losses"], simt["losses"], rtol=3e-3, atol=0), (got["losses"], simt["losses"])
    assert np.array_equal(got["losses"], again["losses"]) and np.array_equal(got["rows"], again["rows"])
    assert np.array_equal(got["B"][0], again["B"][0])


@pytest.mark.parametrize("arch,S", [(ARCH_LLAMA, 100), (ARCH_OPT, 64), (ARCH_LLAMA, 1), (ARCH_LLAMA, 300)])
def test_decoder_bf16_head_dim_128(arch, S):
    """Tensor-core attention with head_dim 128 (rotary embedding applied while staging), ragged
    and single-token sequences; compared with the oracle and with the CUDA-core attention."""
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=True,
                     **{**TINY, "d_model": 256, "n_heads": 2, "d_ffn": 264, "vocab": 517, "S": S,
                        "E": 2, "max_seq": max(S, 2), "q": 2, "n_layers": 2,
                        "n_labelled": 1 if S == 1 else 5})
    p, tok, lab = make_problem(spec, b_std=0.05)
    if S == 1:                       # a one-token sequence has no next token: label the token itself
        lab = tok.copy()
        p["labels"] = lab
    ref = run_oracle(spec, p, tok, lab, 41)
    got = run_gpu(spec, p, 41)
    simt = run_gpu(spec, p, 41, flags=SIMT)
    assert np.allclose(got["losses"], ref["losses"], rtol=2e-2, atol=0), (got["losses"], ref["losses"])
    assert np.allclose(got["losses"], simt["losses"], rtol=2e-3, atol=0), (got["losses"], simt["losses"])


def _mp_lora_linear_case(x_replicated, r, T, ki, ko, q, pair_identical=True):
    """Runs the MP-LoRA layer on its own through every GEMM implementation and checks it against the
    oracle's layer: the outputs, and the difference of every +/- replica pair (which isolates the
    perturbation term: its sign, its query index and its scale)."""
    import torch
    import paper_2409_15520_b200 as zo
    from workloads import bf16_round
    rng = np.random.default_rng(r + x_replicated)
    eps, scale, seed, tid = 1e-2, 2.0, 77, 3
    n = 2 * q
    X = bf16_round(rng.standard_normal((n if x_replicated else 1, T, ki)).astype(np.float32))
    W = bf16_round(0.05 * rng.standard_normal((ko, ki)).astype(np.float32))
    bias = bf16_round(0.05 * rng.standard_normal(ko).astype(np.float32))
    A = bf16_round(0.05 * rng.standard_normal((r, ki)).astype(np.float32))
    B = (0.05 * rng.standard_normal((r, ko))).astype(np.float32)
    Bn = np.stack([B.astype(np.float64) + (1 if i % 2 == 0 else -1) * eps * perturbation(seed, tid, i // 2, (r, ko))
                   for i in range(n)])
    Xn = np.broadcast_to(X, (n, T, ki)).astype(np.float64)
    ref = oracle.mp_lora_linear(Xn, W, bias, A, Bn, scale)
    dev = lambda a: torch.tensor(a, device="cuda").to(torch.bfloat16).contiguous()
    Bd = torch.tensor(B, device="cuda")
    outs = {}
    for flags in (0, SIMT, PAIR):
        Y = zo.mp_lora_linear(dev(X.reshape(-1, ki)), dev(W), dev(bias), dev(A), Bd, T, q, scale, seed,
                              tid, eps, x_replicated, flags=flags)
        outs[flags] = Y.float().cpu().numpy().astype(np.float64)
        err = np.max(np.abs(outs[flags] - ref))
        assert err < 2e-2 * np.max(np.abs(ref)), (flags, err, np.max(np.abs(ref)))
    if pair_identical:     # CTA-pair and single-CTA kernels accumulate in the same order
        assert np.array_equal(outs[0], outs[PAIR])
    # the perturbation must be visible in the outputs: replicas 2i and 2i+1 differ as the oracle's do
    for i in range(q):
        d_gpu, d_ref = outs[0][2 * i] - outs[0][2 * i + 1], ref[2 * i] - ref[2 * i + 1]
        assert np.max(np.abs(d_ref)) > 0
        assert np.max(np.abs(d_gpu - d_ref)) < 0.1 * np.max(np.abs(d_ref)) + 2 * 2.0 ** -8 * np.max(np.abs(ref))
    return outs


@pytest.mark.parametrize("x_replicated", [0, 1])
@pytest.mark.parametrize("r", [8, 16, 64])
def test_mp_lora_linear_bf16_tensor_core(x_replicated, r):
    """The MP-LoRA layer equation on its own, both input modes, against the oracle's layer (k_out is
    not a multiple of the column tiles: the low-rank term runs in the GEMM epilogue or in the
    CUDA-core expansion)."""
    _mp_lora_linear_case(x_replicated, r, T=256, ki=328, ko=544, q=2)


@pytest.mark.parametrize("r", [5, 8, 12, 16, 32, 64])
def test_mp_lora_linear_shared_input_expansion(r):
    """Shared input with k_out a multiple of 128: the expansion kernels (operand generated once per
    replica and column tile, warp-level tensor-core product) for every rank class: the bulk-tensor
    form with the duplicated operand half in shared registers (8, 16) and with the element-wise
    gather (5, 12: not a multiple of 8), the cp.async form (32, 64); a ragged last row tile (T = 200:
    the last tile has 72 rows, so one warp's box is clipped by the store and one is skipped)."""
    outs = _mp_lora_linear_case(0, r, T=200, ki=328, ko=384, q=3)
    # the CUDA-core expansion computes the same sums in fp32 from unrounded operands: the two agree to bf16 rounding
    assert np.max(np.abs(outs[0] - outs[SIMT])) < 2.0 ** -6 * np.max(np.abs(outs[SIMT]))


@pytest.mark.parametrize("r", [8, 64])
def test_mp_lora_linear_replicated_input_slab(r):
    """Replicated input with k_out a multiple of 256 and T of 128: the low-rank term as generated
    tensor-core k-blocks (one for r <= 32, two above).  The CTA-pair kernel keeps the low-rank term in
    its epilogue (fp32 from unrounded operands), so the two agree to bf16 rounding only."""
    outs = _mp_lora_linear_case(1, r, T=256, ki=328, ko=512, q=2, pair_identical=False)
    assert np.max(np.abs(outs[0] - outs[PAIR])) < 2.0 ** -6 * np.max(np.abs(outs[PAIR]))
    if r <= 32:
        # a replica is a whole 256-row tile here, so the pair kernel runs the one-block tensor-core form
        # too (each CTA generates the operand rows of its half): same operands, same order, same bits
        assert np.array_equal(outs[0], outs[PAIR])


@pytest.mark.parametrize("arch", [ARCH_LLAMA, ARCH_OPT])
def test_decoder_pair_kernel_with_tensor_core_lora_block(arch):
    """256 rows per replica and d = 256: under ZO_FLAG_GEMM_PAIR the q|k|v launch runs CTA pairs with the
    low-rank term as a generated k-block and (Llama) the rotary embedding in its epilogue.  Same bits
    as the single-CTA kernels; the oracle within the bf16 tolerance."""
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=True,
                     **{**TINY, "d_model": 256, "n_heads": 2, "d_ffn": 512, "vocab": 517, "S": 128, "E": 2,
                        "max_seq": 128, "q": 2, "lora_rank": 8, "n_layers": 3, "n_labelled": 6})
    p, tok, lab = make_problem(spec, b_std=0.05)
    ref = run_oracle(spec, p, tok, lab, 13)
    got = run_gpu(spec, p, 13)
    pair = run_gpu(spec, p, 13, flags=PAIR)
    assert np.allclose(pair["losses"], ref["losses"], rtol=2e-2, atol=0), (pair["losses"], ref["losses"])
    assert np.array_equal(got["losses"], pair["losses"]) and np.array_equal(got["rows"], pair["rows"])
    assert all(np.array_equal(a, b) for a, b in zip(got["B"], pair["B"]))


def test_automatic_tile_shape_matches_both_forced_shapes():
    """A base product large enough for the default dispatch to pick CTA pairs (16384 shared rows x 2560
    columns = 640 tiles of 256 x 256, more than eight waves of pairs): the default, the forced single-CTA
    and the forced pair kernels return the same bits, and the oracle's layer within bf16 rounding on a
    sample of rows (ragged K: 72 is not a multiple of the 64-deep k-block)."""
    import torch
    import paper_2409_15520_b200 as zo
    from workloads import bf16_round
    rng = np.random.default_rng(3)
    T, ki, ko, r, q = 16384, 72, 2560, 8, 1
    eps, scale, seed, tid = 1e-2, 1.0, 5, 2
    X = bf16_round(rng.standard_normal((T, ki)).astype(np.float32))
    W = bf16_round(0.05 * rng.standard_normal((ko, ki)).astype(np.float32))
    A = bf16_round(0.05 * rng.standard_normal((r, ki)).astype(np.float32))
    B = (0.05 * rng.standard_normal((r, ko))).astype(np.float32)
    dev = lambda a: torch.tensor(a, device="cuda").to(torch.bfloat16).contiguous()
    outs = {f: zo.mp_lora_linear(dev(X), dev(W), None, dev(A), torch.tensor(B, device="cuda"), T, q, scale, seed,
                                 tid, eps, 0, flags=f).float().cpu().numpy() for f in (0, SINGLE, PAIR)}
    assert np.array_equal(outs[0], outs[SINGLE]) and np.array_equal(outs[0], outs[PAIR])
    rows = np.r_[0:3, 127:130, 255:258, 4095:4098, T - 3:T]
    Bn = np.stack([B.astype(np.float64) + k * eps * perturbation(seed, tid, 0, (r, ko)) for k in (1, -1)])
    ref = oracle.mp_lora_linear(np.broadcast_to(X[rows], (2, len(rows), ki)).astype(np.float64), W, None, A, Bn, scale)
    assert np.max(np.abs(outs[0][:, rows] - ref)) < 2.0 ** -7 * np.max(np.abs(ref))


@pytest.mark.parametrize("bf16", [False, True])
def test_schedules_give_the_same_step(bf16):
    """Outer-only, inner-only and sequential cuts of the step (the paper's ablation of its two
    parallelisations) reproduce the single-pass step: same losses, projected gradients and update."""
    spec = ModelSpec(arch=ARCH_LLAMA, bf16=bf16, **{**TINY, "d_model": 128, "n_heads": 2, "S": 40,
                                                   "max_seq": 40, "q": 3})
    p, tok, lab = make_problem(spec, b_std=0.05)
    full = run_gpu(spec, p, 17)
    ref = run_oracle(spec, p, tok, lab, 17)
    assert np.allclose(full["losses"], ref["losses"], rtol=2e-2 if bf16 else 1e-4)
    for sched in ("outer_only", "inner_only", "sequential"):
        got = run_gpu(spec, p, 17, schedule=sched)
        assert np.array_equal(got["losses"], full["losses"]), sched
        assert np.array_equal(got["g"], full["g"]), sched
        assert np.array_equal(got["rows"], full["rows"]), sched
        assert all(np.array_equal(a, b) for a, b in zip(got["B"], full["B"])), sched
        assert got["launches"] > full["launches"]
    lin = config("linear_fp32", q=3)
    pl, _, _ = make_problem(lin, b_std=0.02)
    a = run_gpu(lin, pl, 4)
    for sched in ("outer_only", "inner_only", "sequential"):
        b = run_gpu(lin, pl, 4, schedule=sched)
        assert np.array_equal(a["losses"], b["losses"]) and np.array_equal(a["B"][0], b["B"][0])


@pytest.mark.parametrize("x_replicated", [1, 0])
@pytest.mark.parametrize("r", [4, 16, 24, 32, 48, 64])
def test_mp_lora_linear_tensor_core_lora_block(r, x_replicated):
    """k_out a multiple of the 256-column tile: the low-rank term runs as one (rank <= 32) or two
    extra tensor-core k-blocks (bf16 U, B and k eps z); with a shared input the expansion to the 2q
    outputs is a GEMM made of those blocks alone.  Checked against the oracle's
    layer, against the CUDA-core epilogue form, and for the visibility of the perturbation when
    |B| is 100x larger than eps."""
    import torch
    import paper_2409_15520_b200 as zo
    from workloads import bf16_round
    rng = np.random.default_rng(r)
    T, ki, ko, q, eps, scale, seed, tid = 256, 192, 768, 3, 1e-3, 2.0, 91, 5
    n = 2 * q
    X = bf16_round(rng.standard_normal((n if x_replicated else 1, T, ki)).astype(np.float32))
    W = bf16_round(0.05 * rng.standard_normal((ko, ki)).astype(np.float32))
    A = bf16_round(0.05 * rng.standard_normal((r, ki)).astype(np.float32))
    B = (0.1 * rng.standard_normal((r, ko))).astype(np.float32)
    Bn = np.stack([B.astype(np.float64) + (1 if i % 2 == 0 else -1) * eps * perturbation(seed, tid, i // 2, (r, ko))
                   for i in range(n)])
    ref = oracle.mp_lora_linear(np.broadcast_to(X, (n, T, ki)).astype(np.float64), W, None, A, Bn, scale)
    dev = lambda a: torch.tensor(a, device="cuda").to(torch.bfloat16).contiguous()
    Bd = torch.tensor(B, device="cuda")
    outs = {}
    for flags in (0, LORA_EPI):
        Y = zo.mp_lora_linear(dev(X.reshape(-1, ki)), dev(W), None, dev(A), Bd, T, q, scale, seed, tid, eps,
                              x_replicated, flags=flags)
        outs[flags] = Y.float().cpu().numpy().astype(np.float64)
        assert np.max(np.abs(outs[flags] - ref)) < 2e-2 * np.max(np.abs(ref)), flags
    assert np.max(np.abs(outs[0] - outs[LORA_EPI])) < 1e-2 * np.max(np.abs(ref))
    # +/- replicas of one query differ by 2 eps s U z: compare with the exact difference, before the
    # bf16 rounding of the outputs swamps it, by averaging over rows (the rounding is unbiased)
    d_ref = (ref[0] - ref[1]).mean(axis=0)
    d_gpu = (outs[0][0] - outs[0][1]).mean(axis=0)
    assert np.abs(d_ref).max() > 0
    assert np.abs(d_gpu - d_ref).max() < 0.25 * np.abs(d_ref).max() + 2.0 ** -8 * np.abs(ref).max() / np.sqrt(T) * 4


def test_degenerate_steps():
    spec = ModelSpec(arch=ARCH_OPT, tie_lm_head=True, bf16=False, **TINY)
    p, tok, lab = make_problem(spec, b_std=0.05)
    got = run_gpu(spec, p, 3, eps=0.0)                     # eps = 0: identical replicas, no update
    assert np.all(got["losses"] == got["losses"][0]) and np.all(got["g"] == 0)
    assert all(np.array_equal(a, b) for a, b in zip(got["B"], [b.astype(np.float32) for b in old_B(spec, p)]))
    ref = run_oracle(spec, p, tok, lab, 3, eps=0.0)
    assert np.allclose(got["losses"], ref["losses"], rtol=1e-4)
    got = run_gpu(spec, p, 3, lr=0.0)                      # lr = 0: g but no update
    assert np.any(got["g"] != 0)
    assert all(np.array_equal(a, b) for a, b in zip(got["B"], [b.astype(np.float32) for b in old_B(spec, p)]))
    p0, _, _ = make_problem(spec, b_std=0.0)               # B = 0: first step of a fine-tuning run
    ref = run_oracle(spec, p0, tok, lab, 3)
    got = run_gpu(spec, p0, 3)
    assert np.allclose(got["losses"], ref["losses"], rtol=1e-4)
    assert update_rel_err(spec, p0, got["B"], ref["B"]) < 2e-3


@pytest.mark.parametrize("heads,targets", [(2, TARGET_Q | TARGET_V), (4, TARGET_Q | TARGET_K | TARGET_V),
                                           (8, TARGET_V), (16, TARGET_Q | TARGET_V), (4, 0)])
def test_llama_bf16_fused_rope_all_head_dims(heads, targets):
    """d = 256 (one 256-column tile per section): the rotary embedding is applied in the epilogue of the
    q|k|v GEMM for head_dim 128, 64 (pairs in different 32-column chunks), 32 and 16 (pairs inside a
    chunk), with adapted q/k/v sections in any combination and with no adapted section at all."""
    spec = ModelSpec(arch=ARCH_LLAMA, bf16=True, lora_targets=targets,
                     **{**TINY, "d_model": 256, "n_heads": heads, "d_ffn": 264, "vocab": 517, "S": 72,
                        "E": 2, "max_seq": 72, "q": 2, "n_layers": 2, "lora_rank": 8})
    p, tok, lab = make_problem(spec, b_std=0.05)
    ref = run_oracle(spec, p, tok, lab, 43)
    got = run_gpu(spec, p, 43)
    simt = run_gpu(spec, p, 43, flags=SIMT)
    assert np.allclose(got["losses"], ref["losses"], rtol=2e-2, atol=0), (got["losses"], ref["losses"])
    assert np.allclose(got["losses"], simt["losses"], rtol=3e-3, atol=0), (got["losses"], simt["losses"])


def test_maximum_queries_and_no_labelled_positions():
    """q = 32 (64 replicas, the largest the library accepts) on a small model in both precisions;
    a batch without any labelled position gives zero losses and leaves B untouched."""
    for bf16 in (False, True):
        spec = ModelSpec(arch=ARCH_OPT, tie_lm_head=True, bf16=bf16,
                         **{**TINY, "q": 32, "E": 1, "S": 9, "max_seq": 9, "n_layers": 1, "n_labelled": 2})
        p, tok, lab = make_problem(spec, b_std=0.05)
        ref = run_oracle(spec, p, tok, lab, 13)
        got = run_gpu(spec, p, 13)
        assert got["losses"].shape == (64,)
        assert np.allclose(got["losses"], ref["losses"], rtol=2e-2 if bf16 else 1e-4)
        if not bf16:
            assert np.all(np.abs(got["g"] - ref["g"]) <= 1e-2 * np.abs(ref["g"]).max())
    spec = ModelSpec(arch=ARCH_LLAMA, bf16=False, **TINY)
    p, tok, lab = make_problem(spec, b_std=0.05)
    p["labels"] = np.full_like(lab, -1)
    got = run_gpu(spec, p, 2)
    assert np.all(got["losses"] == 0) and np.all(got["g"] == 0)
    assert all(np.array_equal(a, b.astype(np.float32)) for a, b in zip(got["B"], old_B(spec, p)))


def test_argument_errors_are_reported_not_faulted():
    import ctypes as C
    import paper_2409_15520_b200 as zo
    from paper_2409_15520_b200 import binding as b
    spec = ModelSpec(arch=ARCH_OPT, tie_lm_head=True, bf16=False, **TINY)
    p, tok, lab = make_problem(spec)
    cfg = zo.make_config(spec)
    est = zo.Estimator(cfg)
    prob = zo.DeviceProblem(p, False)
    for kw, code in [(dict(q=0), 1), (dict(q=spec.q + 1), 1), (dict(E=spec.E + 1), 1), (dict(E=0), 1), (dict(S=0), 1),
                     (dict(S=spec.max_seq + 1), 1), (dict(eps=-1.0), 1), (dict(eps=float("nan")), 1)]:
        a = dict(E=spec.E, S=spec.S, seed=1, q=spec.q, eps=1e-3, lr=1e-3)
        a.update(kw)
        with pytest.raises(zo.ZoError) as ei:
            est.step(prob, **a)
        assert ei.value.status == code
    with pytest.raises(zo.ZoError) as ei:
        est.losses()
    assert ei.value.status == 7                             # ZO_ERR_STATE: no step yet
    # too many labelled positions for max_labelled -> deferred ZO_ERR_INVALID_ARG, B untouched
    import torch
    bad = torch.zeros_like(prob.labels)
    est.step(prob, spec.E, spec.S, 1, spec.q, 1e-3, 1e-3, labels=bad)
    with pytest.raises(zo.ZoError) as ei:
        est.losses()
    assert ei.value.status == 1
    assert all(np.array_equal(a, c.astype(np.float32)) for a, c in zip(prob.B_numpy(), old_B(spec, p)))
    est.step(prob, spec.E, spec.S, 1, spec.q, 1e-3, 1e-3)  # the context is still usable
    est.losses()
    bad_cfg = zo.make_config(spec.with_(n_heads=5))
    assert b.zo_workspace_bytes(C.byref(bad_cfg)) == 0
    with pytest.raises(zo.ZoError) as ei:
        zo.Estimator(bad_cfg)
    assert ei.value.status == 2


@pytest.mark.parametrize("arch", [ARCH_OPT, ARCH_LLAMA])
def test_decoder_fp32_at_the_configured_eps(arch):
    """The named configurations state eps = 1e-3 (the decoder cases above run the paper's MobiZO
    setting, 1e-2).  The loss difference of a query is then ten times smaller against the same fp32
    rounding of the losses; measured on a B200: g within 5e-4 (OPT) and 6e-5 (Llama) of max|g|."""
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=False, lora_scale=2.0, **{**TINY, "eps": 1e-3})
    p, tok, lab = make_problem(spec, b_std=0.05)
    ref = run_oracle(spec, p, tok, lab, 11)
    got = run_gpu(spec, p, 11)
    rel_g = np.max(np.abs(got["g"] - ref["g"])) / np.max(np.abs(ref["g"]))
    print(f"fp32 decoder arch={arch} eps=1e-3: max|dg|/max|g| = {rel_g:.2e}, update err {update_rel_err(spec, p, got['B'], ref['B']):.2e}")
    assert np.allclose(got["losses"], ref["losses"], rtol=1e-4, atol=0)
    assert rel_g < 1e-2
    assert update_rel_err(spec, p, got["B"], ref["B"]) < 1e-3


@pytest.mark.parametrize("arch,vocab,flags", [(ARCH_LLAMA, 1003, 0), (ARCH_OPT, 517, 0), (ARCH_OPT, 1003, PAIR),
                                              (ARCH_LLAMA, 256, 0), (ARCH_LLAMA, 70, 0)])
def test_fused_head_loss_matches_stored_logits(arch, vocab, flags):
    """bf16 mode folds the LM-head tile into (max, sum of exp) pairs inside the GEMM epilogue; with
    ZO_FLAG_CE_LOGITS the logits are stored and reduced by the stand-alone kernel.  Same accumulators,
    another summation order: per-row losses agree to fp32 rounding, both stay within the bf16 tolerance
    of the oracle.  Vocabularies with a ragged last column tile, exactly one tile, and less than one
    32-column chunk; single-CTA and CTA-pair kernels."""
    CE_LOGITS = 32
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=True,
                     **{**TINY, "d_model": 256, "n_heads": 4, "d_ffn": 512, "vocab": vocab, "S": 80, "E": 4,
                        "max_seq": 80, "q": 2, "n_labelled": 7, "lora_rank": 8})
    p, tok, lab = make_problem(spec, b_std=0.05)
    ref = run_oracle(spec, p, tok, lab, 37)
    fused = run_gpu(spec, p, 37, flags=flags)
    stored = run_gpu(spec, p, 37, flags=flags | CE_LOGITS)
    assert np.allclose(fused["losses"], ref["losses"], rtol=2e-2, atol=0), (fused["losses"], ref["losses"])
    assert np.allclose(fused["rows"], stored["rows"], rtol=2e-6, atol=0)
    assert np.allclose(fused["losses"], stored["losses"], rtol=1e-6, atol=0)
    assert fused["launches"] == stored["launches"]
    again = run_gpu(spec, p, 37, flags=flags)
    assert np.array_equal(fused["rows"], again["rows"])     # fixed merge order: same bits from run to run
