"""Causal attention on the tcgen05 path (head_dim 64 / 128, sequences of at most 256 tokens) against the
oracle's step, the warp-level tensor-core kernel (ZO_FLAG_ATTN_WARP_MMA) and the CUDA-core kernel
(ZO_FLAG_SIMT_GEMM): one and two query tiles, ragged tails, a single token, key tiles that end inside a
64-key chunk, several sequences and heads per thread block, packed variable-length batches."""
import numpy as np
import pytest

from workloads import ModelSpec, make_decoder_problem, make_ragged_batch
from workloads.spec import ARCH_LLAMA, ARCH_OPT

from gpu_util import make_problem, run_gpu, run_oracle

pytestmark = pytest.mark.gpu

SIMT, WARP_MMA = 1, 64


@pytest.mark.parametrize("dh", [64, 128])
@pytest.mark.parametrize("S,E", [(1, 2), (37, 3), (64, 2), (128, 2), (129, 2), (200, 1), (256, 2)])
def test_tcgen05_attention_against_oracle_and_other_kernels(dh, S, E):
    arch = ARCH_LLAMA if dh == 128 else ARCH_OPT
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=True, n_layers=2, d_model=2 * dh, n_heads=2,
                     d_ffn=256, vocab=311, max_seq=max(S, 2), lora_rank=4, E=E, S=S, q=2,
                     n_labelled=1 if S == 1 else min(5, S - 1), eps=1e-2, lr=1e-2)
    p, tok, lab = make_problem(spec, b_std=0.05)
    if S == 1:                       # a one-token sequence has no next token: label the token itself
        lab = tok.copy()
        p["labels"] = lab
    ref = run_oracle(spec, p, tok, lab, 41)
    got = run_gpu(spec, p, 41)
    warp = run_gpu(spec, p, 41, flags=WARP_MMA)
    simt = run_gpu(spec, p, 41, flags=SIMT)
    assert np.allclose(got["losses"], ref["losses"], rtol=2e-2, atol=0), (got["losses"], ref["losses"])
    assert np.allclose(got["losses"], warp["losses"], rtol=2e-3, atol=0), (got["losses"], warp["losses"])
    assert np.allclose(got["losses"], simt["losses"], rtol=3e-3, atol=0), (got["losses"], simt["losses"])
    assert np.allclose(got["rows"], warp["rows"], rtol=0, atol=0.05)
    again = run_gpu(spec, p, 41)
    assert np.array_equal(got["rows"], again["rows"])


@pytest.mark.parametrize("dh", [64, 128])
def test_tcgen05_attention_many_jobs_per_block(dh):
    """More (sequence, head) jobs than thread blocks: 8 replicas x 6 sequences x 8 heads = 384 jobs, so every
    persistent block runs several jobs back to back through its rings."""
    spec = ModelSpec(arch=ARCH_LLAMA, bf16=True, n_layers=1, d_model=8 * dh, n_heads=8, d_ffn=256, vocab=311,
                     max_seq=192, lora_rank=4, E=6, S=192, q=4, n_labelled=9, eps=1e-2, lr=1e-2)
    p, tok, lab = make_problem(spec, b_std=0.05)
    ref = run_oracle(spec, p, tok, lab, 5)
    got = run_gpu(spec, p, 5)
    warp = run_gpu(spec, p, 5, flags=WARP_MMA)
    assert np.allclose(got["losses"], ref["losses"], rtol=2e-2, atol=0), (got["losses"], ref["losses"])
    assert np.allclose(got["rows"], warp["rows"], rtol=0, atol=0.05)


@pytest.mark.parametrize("dh", [64, 128])
def test_tcgen05_attention_packed_variable_length(dh):
    import torch
    import paper_2409_15520_b200 as zo
    spec = ModelSpec(arch=ARCH_LLAMA, bf16=True, n_layers=2, d_model=2 * dh, n_heads=2, d_ffn=192, vocab=211,
                     max_seq=230, lora_rank=4, E=5, S=230, q=2, n_labelled=4, eps=1e-2, lr=1e-2)
    p = make_decoder_problem(spec, seed=4, b_std=0.05)
    toks, labs = make_ragged_batch(spec, seed=6)
    ref = run_oracle(spec, p, toks, labs, 19)
    outs = {}
    for flags in (0, WARP_MMA):
        est, prob = zo.Estimator(zo.make_config(spec, flags=flags)), zo.DeviceProblem(p, True)
        cu = np.concatenate([[0], np.cumsum([len(t) for t in toks])]).astype(np.int32)
        dev = lambda a: torch.tensor(np.ascontiguousarray(a), dtype=torch.int32, device="cuda")
        est.step_varlen(prob, dev(np.concatenate(toks)), dev(np.concatenate(labs)), dev(cu), spec.S, 19, spec.q,
                        spec.eps, spec.lr)
        outs[flags] = est.losses()[0].astype(np.float64)
        est.close()
    assert np.allclose(outs[0], ref["losses"], rtol=2e-2, atol=0), (outs[0], ref["losses"])
    assert np.allclose(outs[0], outs[WARP_MMA], rtol=2e-3, atol=0)
