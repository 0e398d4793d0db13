"""GPU parity for weight-only quantised frozen weights (INT8 / NF4): the decoder is bit-exact against the
oracle's, and a step on a quantised checkpoint matches the oracle's step on the same stored bytes."""
import ctypes as C

import numpy as np
import pytest

from oracle import quant as oq
from workloads import ModelSpec, make_decoder_problem, quantize_int8, quantize_layer, quantize_nf4
from workloads.spec import ARCH_LLAMA, ARCH_OPT

from gpu_util import run_gpu, run_oracle, update_rel_err

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fmt", ["int8", "nf4"])
@pytest.mark.parametrize("bf16", [True, False])
def test_dequantize_bit_exact(fmt, bf16):
    import torch
    from paper_2409_15520_b200 import binding as b
    rng = np.random.default_rng(3)
    rows, K = 37, 192
    w = (0.05 * rng.standard_normal((rows, K))).astype(np.float32)
    codes, scale = (quantize_int8 if fmt == "int8" else quantize_nf4)(w)
    ref = (oq.dequant_int8 if fmt == "int8" else oq.dequant_nf4)(codes, scale, bf16)
    dc = torch.tensor(codes, device="cuda").contiguous()
    ds = torch.tensor(scale, device="cuda").contiguous()
    out = torch.empty((rows, K), dtype=torch.bfloat16 if bf16 else torch.float32, device="cuda")
    st = b.zo_dequantize(C.c_void_p(torch.cuda.current_stream().cuda_stream), b.WEIGHT_FORMATS[fmt], int(bf16),
                         C.c_void_p(dc.data_ptr()), C.c_void_p(ds.data_ptr()), C.c_void_p(out.data_ptr()), rows, K)
    assert st == 0
    torch.cuda.synchronize()
    assert np.array_equal(out.float().cpu().numpy().astype(np.float64), ref)


SMALL = dict(n_layers=2, d_model=128, n_heads=2, d_ffn=192, vocab=211, max_seq=40, lora_rank=4,
             E=2, S=40, q=2, n_labelled=5, eps=1e-2, lr=1e-2)


@pytest.mark.parametrize("fmt", ["int8", "nf4"])
@pytest.mark.parametrize("arch,bf16", [(ARCH_LLAMA, True), (ARCH_OPT, True), (ARCH_LLAMA, False)])
def test_step_on_quantised_checkpoint(arch, bf16, fmt):
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=bf16, **SMALL)
    p = make_decoder_problem(spec, seed=8, b_std=0.05)
    p["layers"] = [quantize_layer(L, fmt) for L in p["layers"]]
    ref = run_oracle(spec, p, p["tokens"], p["labels"], 23)
    got = run_gpu(spec, p, 23, weight_format=fmt)
    assert np.allclose(got["losses"], ref["losses"], rtol=2e-2 if bf16 else 1e-4, atol=0), (got["losses"], ref["losses"])
    if not bf16:
        assert np.all(np.abs(got["g"] - ref["g"]) <= 1e-2 * np.abs(ref["g"]).max())
        assert update_rel_err(spec, p, got["B"], ref["B"]) < 1e-3
    # the sequential schedule decodes the weights once per pass and still gives the same step
    seq = run_gpu(spec, p, 23, weight_format=fmt, schedule="sequential")
    assert np.array_equal(seq["losses"], got["losses"])


@pytest.mark.parametrize("fmt", ["int8", "nf4"])
@pytest.mark.parametrize("arch,E,S,sched", [(ARCH_LLAMA, 1, 100, None), (ARCH_OPT, 2, 128, "sequential"),
                                            (ARCH_LLAMA, 1, 128, "sequential")])
def test_decode_inside_the_gemm_matches_decode_to_scratch(arch, E, S, sched, fmt):
    """With ZO_FLAG_DEQUANT_FUSED, GEMM launches of at most 256 rows decode the codes inside the tensor-core
    kernel's operand producer; the default decodes every weight into scratch first.  Same bf16 operands,
    same accumulation order: the two steps agree bit for bit, whole tiles (E*S*2 = 200 -> 256 rows, two row
    tiles), K ranges of split launches (d = 512, ffn = 1024) and the SwiGLU gate|up layout included.
    The oracle's step on the same stored bytes bounds both."""
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=True,
                     **{**SMALL, "d_model": 512, "n_heads": 4, "d_ffn": 1024, "vocab": 517, "E": E, "S": S,
                        "max_seq": S, "q": 1 if sched is None else 2, "lora_rank": 8, "n_layers": 2})
    p = make_decoder_problem(spec, seed=8, b_std=0.05)
    p["layers"] = [quantize_layer(L, fmt) for L in p["layers"]]
    ref = run_oracle(spec, p, p["tokens"], p["labels"], 29)
    fused = run_gpu(spec, p, 29, weight_format=fmt, schedule=sched, flags=16)
    scratch = run_gpu(spec, p, 29, weight_format=fmt, schedule=sched)
    assert np.allclose(fused["losses"], ref["losses"], rtol=2e-2, atol=0), (fused["losses"], ref["losses"])
    assert np.array_equal(fused["losses"], scratch["losses"]) and np.array_equal(fused["rows"], scratch["rows"])
    assert np.array_equal(fused["g"], scratch["g"])
    assert all(np.array_equal(a, b) for a, b in zip(fused["B"], scratch["B"]))
    assert fused["launches"] < scratch["launches"]          # no decode passes
