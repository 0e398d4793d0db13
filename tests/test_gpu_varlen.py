"""GPU parity for packed variable-length batches (zo_step_varlen) against the oracle's ragged step."""
import numpy as np
import pytest

from workloads import ModelSpec, make_decoder_problem, make_ragged_batch
from workloads.spec import ARCH_LLAMA, ARCH_OPT, LOSS_CE_FULL, LOSS_CE_LABEL_WORDS

from gpu_util import old_B, run_oracle, update_rel_err

pytestmark = pytest.mark.gpu

BASE = dict(n_layers=2, d_model=128, n_heads=2, d_ffn=192, vocab=211, max_seq=150, lora_rank=4,
            E=5, S=150, q=2, n_labelled=4, eps=1e-2, lr=1e-2)


def _run_varlen(spec, p, toks, labs, seed, flags=0):
    import torch
    import paper_2409_15520_b200 as zo
    est = zo.Estimator(zo.make_config(spec, flags=flags))
    prob = zo.DeviceProblem(p, spec.bf16)
    cu = np.concatenate([[0], np.cumsum([len(t) for t in toks])]).astype(np.int32)
    dev = lambda a: torch.tensor(np.ascontiguousarray(a), dtype=torch.int32, device="cuda")
    est.step_varlen(prob, dev(np.concatenate(toks)), dev(np.concatenate(labs)), dev(cu), spec.S, seed,
                    spec.q, spec.eps, spec.lr)
    losses, g = est.losses()
    out = dict(losses=losses.astype(np.float64), g=g.astype(np.float64), B=prob.B_numpy())
    est.close()
    return out


@pytest.mark.parametrize("arch,bf16,loss", [(ARCH_LLAMA, False, LOSS_CE_FULL), (ARCH_OPT, False, LOSS_CE_LABEL_WORDS),
                                            (ARCH_LLAMA, True, LOSS_CE_FULL), (ARCH_OPT, True, LOSS_CE_FULL)])
def test_packed_variable_length_step(arch, bf16, loss):
    """Five sequences of 37..150 tokens packed back to back (several attention tiles, ragged tails,
    rows per replica not a multiple of anything): positions restart per sequence, attention stays inside
    a sequence, the loss is the mean over all labelled positions of the batch."""
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=bf16, loss_kind=loss, label_words=(3, 99),
                     **{**BASE, "n_labelled": 1 if loss == LOSS_CE_LABEL_WORDS else 4,
                        # five labelled rows only: a larger eps keeps the loss difference above fp32 noise
                        "eps": 5e-2 if loss == LOSS_CE_LABEL_WORDS else 1e-2})
    p = make_decoder_problem(spec, seed=4, b_std=0.05)
    toks, labs = make_ragged_batch(spec, seed=6)
    assert len({len(t) for t in toks}) > 1
    ref = run_oracle(spec, p, toks, labs, 19)
    got = _run_varlen(spec, p, toks, labs, 19)
    assert np.allclose(got["losses"], ref["losses"], rtol=2e-2 if bf16 else 1e-4, atol=0), (got["losses"], ref["losses"])
    if not bf16:
        assert np.all(np.abs(got["g"] - ref["g"]) <= 1e-2 * np.abs(ref["g"]).max())
        assert update_rel_err(spec, p, got["B"], ref["B"]) < 1e-3
    else:
        simt = _run_varlen(spec, p, toks, labs, 19, flags=1)
        assert np.allclose(got["losses"], simt["losses"], rtol=3e-3, atol=0)


def test_equal_lengths_reduce_to_the_fixed_length_step_and_bad_cu_is_reported():
    import torch
    import paper_2409_15520_b200 as zo
    from gpu_util import run_gpu
    spec = ModelSpec(arch=ARCH_LLAMA, bf16=False, **{**BASE, "E": 3, "S": 24, "max_seq": 24})
    p = make_decoder_problem(spec, seed=4, b_std=0.05)
    fixed = run_gpu(spec, p, 5)
    toks, labs = list(p["tokens"]), list(p["labels"])
    packed = _run_varlen(spec, p, toks, labs, 5)
    assert np.array_equal(packed["losses"], fixed["losses"]) and np.array_equal(packed["g"], fixed["g"])
    # a sequence longer than max_len: reported by zo_losses, B untouched
    est = zo.Estimator(zo.make_config(spec))
    prob = zo.DeviceProblem(p, False)
    dev = lambda a: torch.tensor(np.ascontiguousarray(a), dtype=torch.int32, device="cuda")
    est.step_varlen(prob, dev(np.concatenate(toks)), dev(np.concatenate(labs)), dev(np.array([0, 30, 50, 72])),
                    24, 5, spec.q, spec.eps, spec.lr)
    with pytest.raises(zo.ZoError) as ei:
        est.losses()
    assert ei.value.status == 1
    assert all(np.array_equal(a, b.astype(np.float32)) for a, b in zip(prob.B_numpy(), old_B(spec, p)))
    est.close()
