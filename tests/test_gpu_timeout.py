"""The bounded-wait path of the tensor-core GEMM, exercised without faulting anything.

Every device-side wait of that kernel has a time limit; when one runs out the thread block raises
the time-out bit of the status word, drains what it has in flight, frees its tensor memory and
returns.  Nothing in a correct run makes a wait run out, so the library has a test aid that makes
one thread block's copy engine go silent (nothing armed, nothing in flight) and shortens the limit
to 1 ms.  These tests check that the failure is reported (ZO_ERR_TIMEOUT), that the trainable
tensors are left untouched, and that the same context then runs a normal step with the same bits
as a context that never saw the failure."""
import numpy as np
import pytest

from workloads import ModelSpec
from workloads.spec import ARCH_LLAMA, ARCH_OPT

from gpu_util import make_problem, old_B, run_gpu

pytestmark = pytest.mark.gpu

TIMEOUT = 5  # ZO_ERR_TIMEOUT


@pytest.mark.parametrize("arch,E", [(ARCH_LLAMA, 2), (ARCH_OPT, 1)])
def test_expired_wait_is_reported_and_the_context_stays_usable(arch, E):
    """E = 2: whole tiles per thread block; E = 1 (128 rows per pass under the sequential schedule):
    the launches are split along K and the wait runs out inside a K range."""
    import paper_2409_15520_b200 as zo
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), bf16=True, n_layers=2, d_model=512, n_heads=4,
                     d_ffn=1024, vocab=517, max_seq=128, lora_rank=8, E=E, S=128, q=2, n_labelled=6, eps=1e-2, lr=1e-2)
    p, tok, lab = make_problem(spec, b_std=0.05)
    sched = "sequential" if E == 1 else None
    clean = run_gpu(spec, p, 3, schedule=sched)
    est, prob = zo.Estimator(zo.make_config(spec)), zo.DeviceProblem(p, True)
    if sched:
        est.set_schedule(sched)
    est.test_expire_wait(1_000_000)
    est.step(prob, spec.E, spec.S, 3, spec.q, spec.eps, spec.lr)
    with pytest.raises(zo.ZoError) as ei:
        est.losses()
    assert ei.value.status == TIMEOUT
    assert all(np.array_equal(a, b.astype(np.float32)) for a, b in zip(prob.B_numpy(), old_B(spec, p)))
    est.test_expire_wait(0)
    est.step(prob, spec.E, spec.S, 3, spec.q, spec.eps, spec.lr)
    losses, g = est.losses()
    assert np.array_equal(losses.astype(np.float64), clean["losses"]) and np.array_equal(g.astype(np.float64), clean["g"])
    assert all(np.array_equal(a, b) for a, b in zip(prob.B_numpy(), clean["B"]))
    est.close()


def test_expired_wait_in_the_layer_entry_points():
    import torch
    import paper_2409_15520_b200 as zo
    from paper_2409_15520_b200 import binding as b
    rng = np.random.default_rng(2)
    T, ki, ko, r, q = 128, 256, 512, 8, 2
    mk = lambda a: torch.tensor(a.astype(np.float32), device="cuda").to(torch.bfloat16).contiguous()
    X, W, A = mk(rng.standard_normal((2 * q * T, ki))), mk(0.05 * rng.standard_normal((ko, ki))), mk(0.05 * rng.standard_normal((r, ki)))
    B = torch.tensor((0.05 * rng.standard_normal((r, ko))).astype(np.float32), device="cuda")
    good = zo.mp_lora_linear(X, W, None, A, B, T, q, 1.0, 5, 0, 1e-2, 1)
    with pytest.raises(zo.ZoError) as ei:
        zo.mp_lora_linear(X, W, None, A, B, T, q, 1.0, 5, 0, 1e-2, 1, flags=b.ZO_FLAG_TEST_EXPIRE_WAIT)
    assert ei.value.status == TIMEOUT
    again = zo.mp_lora_linear(X, W, None, A, B, T, q, 1.0, 5, 0, 1e-2, 1)
    assert torch.equal(good, again)
    # the entry point with built-in scratch keeps its status word out of the caller's reach: its accessor reports it
    Y = torch.empty_like(good)
    zo.mp_lora_linear_static(X, W, None, A, B, Y, T, q, 1.0, 5, 0, 1e-2, 1, flags=b.ZO_FLAG_TEST_EXPIRE_WAIT)
    with pytest.raises(zo.ZoError) as ei:
        b.mp_lora_linear_static_status()
    assert ei.value.status == TIMEOUT
    zo.mp_lora_linear_static(X, W, None, A, B, Y, T, q, 1.0, 5, 0, 1e-2, 1)
    assert b.mp_lora_linear_static_status() == 0 and torch.equal(Y, good)
