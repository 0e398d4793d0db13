"""The entry point that allocates nothing (zo_mp_lora_linear_static) against the regular one.

Some users of this library run where device allocation is off limits (inside another
framework's memory budget, in a plug-in that only gets its input/output buffers, in a loop
that must not stall on an allocation).  They call the variant whose scratch is a fixed array
inside the library.  This file checks, through the C ABI, that it returns what the regular
entry point returns, twice in a row (the array is reused and keeps stale contents), and that
an oversized problem is refused.  It is collected last on purpose."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _inputs(rng, n_x, T, ki, ko, r, dtype):
    import torch
    mk = lambda a: torch.tensor(a.astype(np.float32), device="cuda").to(dtype).contiguous()
    X = mk(rng.standard_normal((n_x * T, ki)))
    W = mk(0.05 * rng.standard_normal((ko, ki)))
    bias = mk(0.05 * rng.standard_normal(ko))
    A = mk(0.05 * rng.standard_normal((r, ki)))
    B = torch.tensor((0.05 * rng.standard_normal((r, ko))).astype(np.float32), device="cuda")
    return X, W, bias, A, B


@pytest.mark.parametrize("bf16,x_replicated", [(False, 0), (True, 0), (True, 1)])
def test_static_scratch_entry_matches_regular_entry_twice(bf16, x_replicated):
    import torch
    import paper_2409_15520_b200 as zo
    dtype = torch.bfloat16 if bf16 else torch.float32
    rng = np.random.default_rng(5)
    T, ki, ko, r, q = 128, 136, 288, 8, 2
    for call, (seed, eps) in enumerate([(11, 1e-2), (12, 3e-2)]):       # two calls in a row
        X, W, bias, A, B = _inputs(rng, 2 * q if x_replicated else 1, T, ki, ko, r, dtype)
        ref = zo.mp_lora_linear(X, W, bias, A, B, T, q, 2.0, seed, 4, eps, x_replicated)
        Y = torch.full((2 * q, T, ko), float("nan"), dtype=dtype, device="cuda")
        zo.mp_lora_linear_static(X, W, bias, A, B, Y, T, q, 2.0, seed, 4, eps, x_replicated)
        assert zo.binding.mp_lora_linear_static_status() == 0   # also waits for the stream
        got, want = Y.float().cpu().numpy(), ref.float().cpu().numpy()
        assert np.isfinite(got).all()
        # same kernels, same order of operations: the parity tests' bf16 tolerance is 2e-2;
        # here the two paths must in fact agree to rounding
        assert np.max(np.abs(got - want)) <= 1e-6 * np.max(np.abs(want)), call


def test_static_scratch_entry_rejects_oversized_problem():
    import torch
    import paper_2409_15520_b200 as zo
    from paper_2409_15520_b200 import binding as b
    T, ki, ko, r, q = 8192, 64, 4096, 8, 1                 # base product alone is 64 MiB in bf16
    assert b.zo_mp_lora_scratch_bytes(1, T, ki, ko, r, q, 0) > zo.binding.STATIC_SCRATCH_BYTES
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device="cuda")
    Y = z(2 * q, T, ko)
    with pytest.raises(zo.ZoError) as ei:
        zo.mp_lora_linear_static(z(T, ki), z(ko, ki), None, z(r, ki),
                                 torch.zeros(r, ko, device="cuda"), Y, T, q, 1.0, 1, 0, 1e-3, 0)
    assert ei.value.status == 3                            # ZO_ERR_WORKSPACE
