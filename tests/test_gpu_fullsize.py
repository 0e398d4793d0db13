"""Parity at the benchmark's launch configuration: the Llama-2-7B widths, q = 16, E = 16, S = 256
(131 072 token rows per GEMM, the tile grid bench.py times), depth cut to 2 blocks so that the
oracle can evaluate sampled (replica, sequence) outputs one by one in seconds; plus properties
that hold at any size."""
import numpy as np
import pytest

import oracle
from oracle.zo import draw_z
from workloads import config, make_decoder_problem

from gpu_util import run_gpu
from test_gpu_bf16_estimate import UPDATE_TOL, update_from_gpu_g

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def problem():
    spec = config("llama7b", n_layers=2)
    return spec, make_decoder_problem(spec, seed=1234, b_std=0.01)


def test_sampled_row_losses_against_oracle(problem):
    spec, p = problem
    seed = 5
    got = run_gpu(spec, p, seed)
    q, E, P = spec.q, spec.E, spec.n_labelled
    rows = got["rows"].reshape(2 * q, E, P)
    assert np.isfinite(got["losses"]).all() and got["launches"] > 0
    # the update line of Algorithm 1 alone: the oracle's formula fed the GPU's g
    assert update_from_gpu_g(spec, p, seed, got) < UPDATE_TOL
    # replica means are the means of their rows
    assert np.allclose(rows.mean(axis=(1, 2)), got["losses"], rtol=1e-5)
    zs = {}
    for n, b in [(0, 0), (1, 0), (2 * q - 1, E - 1), (17, 7)]:        # sampled (replica, sequence)
        i, k = n // 2, (1.0 if n % 2 == 0 else -1.0)
        if i not in zs:
            zs[i] = draw_z(spec, p, seed, i)
        Bn = [(np.asarray(L["B"], np.float64) + k * spec.eps * zs[i][l])[None] for l, L in enumerate(p["layers"])]
        sub = spec.with_(E=1)
        _, ref = oracle.replica_losses(sub, p, Bn, p["tokens"][b:b + 1], p["labels"][b:b + 1], return_rows=True)
        assert np.allclose(rows[n, b], ref[0], rtol=2e-2, atol=0), (n, b, rows[n, b], ref[0])


def test_eps_zero_replicas_identical_at_full_size(problem):
    spec, p = problem
    got = run_gpu(spec, p, 9, eps=0.0)
    assert np.all(got["losses"] == got["losses"][0])
    assert np.all(got["rows"] == got["rows"][0])                        # bit-identical replicas
    assert abs(got["losses"][0] - np.log(spec.vocab)) < 0.15 * np.log(spec.vocab)
