"""Parity at the named workload shapes (workloads.spec.CONFIGS), in the launch configuration
bench.py times them in (default flags, default tile-shape dispatch).

  opt125m      whole model, whole step, every replica, against the oracle's step (the oracle needs
               under a minute for it); bf16 at the 2e-2 loss tolerance, and the same weights in fp32
               mode at the fp32 tolerances with eps = 1e-3 as the configuration states.
  opt1p3b      full widths (d = 2048, 32 heads, vocabulary 50272 with a tied head, label-word loss),
               q = 8, E = 16, S = 256, depth cut to 2 blocks; the oracle evaluates the replicas
               {0, 1, 2q-2, 2q-1} on the whole batch.
  linear_sweep the 4096 x 4096 MP-LoRA layer on 4096 tokens, rank 8 / 16 / 64, q = 1 / 16, both
               input modes, sampled rows against the oracle's layer, including the +/- difference.
In every case the update line of Algorithm 1 is isolated by feeding the oracle's update formula
the GPU's own g."""
import numpy as np
import pytest

import oracle
from oracle.philox import perturbation
from oracle.zo import draw_z
from workloads import bf16_round, config, make_decoder_problem

from gpu_util import run_gpu, run_oracle, update_rel_err
from test_gpu_bf16_estimate import UPDATE_TOL, update_from_gpu_g

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def opt125m():
    spec = config("opt125m")
    p = make_decoder_problem(spec, seed=1234, b_std=0.01)
    seed = 5
    return spec, p, seed, run_oracle(spec, p, p["tokens"], p["labels"], seed)


def test_opt125m_whole_step_bf16(opt125m):
    spec, p, seed, ref = opt125m
    got = run_gpu(spec, p, seed)
    assert np.allclose(got["losses"], ref["losses"], rtol=2e-2, atol=0), (got["losses"], ref["losses"])
    assert abs(got["losses"].mean() - np.log(spec.vocab)) < 0.1 * np.log(spec.vocab)
    assert update_from_gpu_g(spec, p, seed, got) < UPDATE_TOL
    print("opt125m bf16: max rel loss err", np.max(np.abs(got["losses"] / ref["losses"] - 1)))


def test_opt125m_whole_step_fp32_mode(opt125m):
    """Same bf16-representable weights, fp32 activations and arithmetic, eps = 1e-3: the loss
    difference of a query is about 1e-5 of the loss, so g rests on the last digits of fp32 sums
    through 12 blocks and a 50272-way softmax.  Measured on a B200: losses 4e-8 relative, g 5e-4 of
    max|g|, update 4e-4 of the update; the stated fp32 tolerances hold at the full configuration."""
    spec, p, seed, ref = opt125m
    got = run_gpu(spec, p, seed, precision=0)
    rel_l = np.max(np.abs(got["losses"] / ref["losses"] - 1))
    rel_g = np.max(np.abs(got["g"] - ref["g"])) / np.max(np.abs(ref["g"]))
    upd = update_rel_err(spec, p, got["B"], ref["B"])
    print(f"opt125m fp32 mode, eps=1e-3: max rel loss err {rel_l:.2e}, max|dg|/max|g| {rel_g:.2e}, "
          f"update err / update {upd:.2e}; g_gpu={got['g']} g_oracle={ref['g']}")
    assert rel_l < 1e-4
    assert rel_g < 1e-2
    assert upd < 1e-3
    assert update_from_gpu_g(spec, p, seed, got) < UPDATE_TOL


def test_opt1p3b_sampled_replicas():
    spec = config("opt1p3b", n_layers=2)
    p = make_decoder_problem(spec, seed=1234, b_std=0.01)
    seed = 7
    got = run_gpu(spec, p, seed)
    q, E = spec.q, spec.E
    rows = got["rows"].reshape(2 * q, E)                    # one labelled row per sequence
    assert np.isfinite(got["losses"]).all()
    assert np.allclose(rows.mean(axis=1), got["losses"], rtol=1e-5)
    zs = {}
    for n in (0, 1, 2 * q - 2, 2 * q - 1):
        i, k = n // 2, (1.0 if n % 2 == 0 else -1.0)
        if i not in zs:
            zs[i] = draw_z(spec, p, seed, i)
        Bn = [(np.asarray(L["B"], np.float64) + k * spec.eps * zs[i][l])[None] for l, L in enumerate(p["layers"])]
        mean, ref = oracle.replica_losses(spec, p, Bn, p["tokens"], p["labels"], return_rows=True)
        # per-replica loss at the bf16 tolerance; the single rows (2-way cross-entropy of one logit
        # difference each) at twice that figure taken against ln 2
        assert abs(got["losses"][n] / mean[0] - 1) < 2e-2, (n, got["losses"][n], mean[0])
        assert np.max(np.abs(rows[n] - ref[0])) < 2 * 2e-2 * np.log(2.0), (n, rows[n], ref[0])
    assert update_from_gpu_g(spec, p, seed, got) < UPDATE_TOL


@pytest.mark.parametrize("x_replicated", [0, 1])
@pytest.mark.parametrize("q", [1, 16])
@pytest.mark.parametrize("r", [8, 16, 64])
def test_linear_sweep_point_sampled_rows(r, q, x_replicated):
    """One point of the micro-benchmark grid.  Replicated input: the two replicas of a query share
    their rows (queries differ), so Y[2i] - Y[2i+1] is 2 eps s U z_i in both input modes."""
    import torch
    import paper_2409_15520_b200 as zo
    T = k = 4096
    n = 2 * q
    eps, scale, seed, tid = 2e-2, 1.0, 7, 0
    rng = np.random.default_rng([r, q, x_replicated])
    W = bf16_round(0.02 * rng.standard_normal((k, k), dtype=np.float32))
    bias = bf16_round(0.02 * rng.standard_normal(k, dtype=np.float32))
    A = bf16_round(0.02 * rng.standard_normal((r, k), dtype=np.float32))
    B = 0.01 * rng.standard_normal((r, k), dtype=np.float32)
    dev = lambda a: torch.tensor(a, device="cuda").to(torch.bfloat16).contiguous()
    srows = np.r_[0:2, 127:129, 1000, 2047:2049, T - 2:T]    # tile edges, middle, tail
    if x_replicated:
        Xd = torch.empty((n, T, k), dtype=torch.bfloat16, device="cuda")
        Xs = np.empty((n, len(srows), k), np.float32)
        for i in range(q):
            xi = bf16_round(rng.standard_normal((T, k), dtype=np.float32))
            Xd[2 * i] = dev(xi)
            Xd[2 * i + 1] = Xd[2 * i]
            Xs[2 * i] = Xs[2 * i + 1] = xi[srows]
        Xd = Xd.reshape(n * T, k)
    else:
        x0 = bf16_round(rng.standard_normal((T, k), dtype=np.float32))
        Xd = dev(x0)
        Xs = np.broadcast_to(x0[srows], (n, len(srows), k))
    Y = zo.mp_lora_linear(Xd, dev(W), dev(bias), dev(A), torch.tensor(B, device="cuda"), T, q, scale, seed,
                          tid, eps, x_replicated)
    got = Y[:, torch.tensor(srows, device="cuda")].float().cpu().numpy().astype(np.float64)
    Bn = np.stack([B.astype(np.float64) + (1 if j % 2 == 0 else -1) * eps * perturbation(seed, tid, j // 2, (r, k))
                   for j in range(n)])
    ref = oracle.mp_lora_linear(Xs.astype(np.float64), W, bias, A, Bn, scale)
    amax = np.max(np.abs(ref))
    assert np.max(np.abs(got - ref)) < 2e-2 * amax
    # +/- difference of every query: its own z_i, sign and scale.  Both outputs carry one bf16
    # rounding (2^-9 relative) each; U, B and eps z enter the tensor-core form rounded to bf16.
    d_ref, d_gpu = ref[0::2] - ref[1::2], got[0::2] - got[1::2]
    for i in range(q):
        m = np.max(np.abs(d_ref[i]))
        assert m > 0
        assert np.max(np.abs(d_gpu[i] - d_ref[i])) < 0.05 * m + 2.0 ** -8 * amax, (i, m)
        # correlation with its own query's difference, not with a neighbour's
        c = np.sum(d_gpu[i] * d_ref[i]) / np.sqrt(np.sum(d_gpu[i] ** 2) * np.sum(d_ref[i] ** 2))
        assert c > 0.9, (i, c)
