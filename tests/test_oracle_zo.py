"""Pins for the oracle's estimator and update (CPU only)."""
import numpy as np
import pytest

import oracle
from oracle import zo as oz
from oracle.philox import perturbation
from workloads import ModelSpec, config, make_decoder_problem, make_linear_problem
from workloads.spec import ARCH_LINEAR, ARCH_LLAMA, ARCH_OPT, LOSS_MSE

TINY = dict(n_layers=2, d_model=16, n_heads=2, d_ffn=24, vocab=37, max_seq=8,
            lora_rank=2, E=2, S=8, n_labelled=3, bf16=False)


def _tiny(arch, **kw):
    spec = ModelSpec(arch=arch, tie_lm_head=(arch == ARCH_OPT), **{**TINY, **kw})
    return spec, make_decoder_problem(spec, seed=11, b_std=0.05)


@pytest.mark.parametrize("arch", [ARCH_OPT, ARCH_LLAMA])
def test_batched_mp_lora_equals_2q_sequential_forwards(arch):
    """Pin: one pass over the n=2q replicated batch == 2q independent passes."""
    spec, p = _tiny(arch)
    q, eps, seed = 3, 1e-2, 77
    losses, g, newB = oracle.zo_step(spec, p, p["tokens"], p["labels"], seed, q, eps, 1e-3)
    zs = [oz.draw_z(spec, p, seed, i) for i in range(q)]
    Bn = []
    for l, L in enumerate(p["layers"]):
        stack = []
        for n in range(2 * q):
            k = 1.0 if n % 2 == 0 else -1.0
            stack.append(np.asarray(L["B"], np.float64) + k * eps * zs[n // 2][l])
        Bn.append(np.stack(stack))
    batched = oracle.replica_losses(spec, p, Bn, p["tokens"], p["labels"])
    assert batched.shape == (2 * q,)
    assert np.allclose(batched, losses, rtol=1e-12, atol=0)
    assert len(set(np.round(losses, 9))) == 2 * q          # replicas really differ


def test_eps_zero_gives_identical_losses_and_b_zero_gives_base_loss():
    spec, p = _tiny(ARCH_OPT)
    losses, g, newB = oracle.zo_step(spec, p, p["tokens"], p["labels"], 5, 4, 0.0, 1e-3)
    assert np.all(losses == losses[0]) and np.all(g == 0)
    assert all(np.array_equal(a, np.asarray(L["B"], np.float64)) for a, L in zip(newB, p["layers"]))
    # B = 0: the adapted model is the base model (LoRA starts with no deviation)
    p0 = make_decoder_problem(spec, seed=11, b_std=0.0)
    base = make_decoder_problem(spec.with_(lora_targets=0), seed=11)
    for L in base["layers"]:
        L["A"], L["B"] = np.zeros((0, spec.d_model), np.float32), np.zeros((0, spec.lora_rank, spec.d_model), np.float32)
    l0 = oracle.zo_step(spec, p0, p0["tokens"], p0["labels"], 5, 2, 0.0, 0.0)[0]
    lb = oracle.replica_losses(spec.with_(lora_targets=0), base,
                               [np.zeros((1, 0, spec.lora_rank, spec.d_model))] * spec.n_layers,
                               base["tokens"], base["labels"])
    assert np.allclose(l0, lb[0], rtol=1e-13)


def _quadratic(d, rng):
    M = rng.standard_normal((d, d))
    H = M @ M.T / d + np.eye(d)
    b = rng.standard_normal(d)
    return (lambda th: 0.5 * th @ H @ th + b @ th), (lambda th: H @ th + b)


def test_quadratic_loss_central_difference_is_exact_and_variance_scales_as_d_over_q():
    """On L = 1/2 th'H th + b'th, g_i = <z_i, grad L> exactly and
    E||ghat - grad||^2 = (d+1)||grad||^2 / q for Gaussian z."""
    rng = np.random.default_rng(0)
    shape, d, eps = (4, 4), 16, 1e-3
    L, dL = _quadratic(d, rng)
    th = rng.standard_normal(d)
    grad = dL(th)
    for q in (1, 4, 16, 64):
        trials, mse = 1500, 0.0
        for s in range(trials):
            zs = [perturbation(1000 * q + s, 0, i, shape).reshape(-1) for i in range(q)]
            losses = np.array([L(th + k * eps * z) for z in zs for k in (1.0, -1.0)])
            g = oracle.projected_gradients(losses, eps)
            assert np.allclose(g, [z @ grad for z in zs], rtol=1e-7, atol=1e-9)
            new = oracle.zo_sgd_update([th.reshape(shape)], [[z.reshape(shape)] for z in zs], g, 1.0)[0]
            ghat = th - new.reshape(-1)
            mse += np.sum((ghat - grad) ** 2)
        mse /= trials
        expect = (d + 1) * grad @ grad / q
        assert abs(mse / expect - 1.0) < 0.15, (q, mse, expect)


def test_quadratic_estimate_converges_to_gradient_as_q_grows():
    rng = np.random.default_rng(1)
    shape, d, eps = (2, 4), 8, 1e-3
    L, dL = _quadratic(d, rng)
    th = rng.standard_normal(d)
    grad = dL(th)
    errs = []
    for q in (4, 64, 1024, 8192):
        zs = [perturbation(9, 0, i, shape).reshape(-1) for i in range(q)]
        losses = np.array([L(th + k * eps * z) for z in zs for k in (1.0, -1.0)])
        g = oracle.projected_gradients(losses, eps)
        new = oracle.zo_sgd_update([th.reshape(shape)], [[z.reshape(shape)] for z in zs], g, 1.0)[0]
        errs.append(np.linalg.norm(th - new.reshape(-1) - grad) / np.linalg.norm(grad))
    assert errs[-1] < 0.06 and errs[-1] < errs[0] / 10


def test_linear_mse_config_closed_form_gradient():
    """The linear+MSE problem is quadratic in B, so with U = X A^T and residual
    R = X W^T + b + s U B - target: grad_B L = (2 s / (T k_out)) U^T R,
    g_i = <z_i, grad_B L>, and (l+ + l-)/2 - L(B) = eps^2 s^2 ||U z_i||_F^2 / (T k_out)."""
    spec = config("linear_fp32", lora_scale=2.0)
    p = make_linear_problem(spec, seed=1234, b_std=0.02)
    q, eps, lr, seed = spec.q, spec.eps, spec.lr, 1
    losses, g, newB = oracle.zo_step(spec, p, p["X"], p["target"], seed, q, eps, lr)
    X, W, A, B = (np.asarray(p[k], np.float64) for k in ("X", "W", "A", "B"))
    s, T, ko = spec.lora_scale, X.shape[0], W.shape[0]
    U = X @ A.T
    R = X @ W.T + p["bias"] + s * U @ B - p["target"]
    grad = 2 * s / (T * ko) * U.T @ R
    L0 = (R ** 2).mean()
    upd = np.zeros_like(B)
    for i in range(q):
        z = perturbation(seed, 0, i, B.shape)
        assert abs(g[i] - (z * grad).sum()) < 1e-7 * abs(g[i]) + 1e-12
        curv = eps ** 2 * s ** 2 * ((U @ z) ** 2).sum() / (T * ko)
        assert abs((losses[2 * i] + losses[2 * i + 1]) / 2 - L0 - curv) < 1e-12
        upd += g[i] * z
    assert np.allclose(newB[0], B - lr * upd / q, rtol=1e-12, atol=1e-15)
    assert losses[0] != losses[1]


@pytest.mark.parametrize("arch", [ARCH_OPT, ARCH_LLAMA])
def test_brute_force_coordinate_finite_differences(arch):
    """g_i -> <z_i, grad L> with grad L from coordinate-wise differences; O(eps^2) error."""
    spec, p = _tiny(arch, n_layers=1, S=6, max_seq=6, E=1)
    Bs = [np.asarray(L["B"], np.float64) for L in p["layers"]]

    def loss(Bl):
        return oracle.replica_losses(spec, p, [b[None] for b in Bl], p["tokens"], p["labels"])[0]

    h = 1e-5
    grads = []
    for t, B in enumerate(Bs):
        G = np.zeros_like(B)
        for idx in np.ndindex(B.shape):
            Bp = [b.copy() for b in Bs]; Bm = [b.copy() for b in Bs]
            Bp[t][idx] += h; Bm[t][idx] -= h
            G[idx] = (loss(Bp) - loss(Bm)) / (2 * h)
        grads.append(G)
    seed = 21
    errs = []
    for eps in (1e-2, 1e-3):
        _, g, _ = oracle.zo_step(spec, p, p["tokens"], p["labels"], seed, 2, eps, 0.0)
        zs = [oz.draw_z(spec, p, seed, i) for i in range(2)]
        ref = np.array([sum((z * G).sum() for z, G in zip(zs[i], grads)) for i in range(2)])
        errs.append(np.abs(g - ref).max() / np.abs(ref).max())
    assert errs[1] < 1e-4
    assert errs[1] < errs[0] / 20          # second-order convergence in eps


@pytest.mark.parametrize("arch", [ARCH_LINEAR, ARCH_OPT])
def test_q1_equals_sequential_in_place_mezo(arch):
    if arch == ARCH_LINEAR:
        spec = config("linear_fp32", d_model=32, d_out=24, lora_rank=4, E=2, S=4)
        p = make_linear_problem(spec, seed=3, b_std=0.05)
        tok, lab = p["X"], p["target"]
    else:
        spec, p = _tiny(arch)
        tok, lab = p["tokens"], p["labels"]
    a = oracle.zo_step(spec, p, tok, lab, 99, 1, 1e-3, 1e-2)
    b = oracle.mezo_sequential_step(spec, p, tok, lab, 99, 1e-3, 1e-2)
    assert np.allclose(a[0], b[0], rtol=1e-12)
    assert abs(a[1][0] - b[1]) < 1e-7 * abs(b[1])
    for x, y in zip(a[2], b[2]):
        assert np.allclose(x, y, rtol=0, atol=1e-9 * np.abs(y).max())


def test_mobile_mp_lora_recurrences_equal_master_copy_form():
    """From B[0] = B + eps z_old, B[1] = B - eps z_old the module's lines give
    mean(B') = B - eta g z_old and half-difference(B') = eps z_new, and its
    output is the MP-LoRA layer on the new pair."""
    rng = np.random.default_rng(4)
    T, k, r, eps, lr, g = 5, 6, 3, 1e-2, 3e-3, 0.37
    x = rng.standard_normal((2, T, k))
    W, A, B = rng.standard_normal((k, k)), rng.standard_normal((r, k)), rng.standard_normal((r, k))
    z_old, z_new = perturbation(1, 0, 0, (r, k)), perturbation(1, 0, 1, (r, k))
    pair = np.stack([B + eps * z_old, B - eps * z_old])
    out, new = oracle.mobile_mp_lora_forward(x, W, A, pair, z_new, g, eps, lr)
    master = oracle.zo_sgd_update([B], [[z_old]], np.array([g]), lr)[0]
    assert np.allclose((new[0] + new[1]) / 2, master, atol=1e-14)
    assert np.allclose((new[0] - new[1]) / 2, eps * z_new, atol=1e-14)
    ref = oracle.mp_lora_linear(x, W, None, A, np.stack([master + eps * z_new, master - eps * z_new]), 1.0)
    assert np.allclose(out, ref, atol=1e-12)


def test_update_lies_in_span_of_perturbations_and_tensor_ids():
    spec, p = _tiny(ARCH_LLAMA)
    seed, q, eps, lr = 8, 1, 1e-3, 0.5
    losses, g, newB = oracle.zo_step(spec, p, p["tokens"], p["labels"], seed, q, eps, lr)
    nt = spec.n_targets
    for l, (Bn, L) in enumerate(zip(newB, p["layers"])):
        for t in range(nt):
            z = perturbation(seed, l * nt + t, 0, L["B"].shape[1:])
            ratio = (Bn[t] - L["B"][t]) / z
            assert np.allclose(ratio, -lr * g[0], rtol=1e-6)
    # one scalar per query is shared by every tensor; q > 1 averages
    losses, g, newB = oracle.zo_step(spec, p, p["tokens"], p["labels"], seed, 3, eps, lr)
    acc = sum(g[i] * perturbation(seed, 1 * nt + 1, i, p["layers"][1]["B"].shape[1:]) for i in range(3))
    assert np.allclose(newB[1][1], p["layers"][1]["B"][1] - lr * acc / 3, rtol=1e-12, atol=1e-15)


def test_replica_order_and_sign_convention():
    """Replica 2i carries +eps z_i and 2i+1 carries -eps z_i; g has the sign of <z, grad>."""
    spec = config("linear_fp32", d_model=16, d_out=8, lora_rank=2, E=1, S=4)
    p = make_linear_problem(spec, seed=2, b_std=0.1)
    seed, eps = 3, 1e-2
    losses, g, _ = oracle.zo_step(spec, p, p["X"], p["target"], seed, 2, eps, 0.0)
    for i in range(2):
        z = perturbation(seed, 0, i, p["B"].shape)
        lp = oracle.replica_losses(spec, p, (p["B"] + eps * z)[None], p["X"], p["target"])[0]
        lm = oracle.replica_losses(spec, p, (p["B"] - eps * z)[None], p["X"], p["target"])[0]
        assert losses[2 * i] == lp and losses[2 * i + 1] == lm
        assert np.sign(g[i]) == np.sign(lp - lm)


@pytest.mark.parametrize("arch", [ARCH_OPT, ARCH_LLAMA])
def test_ragged_batch_equals_padded_batch_with_ignored_padding(arch):
    """Causal attention: tokens appended after a sequence cannot change its earlier positions, so the
    ragged (unpadded) evaluation equals the padded one with the padding positions left out of the loss."""
    from workloads import make_ragged_batch
    spec, p = _tiny(arch, E=3, S=8, max_seq=8, n_labelled=2)
    toks, labs = make_ragged_batch(spec, seed=5)
    assert len({len(t) for t in toks}) > 1 and all(2 <= len(t) <= 8 for t in toks)
    pad_t = np.zeros((3, 8), np.int32)
    pad_l = np.full((3, 8), -1, np.int32)
    for b, (t, l) in enumerate(zip(toks, labs)):
        pad_t[b, :len(t)] = t
        pad_t[b, len(t):] = 7                      # arbitrary padding token
        pad_l[b, :len(l)] = l
    a = oracle.zo_step(spec, p, toks, labs, 3, 2, 1e-2, 1e-2)
    b = oracle.zo_step(spec, p, pad_t, pad_l, 3, 2, 1e-2, 1e-2)
    assert np.allclose(a[0], b[0], rtol=1e-12) and np.allclose(a[1], b[1], rtol=1e-9)
    for x, y in zip(a[2], b[2]):
        assert np.allclose(x, y, rtol=0, atol=1e-12)
