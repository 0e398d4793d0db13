"""The step in the form of Algorithm 2 ("Mobile MP-LoRA", q = 1): the +/- pair of every trainable
tensor is stored, the previous step's projected gradient is an input, and the previous update and
the new perturbation are applied inside the forward pass.

  layer       zo_mp_lora_linear_pair against oracle.mobile_mp_lora_forward (the new pair and the output);
  recurrence  k chained zo_step_pair calls against k steps of oracle.zo_step with q = 1: per-step losses
              and g, and after every call the mean of the pair = the oracle's master copy at that point,
              half the difference = eps z of the call's seed;
  no host round trip: the same chain enqueued without reading anything back ends at the same bits."""
import numpy as np
import pytest

import oracle
from oracle.philox import perturbation
from workloads import ModelSpec, bf16_round, config
from workloads.spec import ARCH_LLAMA, ARCH_OPT

from gpu_util import make_problem, old_B

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bf16,x_replicated", [(False, 1), (False, 0), (True, 1), (True, 0)])
def test_mobile_mp_lora_module(bf16, x_replicated):
    import torch
    import paper_2409_15520_b200 as zo
    rng = np.random.default_rng(11 + 2 * bf16 + x_replicated)
    T, ki, ko, r = 128, 192, 256, 8
    eps, lr, g, seed, tid = 1e-2, 5e-2, 0.7, 123, 4
    rnd = bf16_round if bf16 else (lambda a: a)
    # replicated input: distinct rows per replica in fp32 (the 1e-5 output tolerance then checks which
    # B each replica got); in bf16 both replicas get the same rows so that their difference isolates z
    x = rnd(rng.standard_normal((2 if x_replicated and not bf16 else 1, T, ki)).astype(np.float32))
    W = rnd(0.05 * rng.standard_normal((ko, ki)).astype(np.float32))
    A = rnd(0.05 * rng.standard_normal((r, ki)).astype(np.float32))
    B = (0.05 * rng.standard_normal((r, ko))).astype(np.float32)
    z_old = perturbation(77, tid, 0, (r, ko)).astype(np.float32)
    pair = np.stack([B + np.float32(eps) * z_old, B - np.float32(eps) * z_old]).astype(np.float32)
    z_new = perturbation(seed, tid, 0, (r, ko))
    xn = np.broadcast_to(x, (2, T, ki)).astype(np.float64)
    ref_out, ref_pair = oracle.mobile_mp_lora_forward(xn, W, A, pair.astype(np.float64), z_new, g, eps, lr)
    dt = torch.bfloat16 if bf16 else torch.float32
    dev = lambda a: torch.tensor(a, device="cuda").to(dt).contiguous()
    Pd = torch.tensor(pair, device="cuda")
    xd = np.broadcast_to(x, (2, T, ki)) if x_replicated else x
    Y = zo.mp_lora_linear_pair(dev(np.ascontiguousarray(xd).reshape(-1, ki)), dev(W), None, dev(A), Pd, T, 1.0, seed, tid, g, eps, lr, x_replicated)
    got_pair = Pd.cpu().numpy().astype(np.float64)
    # the stored pair after the call: previous update applied, new perturbation in place
    assert np.max(np.abs(got_pair - ref_pair)) < 2e-6 * np.max(np.abs(ref_pair))
    assert np.allclose((got_pair[0] - got_pair[1]) / 2, eps * z_new, rtol=0, atol=16 * 2.0 ** -24 * np.max(np.abs(pair)))
    out = Y.float().cpu().numpy().astype(np.float64)
    tol = 2e-2 if bf16 else 1e-5
    assert np.max(np.abs(out - ref_out)) < tol * np.max(np.abs(ref_out))
    # the two replicas differ by the new perturbation: 2 eps (x A) z_new
    d_ref, d_got = ref_out[0] - ref_out[1], out[0] - out[1]
    if np.array_equal(xn[0], xn[1]):
        bound = (0.1 if bf16 else 1e-3) * np.max(np.abs(d_ref)) + (2.0 ** -8 * np.max(np.abs(ref_out)) if bf16 else 0.0)
        assert np.max(np.abs(d_got - d_ref)) < bound


def _chain(spec, p, tok, lab, seeds, eps, lr):
    """Oracle: k steps of Algorithm 1 with q = 1 -> per-step (losses, g) and the master copies B_0..B_k."""
    from oracle.zo import _b_tensors
    import copy
    pp = copy.copy(p)
    hist, masters = [], [[b.copy() for b in _b_tensors(spec, p)]]
    for s in seeds:
        losses, g, newB = oracle.zo_step(spec, pp, tok, lab, s, 1, eps, lr)
        hist.append((losses, g))
        masters.append([b.copy() for b in newB])
        if "layers" in pp:
            pp = dict(pp, layers=[dict(L, B=b) for L, b in zip(pp["layers"], newB)])
        else:
            pp = dict(pp, B=newB[0])
    return hist, masters


def _rel(a_list, b_list, base_list):
    num = sum(np.sum((a.reshape(b.shape) - b) ** 2) for a, b in zip(a_list, b_list))
    den = sum(np.sum((b - c) ** 2) for b, c in zip(b_list, base_list))
    return np.sqrt(num / den)


@pytest.mark.parametrize("kind", ["linear", "llama_fp32", "opt_bf16"])
def test_pair_steps_follow_the_master_copy_recurrence(kind):
    import torch
    import paper_2409_15520_b200 as zo
    from oracle.zo import draw_z
    if kind == "linear":
        spec = config("linear_fp32", q=1, eps=1e-3, lr=1e-2)
    elif kind == "llama_fp32":
        spec = ModelSpec(arch=ARCH_LLAMA, bf16=False, n_layers=2, d_model=64, n_heads=4, d_ffn=96, vocab=131, max_seq=24,
                         lora_rank=4, E=3, S=24, q=1, n_labelled=5, eps=1e-2, lr=2e-2)
    else:
        spec = ModelSpec(arch=ARCH_OPT, tie_lm_head=True, bf16=True, n_layers=3, d_model=256, n_heads=4, d_ffn=512,
                         vocab=517, max_seq=128, lora_rank=8, E=2, S=128, q=1, n_labelled=6, eps=0.25, lr=2e-2)
    p, tok, lab = make_problem(spec, b_std=0.05)
    seeds = [31, 32, 33, 34]
    hist, masters = _chain(spec, p, tok, lab, seeds, spec.eps, spec.lr)
    est, prob = zo.Estimator(zo.make_config(spec)), zo.DeviceProblem(p, spec.bf16)
    prob.make_pair()
    gbuf = est.g_buffer()
    tol_l, tol_g = (2e-2, 0.04) if spec.bf16 else (1e-4, 1e-2)
    gmax = max(abs(float(g[0])) for _, g in hist)
    for t, s in enumerate(seeds):
        est.step_pair(prob, spec.E, spec.S, s, gbuf if t else None, spec.eps, spec.lr)
        losses, g = est.losses()
        assert np.allclose(losses, hist[t][0], rtol=tol_l, atol=0), (t, losses, hist[t][0])
        assert abs(g[0] - hist[t][1][0]) <= tol_g * gmax, (t, g, hist[t][1])
        pair = prob.pair_numpy()
        mean = [(x[0] + x[1]) / 2 for x in pair]
        half = [(x[0] - x[1]) / 2 for x in pair]
        z = draw_z(spec, p, s, 0)
        for h, zz in zip(half, z):          # the stored perturbation is eps z of this call's seed
            assert np.allclose(h.reshape(zz.shape), spec.eps * zz, rtol=0, atol=16 * 2.0 ** -24 * max(np.max(np.abs(x)) for x in pair))
        if t:                               # mean of the pair = the master copy before this step's update
            if spec.bf16:
                # bf16 g differs from the oracle's by up to tol_g: compare with the oracle's formula fed the GPU's g
                continue
            err = _rel(mean, masters[t], masters[0])
            print(f"pair chain {kind}: step {t} master copy error / cumulative update = {err:.2e}")
            assert err < 5e-3, t
    est.pair_collapse(prob, gbuf, spec.eps, spec.lr)
    final = prob.pair_numpy()
    for x in final:      # both halves at the updated master copy: B[0] - diff and B[1] + diff round apart by an
        # ulp of the perturbed values they are formed from
        assert np.allclose(x[0], x[1], rtol=0, atol=2.0 ** -22 * (np.max(np.abs(x)) + 6 * spec.eps))
    if not spec.bf16:
        assert _rel([x[0] for x in final], masters[-1], masters[0]) < 1e-2
    # the same chain with nothing read back between the steps: g travels on the device only
    est2, prob2 = zo.Estimator(zo.make_config(spec)), zo.DeviceProblem(p, spec.bf16)
    prob2.make_pair()
    g2 = est2.g_buffer()
    for t, s in enumerate(seeds):
        est2.step_pair(prob2, spec.E, spec.S, s, g2 if t else None, spec.eps, spec.lr)
    est2.pair_collapse(prob2, g2, spec.eps, spec.lr)
    torch.cuda.synchronize()
    for a, b in zip(prob2.pair_numpy(), final):
        assert np.array_equal(a, b)
    est.close()
    est2.close()


def test_pair_step_argument_errors():
    import paper_2409_15520_b200 as zo
    spec = config("linear_fp32", q=1)
    p, tok, lab = make_problem(spec, b_std=0.02)
    est, prob = zo.Estimator(zo.make_config(spec, max_q=2)), zo.DeviceProblem(p, False)
    prob.make_pair()
    with pytest.raises(zo.ZoError) as ei:
        est.step_pair(prob, spec.E, spec.S, 1, None, 0.0, 1e-3)      # eps = 0: the update divides by eps
    assert ei.value.status == 1
    est.set_query_shard(0, 1)
    with pytest.raises(zo.ZoError) as ei:
        est.step_pair(prob, spec.E, spec.S, 1, None, 1e-3, 1e-3)
    assert ei.value.status == 7
    est.set_query_shard(0, 0)
    est.step_pair(prob, spec.E, spec.S, 1, None, 1e-3, 1e-3)
    losses, g = est.losses()
    assert losses.shape == (2,) and np.isfinite(losses).all()
    est.close()
