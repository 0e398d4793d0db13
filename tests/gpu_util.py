"""Helpers shared by the GPU parity tests: run one zo_step through the C ABI and the
oracle's zo_step on the same seeded inputs."""
import numpy as np

import oracle
from workloads import make_decoder_problem, make_linear_problem
from workloads.spec import ARCH_LINEAR


def make_problem(spec, seed=1234, b_std=0.0):
    if spec.arch == ARCH_LINEAR:
        p = make_linear_problem(spec, seed=seed, b_std=b_std)
        return p, p["X"], p["target"]
    p = make_decoder_problem(spec, seed=seed, b_std=b_std)
    return p, p["tokens"], p["labels"]


def run_gpu(spec, p, seed, q=None, eps=None, lr=None, flags=0, host=False, schedule=None, **cfg_kw):
    import paper_2409_15520_b200 as zo
    q = spec.q if q is None else q
    eps = spec.eps if eps is None else eps
    lr = spec.lr if lr is None else lr
    cfg = zo.make_config(spec, flags=flags, max_q=max(q, spec.q), **cfg_kw)
    est = zo.Estimator(cfg)
    # a precision override runs the same (bf16-representable) numbers through the other mode
    prob = zo.DeviceProblem(p, spec.bf16 if cfg_kw.get("precision") is None else bool(cfg_kw["precision"]))
    if schedule:
        est.set_schedule(schedule)
    (est.step_host if host else est.step)(prob, spec.E, spec.S, seed, q, eps, lr)
    losses, g = est.losses()
    rows = est.row_losses()
    newB = prob.B_numpy()
    n_launch = est.launch_count()
    est.close()
    return dict(losses=losses.astype(np.float64), g=g.astype(np.float64), B=newB, rows=rows,
                launches=n_launch)


def run_oracle(spec, p, tok, lab, seed, q=None, eps=None, lr=None):
    q = spec.q if q is None else q
    eps = spec.eps if eps is None else eps
    lr = spec.lr if lr is None else lr
    losses, g, newB = oracle.zo_step(spec, p, tok, lab, seed, q, eps, lr)
    return dict(losses=losses, g=g, B=newB)


def old_B(spec, p):
    if spec.arch == ARCH_LINEAR:
        return [np.asarray(p["B"], np.float64)]
    return [np.asarray(L["B"], np.float64) for L in p["layers"]]


def update_rel_err(spec, p, got_B, ref_B):
    """|| B'_gpu - B'_oracle || / || B'_oracle - B || over all trainable tensors."""
    num = den = 0.0
    for b0, bg, br in zip(old_B(spec, p), got_B, ref_B):
        num += np.sum((bg.reshape(br.shape) - br) ** 2)
        den += np.sum((br - b0) ** 2)
    return np.sqrt(num / den)
