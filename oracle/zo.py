"""The randomized gradient estimator and ZO-SGD step (test infrastructure).

`zo_step` is the plain definition the MP-LoRA batching must reproduce: 2q
independent forward passes, one per (query, sign), each with its own perturbed
copy of the trainable tensors (Algorithm 1; RGE equation of the Background
section), then the projected gradients and the SGD update.
"""
import numpy as np

from .model import ARCH_LINEAR, replica_losses
from .philox import perturbation


def _b_tensors(spec, p):
    """The trainable tensors in tensor_id order: [(B array, tensor_id)]."""
    if spec.arch == ARCH_LINEAR:
        return [np.asarray(p["B"], np.float64)]
    return [np.asarray(L["B"], np.float64) for L in p["layers"]]


def draw_z(spec, p, seed, i):
    """z_i over all trainable tensors (Algorithm 1: z_i ~ N(0, I_{d_l}) using s_i).
    tensor_id = layer * n_targets + target slot; s_i = (seed, i)."""
    if spec.arch == ARCH_LINEAR:
        return [perturbation(seed, 0, i, p["B"].shape)]
    nt = spec.n_targets
    zs = []
    for l, L in enumerate(p["layers"]):
        zs.append(np.stack([perturbation(seed, l * nt + t, i, L["B"].shape[1:])
                            for t in range(nt)]) if nt else np.zeros(np.shape(L["B"])))
    return zs


def _loss_with(spec, p, Bs, tokens, labels):
    if spec.arch == ARCH_LINEAR:
        return replica_losses(spec, p, Bs[0][None], tokens, labels)[0]
    return replica_losses(spec, p, [b[None] for b in Bs], tokens, labels)[0]


def projected_gradients(losses, eps):
    """g_i = (l^(+1) - l^(-1)) / (2 eps) (Algorithm 1); replica order n = 2i + {0:+, 1:-}."""
    losses = np.asarray(losses, np.float64)
    return (losses[0::2] - losses[1::2]) / (2.0 * eps)


def zo_sgd_update(Bs, zs, g, lr):
    """theta_l <- theta_l - eta * (1/q) * sum_i g_i z_i (Algorithm 1, last line of the step)."""
    q = len(g)
    out = []
    for t, B in enumerate(Bs):
        acc = np.zeros_like(B)
        for i in range(q):
            acc += g[i] * zs[i][t]
        out.append(B - lr * acc / q)
    return out


def zo_step(spec, p, tokens, labels, seed, q, eps, lr):
    """One step of Algorithm 1 by its definition -> (losses[2q], g[q], new B list)."""
    Bs = _b_tensors(spec, p)
    zs = [draw_z(spec, p, seed, i) for i in range(q)]
    losses = np.zeros(2 * q)
    for i in range(q):
        for j, k in enumerate((+1.0, -1.0)):
            Bk = [B + k * eps * z for B, z in zip(Bs, zs[i])]     # theta_l^(k) = theta_l + k eps z_i
            losses[2 * i + j] = _loss_with(spec, p, Bk, tokens, labels)
    if eps == 0.0:
        return losses, np.zeros(q), Bs
    g = projected_gradients(losses, eps)
    return losses, g, zo_sgd_update(Bs, zs, g, lr)


def mezo_sequential_step(spec, p, tokens, labels, seed, eps, lr):
    """q = 1 sequential baseline (appendix "MeZO with q>1" at q=1): perturb the
    parameters in place by +eps z, then -2 eps z, then +eps z, then update."""
    Bs = [b.copy() for b in _b_tensors(spec, p)]
    z = draw_z(spec, p, seed, 0)
    for B, zz in zip(Bs, z):
        B += eps * zz
    lp = _loss_with(spec, p, Bs, tokens, labels)
    for B, zz in zip(Bs, z):
        B += -2.0 * eps * zz
    lm = _loss_with(spec, p, Bs, tokens, labels)
    for B, zz in zip(Bs, z):
        B += eps * zz
    g = (lp - lm) / (2.0 * eps)
    for B, zz in zip(Bs, z):
        B -= lr * g * zz
    return np.array([lp, lm]), g, Bs


def mobile_mp_lora_forward(x, W, A, B_pair, z_new, g, eps, lr):
    """Mobile MP-LoRA module (Algorithm 2, q = 1): the stored pair B[0], B[1]
    carries the previous perturbation; the previous step's update and the new
    +-eps z are applied inside the forward.  x [2,T,k]; B_pair [2,r,k_out];
    z_new is the standard-normal draw.  Returns (output [2,T,k_out], new pair)."""
    diff = (B_pair[0] - B_pair[1]) / 2.0
    update = lr * g * diff / eps
    z = eps * z_new
    B0 = B_pair[0] - diff - update + z
    B1 = B_pair[1] + diff - update - z
    Bn = np.stack([B0, B1])
    out = x @ np.asarray(W, np.float64).T + np.matmul(x @ np.asarray(A, np.float64).T, Bn)
    return out, Bn
