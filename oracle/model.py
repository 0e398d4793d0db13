"""Forward passes of the MP-LoRA models in fp64 (test infrastructure).

Every adapted linear follows the MP-LoRA layer equation of the paper's
"MP-LoRA" paragraph, Y^(n) = X^(n) W + (X^(n) A) (.) B^(n), with W and A shared
by the n paths and (.) a batched matmul against the per-path B.  Tensors are
stored transposed with respect to the paper (W [k_out,k_in], A [r,k_in]);
`lora_scale` multiplies the low-rank term (1.0 = the equation as printed).

The decoder families are the stock ones the paper fine-tunes (OPT, Llama); the
paper does not restate them, so they are pinned against the `transformers`
library in the tests.
"""
import numpy as np

from .quant import weight as _wq

ARCH_LINEAR, ARCH_OPT, ARCH_LLAMA = 0, 1, 2
LOSS_MSE, LOSS_CE_FULL, LOSS_CE_LABEL_WORDS = 0, 1, 2


def _f64(x):
    return np.asarray(x, dtype=np.float64)


def mp_lora_linear(X, W, bias, A, Bn, scale):
    """MP-LoRA layer ("MP-LoRA" paragraph, layer equation).
    X [n,T,k_in]; W [k_out,k_in]; A [r,k_in]; Bn [n,r,k_out] -> [n,T,k_out]."""
    Y = X @ _f64(W).T
    if bias is not None:
        Y = Y + _f64(bias)
    U = X @ _f64(A).T                       # shared down-projection
    return Y + scale * np.matmul(U, Bn)     # batched over the n paths


def _layer_norm(x, g, b, eps):
    mu = x.mean(-1, keepdims=True)
    var = ((x - mu) ** 2).mean(-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * _f64(g) + _f64(b)


def _rms_norm(x, g, eps):
    return x / np.sqrt((x * x).mean(-1, keepdims=True) + eps) * _f64(g)


def _rope(x, theta):
    """x [n,E,S,H,dh]; rotate-half pairing (j, j+dh/2), angle = pos * theta^(-2j/dh)."""
    S, dh = x.shape[2], x.shape[4]
    half = dh // 2
    inv = theta ** (-2.0 * np.arange(half, dtype=np.float64) / dh)
    ang = np.arange(S, dtype=np.float64)[:, None] * inv[None, :]      # [S,half]
    c, s = np.cos(ang)[None, None, :, None, :], np.sin(ang)[None, None, :, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def _causal_attention(q, k, v):
    """q,k,v [n,E,S,H,dh] -> [n,E,S,H,dh]; softmax(q k^T / sqrt(dh) + causal) v."""
    dh, S = q.shape[-1], q.shape[2]
    sc = np.einsum("nethd,neshd->nehts", q, k) / np.sqrt(dh)
    mask = np.triu(np.ones((S, S), bool), 1)
    sc = np.where(mask, -np.inf, sc)
    sc = sc - sc.max(-1, keepdims=True)
    p = np.exp(sc)
    p = p / p.sum(-1, keepdims=True)
    return np.einsum("nehts,neshd->nethd", p, v)


def _section_lora(spec, L, Bn_layer, d):
    """Expand the per-target A/B of one layer to per-section (q,k,v) entries."""
    r = spec.lora_rank
    out = {}
    for t, sec in enumerate(spec.target_sections):
        out[sec] = (L["A"][t * r:(t + 1) * r], Bn_layer[:, t])
    return out


def _qkv(spec, L, x, Bn_layer):
    d = spec.d_model
    lora = _section_lora(spec, L, Bn_layer, d)
    Wqkv = _wq(L["w_qkv"], spec.bf16)
    outs = []
    for sec in range(3):
        W = Wqkv[sec * d:(sec + 1) * d]
        b = L["b_qkv"][sec * d:(sec + 1) * d] if "b_qkv" in L else None
        if sec in lora:
            A, Bn = lora[sec]
            outs.append(mp_lora_linear(x, W, b, A, Bn, spec.lora_scale))
        else:
            y = x @ _f64(W).T
            outs.append(y if b is None else y + _f64(b))
    return outs


def decoder_hidden(spec, p, Bn, tokens):
    """Final hidden states [n,T,d] (before the final norm) of n paths that
    share the tokens [E,S]; Bn[l] is [n, n_targets, r, d]."""
    E, S = tokens.shape
    n = Bn[0].shape[0]
    d, H = spec.d_model, spec.n_heads
    dh = d // H
    h = _f64(p["tok_emb"])[tokens.reshape(-1)]
    if spec.arch == ARCH_OPT:
        h = h + np.tile(_f64(p["pos_emb"])[:S], (E, 1))
    h = np.broadcast_to(h, (n, E * S, d)).copy()          # X^(n): n copies of the batch
    for l, L in enumerate(p["layers"]):
        if spec.arch == ARCH_OPT:
            x = _layer_norm(h, L["norm1_g"], L["norm1_b"], spec.norm_eps)
        else:
            x = _rms_norm(h, L["norm1_g"], spec.norm_eps)
        q, k, v = [t.reshape(n, E, S, H, dh) for t in _qkv(spec, L, x, Bn[l])]
        if spec.arch == ARCH_LLAMA:
            q, k = _rope(q, spec.rope_theta), _rope(k, spec.rope_theta)
        ctx = _causal_attention(q, k, v).reshape(n, E * S, d)
        o = ctx @ _wq(L["w_o"], spec.bf16).T
        if "b_o" in L:
            o = o + _f64(L["b_o"])
        h = h + o
        if spec.arch == ARCH_OPT:
            x = _layer_norm(h, L["norm2_g"], L["norm2_b"], spec.norm_eps)
            a = np.maximum(x @ _wq(L["w_fc1"], spec.bf16).T + _f64(L["b_fc1"]), 0.0)
            h = h + a @ _wq(L["w_fc2"], spec.bf16).T + _f64(L["b_fc2"])
        else:
            x = _rms_norm(h, L["norm2_g"], spec.norm_eps)
            gu = x @ _wq(L["w_fc1"], spec.bf16).T
            g, u = gu[..., :spec.d_ffn], gu[..., spec.d_ffn:]
            a = g / (1.0 + np.exp(-g)) * u                 # SiLU(gate) * up
            h = h + a @ _wq(L["w_fc2"], spec.bf16).T
    return h


def _log_softmax(z):
    z = z - z.max(-1, keepdims=True)
    return z - np.log(np.exp(z).sum(-1, keepdims=True))


def row_losses(spec, p, h, labels):
    """Per labelled row losses [n, rows] (rows in (b,t) order) from hidden [n,T,d]."""
    lab = labels.reshape(-1)
    rows = np.nonzero(lab >= 0)[0]
    x = h[:, rows]
    if spec.arch == ARCH_OPT:
        x = _layer_norm(x, p["final_norm_g"], p["final_norm_b"], spec.norm_eps)
    else:
        x = _rms_norm(x, p["final_norm_g"], spec.norm_eps)
    head = _f64(p["tok_emb"] if spec.tie_lm_head else p["lm_head"])
    if spec.loss_kind == LOSS_CE_FULL:
        # loss over the whole vocabulary (Experiment Setup appendix)
        lp = _log_softmax(x @ head.T)
        return -np.take_along_axis(lp, lab[rows][None, :, None], axis=-1)[..., 0]
    w = np.asarray(spec.label_words)
    lp = _log_softmax(x @ head[w].T)                       # two label-word logits
    return -np.take_along_axis(lp, lab[rows][None, :, None], axis=-1)[..., 0]


def replica_losses(spec, p, Bn, tokens, labels, return_rows=False):
    """Scalar loss of each of the n paths, l^(k) = L((theta_l^(k), theta_f); B)
    (Algorithm 1, inner loop): mean over the labelled positions of the batch.

    ARCH_LINEAR: p has W,bias,A; `tokens` is X [T,k_in], `labels` the target
    [T,k_out]; Bn is [n,r,k_out]; loss = mean squared error."""
    if spec.arch == ARCH_LINEAR:
        X = _f64(tokens)[None]
        Y = mp_lora_linear(np.broadcast_to(X, (Bn.shape[0],) + X.shape[1:]), p["W"],
                           p.get("bias"), p["A"], _f64(Bn), spec.lora_scale)
        per = ((Y - _f64(labels)[None]) ** 2).mean(-1)    # [n,T]
        return (per.mean(-1), per) if return_rows else per.mean(-1)
    Bn = [_f64(b) for b in Bn]
    if isinstance(tokens, (list, tuple)):
        # ragged batch (no padding): every sequence is its own forward pass of its own length; the
        # loss is still the mean over all labelled positions of the batch
        parts = [row_losses(spec, p, decoder_hidden(spec, p, Bn, np.asarray(t)[None]), np.asarray(l)[None])
                 for t, l in zip(tokens, labels)]
        rl = np.concatenate(parts, axis=1)
        return (rl.mean(-1), rl) if return_rows else rl.mean(-1)
    h = decoder_hidden(spec, p, Bn, np.asarray(tokens))
    rl = row_losses(spec, p, h, np.asarray(labels))
    return (rl.mean(-1), rl) if return_rows else rl.mean(-1)
