"""Pins for the oracle's forward passes against library implementations
(transformers' OPT / Llama, torch's cross entropy).  CPU only."""
import numpy as np
import pytest
import torch

from oracle import model as om
from workloads import ModelSpec, make_decoder_problem, make_linear_problem
from workloads.spec import (ARCH_LINEAR, ARCH_LLAMA, ARCH_OPT, LOSS_CE_FULL,
                            LOSS_CE_LABEL_WORDS, LOSS_MSE, TARGET_K, TARGET_Q, TARGET_V)


def _t(x):
    return torch.tensor(np.asarray(x, np.float64))


def _merged(spec, L, Bl):
    """Fold s * (A^T B)^T into the adapted sections of the fused qkv weight."""
    d, r = spec.d_model, spec.lora_rank
    W = np.asarray(L["w_qkv"], np.float64).copy()
    for t, sec in enumerate(spec.target_sections):
        A = np.asarray(L["A"][t * r:(t + 1) * r], np.float64)
        W[sec * d:(sec + 1) * d] += spec.lora_scale * (Bl[t].T @ A)
    return W


def _hf_logits(spec, p, Bs, tokens):
    from transformers import LlamaConfig, LlamaForCausalLM, OPTConfig, OPTForCausalLM
    d = spec.d_model
    if spec.arch == ARCH_OPT:
        cfg = OPTConfig(vocab_size=spec.vocab, hidden_size=d, num_hidden_layers=spec.n_layers,
                        ffn_dim=spec.d_ffn, max_position_embeddings=spec.max_seq,
                        num_attention_heads=spec.n_heads, word_embed_proj_dim=d,
                        do_layer_norm_before=True, activation_function="relu", dropout=0.0,
                        attention_dropout=0.0, layerdrop=0.0)
        m = OPTForCausalLM(cfg).double().eval()
        sd = {"model.decoder.embed_tokens.weight": _t(p["tok_emb"]),
              "lm_head.weight": _t(p["tok_emb"]),
              "model.decoder.final_layer_norm.weight": _t(p["final_norm_g"]),
              "model.decoder.final_layer_norm.bias": _t(p["final_norm_b"])}
        pos = np.zeros((spec.max_seq + 2, d))
        pos[2:] = p["pos_emb"]                      # the library offsets positions by 2
        sd["model.decoder.embed_positions.weight"] = _t(pos)
        for l, L in enumerate(p["layers"]):
            W = _merged(spec, L, Bs[l])
            pre = f"model.decoder.layers.{l}."
            for j, nm in enumerate(("q_proj", "k_proj", "v_proj")):
                sd[pre + f"self_attn.{nm}.weight"] = _t(W[j * d:(j + 1) * d])
                sd[pre + f"self_attn.{nm}.bias"] = _t(L["b_qkv"][j * d:(j + 1) * d])
            sd[pre + "self_attn.out_proj.weight"] = _t(L["w_o"])
            sd[pre + "self_attn.out_proj.bias"] = _t(L["b_o"])
            sd[pre + "self_attn_layer_norm.weight"] = _t(L["norm1_g"])
            sd[pre + "self_attn_layer_norm.bias"] = _t(L["norm1_b"])
            sd[pre + "final_layer_norm.weight"] = _t(L["norm2_g"])
            sd[pre + "final_layer_norm.bias"] = _t(L["norm2_b"])
            sd[pre + "fc1.weight"], sd[pre + "fc1.bias"] = _t(L["w_fc1"]), _t(L["b_fc1"])
            sd[pre + "fc2.weight"], sd[pre + "fc2.bias"] = _t(L["w_fc2"]), _t(L["b_fc2"])
    else:
        cfg = LlamaConfig(vocab_size=spec.vocab, hidden_size=d, intermediate_size=spec.d_ffn,
                          num_hidden_layers=spec.n_layers, num_attention_heads=spec.n_heads,
                          num_key_value_heads=spec.n_heads, max_position_embeddings=spec.max_seq,
                          rms_norm_eps=spec.norm_eps, rope_theta=spec.rope_theta,
                          tie_word_embeddings=False, attention_bias=False, mlp_bias=False)
        m = LlamaForCausalLM(cfg).double().eval()
        sd = {"model.embed_tokens.weight": _t(p["tok_emb"]), "lm_head.weight": _t(p["lm_head"]),
              "model.norm.weight": _t(p["final_norm_g"])}
        f = spec.d_ffn
        for l, L in enumerate(p["layers"]):
            W = _merged(spec, L, Bs[l])
            pre = f"model.layers.{l}."
            for j, nm in enumerate(("q_proj", "k_proj", "v_proj")):
                sd[pre + f"self_attn.{nm}.weight"] = _t(W[j * d:(j + 1) * d])
            sd[pre + "self_attn.o_proj.weight"] = _t(L["w_o"])
            sd[pre + "input_layernorm.weight"] = _t(L["norm1_g"])
            sd[pre + "post_attention_layernorm.weight"] = _t(L["norm2_g"])
            sd[pre + "mlp.gate_proj.weight"] = _t(L["w_fc1"][:f])
            sd[pre + "mlp.up_proj.weight"] = _t(L["w_fc1"][f:])
            sd[pre + "mlp.down_proj.weight"] = _t(L["w_fc2"])
    missing, unexpected = m.load_state_dict(sd, strict=False)
    assert not unexpected, unexpected
    assert all("rotary" in k or "inv_freq" in k for k in missing), missing
    with torch.no_grad():
        return m(input_ids=torch.tensor(tokens, dtype=torch.long)).logits.numpy()


SMALL = dict(n_layers=2, d_model=32, n_heads=4, d_ffn=48, vocab=61, max_seq=12,
             lora_rank=4, E=3, S=12, n_labelled=5, bf16=False)


@pytest.mark.parametrize("arch,targets,scale", [
    (ARCH_OPT, TARGET_Q | TARGET_V, 1.0),
    (ARCH_LLAMA, TARGET_Q | TARGET_V, 2.0),
    (ARCH_LLAMA, TARGET_Q | TARGET_K | TARGET_V, 1.0),
    (ARCH_OPT, TARGET_V, 0.5),
])
def test_decoder_matches_transformers_with_merged_lora(arch, targets, scale):
    spec = ModelSpec(arch=arch, lora_targets=targets, lora_scale=scale,
                     tie_lm_head=(arch == ARCH_OPT), **SMALL)
    p = make_decoder_problem(spec, seed=3, b_std=0.05)
    Bs = [np.asarray(L["B"], np.float64) for L in p["layers"]]
    logits = _hf_logits(spec, p, Bs, p["tokens"])            # [E,S,V]
    lab = torch.tensor(p["labels"].reshape(-1), dtype=torch.long)
    ref = torch.nn.functional.cross_entropy(torch.tensor(logits).reshape(-1, spec.vocab), lab,
                                            ignore_index=-1, reduction="mean").item()
    got, rows = om.replica_losses(spec, p, [b[None] for b in Bs], p["tokens"], p["labels"],
                                  return_rows=True)
    assert got.shape == (1,)
    # the library builds its rotary tables in fp32, hence 1e-7 rather than 1e-12
    assert abs(got[0] - ref) < 1e-7 * abs(ref)
    ref_rows = torch.nn.functional.cross_entropy(
        torch.tensor(logits).reshape(-1, spec.vocab), lab, ignore_index=-1, reduction="none")
    ref_rows = ref_rows[lab >= 0].numpy()
    assert np.allclose(rows[0], ref_rows, rtol=1e-7, atol=0)
    assert (p["labels"] >= 0).sum() == spec.E * spec.n_labelled


def test_label_word_loss_matches_two_way_cross_entropy():
    spec = ModelSpec(arch=ARCH_OPT, tie_lm_head=True, loss_kind=LOSS_CE_LABEL_WORDS,
                     label_words=(7, 40), **SMALL)
    p = make_decoder_problem(spec, seed=5, b_std=0.05)
    Bs = [np.asarray(L["B"], np.float64) for L in p["layers"]]
    logits = _hf_logits(spec, p, Bs, p["tokens"])[:, -1, :][:, list(spec.label_words)]
    cls = torch.tensor(p["labels"][:, -1], dtype=torch.long)
    ref = torch.nn.functional.cross_entropy(torch.tensor(logits), cls).item()
    got = om.replica_losses(spec, p, [b[None] for b in Bs], p["tokens"], p["labels"])
    assert abs(got[0] - ref) < 1e-10
    assert set(np.unique(p["labels"][:, -1])) <= {0, 1} and np.all(p["labels"][:, :-1] == -1)


def test_linear_mse_matches_torch():
    spec = ModelSpec(arch=ARCH_LINEAR, d_model=24, d_out=20, lora_rank=4, lora_scale=2.0,
                     loss_kind=LOSS_MSE, bf16=False, E=2, S=5)
    p = make_linear_problem(spec, seed=9, b_std=0.1)
    Bn = np.stack([p["B"], 2 * p["B"]]).astype(np.float64)
    got = om.replica_losses(spec, p, Bn, p["X"], p["target"])
    X, W, A = _t(p["X"]), _t(p["W"]), _t(p["A"])
    for n in range(2):
        Y = torch.nn.functional.linear(X, W + 2.0 * (_t(Bn[n]).T @ A), _t(p["bias"]))
        ref = torch.nn.functional.mse_loss(Y, _t(p["target"])).item()
        assert abs(got[n] - ref) < 1e-12 * max(1.0, ref)


def test_mp_lora_layer_equals_per_path_dense_layers():
    """Y^(n) = X^(n) W + (X^(n) A) (.) B^(n): path i sees W + A B_i only."""
    rng = np.random.default_rng(0)
    n, T, ki, ko, r = 3, 5, 7, 6, 2
    X = rng.standard_normal((n, T, ki))
    W, A = rng.standard_normal((ko, ki)), rng.standard_normal((r, ki))
    Bn = rng.standard_normal((n, r, ko))
    Y = om.mp_lora_linear(X, W, None, A, Bn, 1.0)
    for i in range(n):
        assert np.allclose(Y[i], X[i] @ (W.T + A.T @ Bn[i]), rtol=1e-12, atol=1e-12)


def test_random_init_loss_is_log_vocab():
    spec = ModelSpec(arch=ARCH_LLAMA, **{**SMALL, "vocab": 997, "d_model": 64, "n_heads": 4})
    p = make_decoder_problem(spec, seed=1)
    Bs = [np.asarray(L["B"], np.float64)[None] for L in p["layers"]]
    got = om.replica_losses(spec, p, Bs, p["tokens"], p["labels"])[0]
    assert abs(got - np.log(997)) < 0.1 * np.log(997)
