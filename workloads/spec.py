"""Shape records of the workloads (no arithmetic).

The five named configurations follow the paper's experimental grid: fixed
sequence lengths 64/128/256 with batch sizes 1..16 (memory and runtime tables
of the System Performance section), LoRA-FA on attention projections with a
small rank (Hyper-parameter appendix), and model families OPT and Llama.
"""
from dataclasses import dataclass, field, replace
from typing import Tuple

ARCH_LINEAR, ARCH_OPT, ARCH_LLAMA = 0, 1, 2
LOSS_MSE, LOSS_CE_FULL, LOSS_CE_LABEL_WORDS = 0, 1, 2
TARGET_Q, TARGET_K, TARGET_V = 1, 2, 4


@dataclass(frozen=True)
class ModelSpec:
    arch: int
    n_layers: int = 1
    d_model: int = 256          # ARCH_LINEAR: k_in
    d_out: int = 256            # ARCH_LINEAR only: k_out
    n_heads: int = 1
    d_ffn: int = 0
    vocab: int = 0
    max_seq: int = 256
    lora_rank: int = 8
    lora_scale: float = 1.0
    lora_targets: int = TARGET_Q | TARGET_V
    loss_kind: int = LOSS_CE_FULL
    label_words: Tuple[int, int] = (0, 1)
    norm_eps: float = 1e-5
    rope_theta: float = 10000.0
    tie_lm_head: bool = False
    bf16: bool = True           # storage type of frozen tensors and activations
    # workload part (per-step arguments of the estimator)
    E: int = 1                  # sequences in the shared batch
    S: int = 32                 # sequence length
    q: int = 1                  # queries
    eps: float = 1e-3
    lr: float = 1e-3
    n_labelled: int = 1         # labelled positions per sequence (last ones)

    @property
    def n_targets(self) -> int:
        return bin(self.lora_targets & 7).count("1")

    @property
    def target_sections(self):
        """Indices (0=q,1=k,2=v) of the adapted sections, ascending."""
        return [j for j in range(3) if (self.lora_targets >> j) & 1]

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_heads

    def with_(self, **kw) -> "ModelSpec":
        return replace(self, **kw)


CONFIGS = {
    # single MP-LoRA linear, MSE loss, fp32 storage
    "linear_fp32": ModelSpec(arch=ARCH_LINEAR, d_model=256, d_out=256, lora_rank=8,
                             loss_kind=LOSS_MSE, bf16=False, E=4, S=32, q=2,
                             eps=1e-3, lr=1e-3),
    "opt125m": ModelSpec(arch=ARCH_OPT, n_layers=12, d_model=768, n_heads=12, d_ffn=3072,
                         vocab=50272, max_seq=128, lora_rank=8, tie_lm_head=True,
                         E=8, S=128, q=4, eps=1e-3, lr=1e-3, n_labelled=16),
    "opt1p3b": ModelSpec(arch=ARCH_OPT, n_layers=24, d_model=2048, n_heads=32, d_ffn=8192,
                         vocab=50272, max_seq=256, lora_rank=8, tie_lm_head=True,
                         loss_kind=LOSS_CE_LABEL_WORDS, label_words=(1037, 29042),
                         E=16, S=256, q=8, eps=1e-3, lr=1e-3, n_labelled=1),
    "llama7b": ModelSpec(arch=ARCH_LLAMA, n_layers=32, d_model=4096, n_heads=32, d_ffn=11008,
                         vocab=32000, max_seq=256, lora_rank=16, tie_lm_head=False,
                         E=16, S=256, q=16, eps=1e-3, lr=1e-3, n_labelled=32),
    # MP-LoRA linear micro-benchmark point (rank and q are swept by the caller)
    "linear_sweep": ModelSpec(arch=ARCH_LINEAR, d_model=4096, d_out=4096, lora_rank=16,
                              loss_kind=LOSS_MSE, bf16=True, E=16, S=256, q=4),
}


def config(name: str, **overrides) -> ModelSpec:
    return CONFIGS[name].with_(**overrides)
