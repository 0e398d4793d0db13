"""CPU oracle of the parallelised zeroth-order estimator (TEST INFRASTRUCTURE).

Plain, slow, fp64 numpy code written from the paper's statement of the method.
It shares no code with the CUDA library and must never be imported by it; only
the tests, the smoke check and the benchmark's CPU-baseline leg call it.

Pins (see tests/test_oracle_*.py): Philox4x32-10 published known-answer
vectors; Box-Muller moments and closed-form points; decoder forward against
the `transformers` library's OPT and Llama implementations with LoRA merged
into the weights; closed-form gradient of the linear+MSE problem; quadratic
loss (exact central difference, variance slope in q); brute-force coordinate
finite differences; q=1 equals sequential in-place MeZO; the stored-pair
recurrences of the Mobile MP-LoRA module; batched MP-LoRA equals 2q
independent forwards; eps=0 degeneracy; NF4 levels against their normal-quantile construction,
INT8/NF4 round-trip bounds and hand-built packing.  No function here is left unpinned.
"""
from .philox import philox4x32_10, perturbation_u32, perturbation  # noqa: F401
from .model import replica_losses, mp_lora_linear  # noqa: F401
from .zo import zo_step, projected_gradients, zo_sgd_update, mezo_sequential_step, \
    mobile_mp_lora_forward  # noqa: F401
