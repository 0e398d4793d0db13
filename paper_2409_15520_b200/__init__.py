"""B200-native parallelised zeroth-order (MobiZO-style) gradient estimator.

Thin Python binding over the C ABI of ``libzo_b200.so`` (see ``include/zo.h``).
All computation runs in the CUDA library; PyTorch is used for device memory and
streams only.  Importing this package loads the library and fails loudly if it
has not been built (``python paper_2409_15520_b200/build.py``).
"""
from .binding import (  # noqa: F401
    LIB, ZoConfig, ZoError, Estimator, DeviceProblem, make_config, perturbation,
    mp_lora_linear, mp_lora_linear_static, mp_lora_linear_pair, STATUS_NAMES,
)
from .sharding import query_shard, exchange_losses, exchange_step, sharded_step  # noqa: F401
