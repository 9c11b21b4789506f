"""B200-native training of PAC+ Parallel Adapters over an activation cache.

The work happens in hand-written sm_100a CUDA kernels behind a C ABI
(include/pac.h, built into libpac_b200.so); this package is the thin binding.
"""
from .binding import (PacError, PacContext, AdamW, load_library, PAC_F32, PAC_BF16, PAC_ACT_RELU,  # noqa: F401
                      PAC_ACT_IDENTITY, PAC_HEAD_MEANPOOL_CLS, PAC_HEAD_FROZEN_LM, STATUS_NAMES, EXPORTS, eval_logits_static, quantize_absmax, dequantize_absmax,
                      CacheWriter, cache_file_info, PAC_BODY_POINTWISE, PAC_BODY_TRANSFORMER)
