"""CoS verification step for B200: Python binding over the C-ABI CUDA library.

`binding` marshals arguments into `libcos_verify.so` (every step of the path runs in the
CUDA kernels; there is no CPU fallback), `synth` makes the seeded synthetic workloads,
`sharding` splits a batch of rows over ranks.
"""
from .binding import (  # noqa: F401
    COS_COMBINE_LOGIT_LINEAR,
    COS_COMBINE_PROB_ENSEMBLE,
    COS_DTYPE_BF16,
    COS_DTYPE_F16,
    COS_DTYPE_F32,
    COS_ROW_BAD_DRAFT,
    COS_ROW_FAULT,
    COS_ROW_NONFINITE,
    COS_ROW_Q_ZERO,
    COS_ROW_RESIDUAL_EMPTY,
    COS_RUN_ALL_RESIDUALS,
    COS_RUN_BONUS_FROM_MODEL,
    COS_RUN_EARLY_EXIT,
    COS_RUN_INPUTS_SETTLED,
    COS_RUN_PROPOSER_PER_POSITION,
    CosVerifier,
    CosVerifyError,
    load_library,
)
