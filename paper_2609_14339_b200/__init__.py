"""B200-native spectral-correction optimizer step: thin Python binding over the C-ABI CUDA library."""
from .binding import (Plan, SCError, project_static, apply_prf_mask, masked_weight_grad, lowrank_compress, lowrank_init_q, Hparams, lib_path, load_library, status_string,  # noqa: F401
                      SC_DTYPE_BF16, SC_DTYPE_FP32, SC_ENGINE_AUTO, SC_ENGINE_SIMT, SC_OK, SC_WARN_NO_ANCHOR,
                      SC_OPT_ADAMW, SC_OPT_ADEMAMIX)
