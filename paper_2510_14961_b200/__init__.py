"""B200-native diffusion-forcing sampler step for recurrent-depth transformers (C ABI + binding)."""
from .binding import (Model, Session, RdError, lib, LIB_PATH, EXPORTS, RD_F32, RD_BF16, RD_OK,  # noqa: F401
                      RD_E_INVALID_ARG, RD_E_STATE, RD_E_CAPACITY, RD_E_OOM, RD_E_CUDA, RD_E_TIMEOUT,
                      RD_DBG_LATENTS, RD_DBG_DELTA, RD_DBG_DRAFTS, RD_DBG_LOGITS, RD_DBG_EMBED)
