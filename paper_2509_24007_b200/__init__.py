"""B200-native hot path of the SDLM Next-Sequence-Prediction decode step.

The product is the C-ABI library ``libsdlm.so`` (see ``include/sdlm.h``); this package is the
thin Python binding over it.  PyTorch is used only for device memory and streams.
"""
from .binding import (CONF_ENTROPY, CONF_LOGIT, Sdlm, SdlmConfig, SdlmError, bf16_tensor_from_bits,
                      bits_from_bf16_tensor, load_library)

__all__ = ["Sdlm", "SdlmConfig", "SdlmError", "CONF_LOGIT", "CONF_ENTROPY", "load_library",
           "bf16_tensor_from_bits", "bits_from_bf16_tensor"]
