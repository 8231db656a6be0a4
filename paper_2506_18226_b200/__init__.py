"""B200-native ADSA decode attention: CUDA kernels behind a C-ABI (libadsa.so) plus a thin binding."""
from .binding import (  # noqa: F401
    AdsaBuffers,
    AdsaConfig,
    AdsaEngine,
    AdsaError,
    EXPORTS,
    cfg_sample,
    decode_attn_static,
    load,
    rmsnorm,
    strerror,
    swiglu,
    workspace_bytes,
)
from .build import build_lib  # noqa: F401
