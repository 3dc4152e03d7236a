"""Top-K+phi residual-mass decode attention for B200 (sm_100a).

Thin Python binding over the C-ABI library ``libtkphi.so`` (see ``include/tkphi.h``).
Every step of the method runs in the library's CUDA kernels; this package only
marshals arguments.  There is no CPU fallback: calls raise if the library is
missing or no CUDA device is present.
"""
from .binding import (  # noqa: F401
    TkphiError,
    KVCache,
    PhiMaps,
    MlpMaps,
    mlp_key_features,
    build_summaries_cached,
    decode_step_mlp,
    WS_MLP_KEY_FEATURES,
    load_library,
    library_path,
    workspace_bytes,
    build_summaries,
    build_summaries_static,
    STATIC_SCRATCH_BYTES,
    topk_decode,
    decode_step,
    device_status,
    static_device_status,
    selftest_timeout,
    ERR_TIMEOUT,
    kernel_timing,
    KERNEL_KINDS,
    WS_BUILD,
    WS_TOPK_DECODE,
    WS_DECODE_STEP,
    FLAG_NONE,
    FLAG_NOSUB,
    EXPORTED_SYMBOLS,
)
