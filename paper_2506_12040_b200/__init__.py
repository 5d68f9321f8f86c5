"""B200 (sm_100a) codebook-binary linear layer: Python names for the C ABI in include/btc.h."""
from .binding import (  # noqa: F401
    BtcError,
    GemvBatch,
    bits_per_weight,
    codebook_pack,
    codebook_pack_host,
    decode_pm1,
    device_status,
    lib,
    linear,
    linear_gemm,
    linear_gemm_static_scratch,
    linear_gemv,
    linear_gemv_batch,
    linear_workspace_bytes,
    validate_indices,
)
