"""ApproxIFER encode / decode / locate for NVIDIA B200 (sm_100a).

The product is the C-ABI shared library ``libapproxifer.so`` (declared in
``include/approxifer.h``, sources in ``csrc/``); this package is its thin
Python binding plus the seeded workload generators used by the tests and the
benchmark.
"""
from .binding import (  # noqa: F401
    ApproxiferError,
    approxifer_debug_weights,
    approxifer_decode,
    approxifer_decode_bf16,
    approxifer_decode_gather,
    approxifer_encode_scatter,
    approxifer_locate_gather,
    approxifer_encode_bf16,
    approxifer_decode_rational,
    approxifer_encode,
    approxifer_encode_host,
    approxifer_encode_host_static,
    approxifer_decode_host,
    approxifer_locate_host,
    approxifer_locate,
    approxifer_locate_decode,
    approxifer_params,
    approxifer_decode_tuning,
    decode_tuning,
    debug_fma_peak,
    debug_pack_rotation,
    device_wait_timeouts,
    reset_device_wait_timeouts,
    launch_count,
    library_path,
    load,
    make_params,
    mask_tensor,
    strerror,
    version,
)
