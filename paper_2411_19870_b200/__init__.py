"""B200-native DeMo optimizer transform (arXiv 2411.19870): thin Python binding over the C ABI.

The product is ``libdemo_b200.so`` (hand-written CUDA for sm_100a behind ``include/demo.h``).
This package only marshals arguments: every step of the path runs in the library's kernels.
"""
# ``paper_2411_19870_b200.distributed`` (one worker per rank, all-gather of the payloads) is imported on
# demand: it needs ``torch.distributed``.
from .binding import (  # noqa: F401
    DEMO_BF16,
    DEMO_F32,
    DEMO_AGG_COUNT_MEAN,
    DEMO_AGG_MEAN,
    DEMO_AGG_SUM,
    DEMO_MOMENTUM_DCT,
    DEMO_MOMENTUM_SPATIAL,
    DEMO_PATH_AUTO,
    DEMO_PHI_IDENTITY,
    DEMO_PHI_SIGN,
    DEMO_PATH_GENERIC,
    DemoConfig,
    DemoError,
    DemoTensorDesc,
    DemoTransform,
    RECORD_BYTES,
    decode_apply_static,
    demo_status_string,
    load_library,
)
