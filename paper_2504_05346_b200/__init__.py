"""B200-native hot path of the Thanos block-wise pruning method (arXiv 2504.05346).

The product is ``libthanos.so`` (hand-written CUDA for sm_100a behind the C ABI declared in
``include/thanos.h``).  This package only marshals arguments: PyTorch supplies device memory
and streams, every step of the path runs in the library's kernels.
"""

from .binding import (  # noqa: F401
    ThanosError,
    PruneStats,
    lib_path,
    load_library,
    hessian_accumulate,
    hessian_status,
    prepare_inverse,
    prune_layer,
    prune_block,
    prune_layer_host,
    prune_layer_noalloc,
    dense_product,
    fp32_fma_probe,
    prune_layer_outliers,
    prune_layer_structured,
    workspace_bytes,
    launch_count,
    status_string,
    version,
    F32,
    BF16,
    UNSTRUCTURED,
    NM,
)
