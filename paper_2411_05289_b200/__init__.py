"""B200-native sampling-verification for multi-draft speculative decoding.

SpecHub (k = 2) with RRS / RRSw as the comparison path (arXiv 2411.05289), as
hand-written sm_100a CUDA kernels behind the C ABI declared in
``include/spechub.h``.  This package is the thin Python binding: it marshals
torch tensors (device memory, streams) into the C calls and does nothing else.
There is no CPU fallback: without the compiled library every call raises.
"""
from .binding import (  # noqa: F401
    ABI_VERSION,
    STATUS_BITS,
    SpecHubError,
    Tree,
    abi_version,
    library_path,
    load_library,
    mdsd_compare_draft_sample,
    mdsd_compare_draft_sample_stats,
    mdsd_compare_verify_tree,
    mdsd_compare_verify_tree_stats,
    rrs_draft_sample,
    rrs_draft_sample_stats,
    rrs_verify_tree,
    rrs_verify_tree_stats,
    set_row_split,
    spechub_draft_sample,
    spechub_draft_sample_stats,
    spechub_verify_tree,
    spechub_verify_tree_stats,
    spechub_verify_tree_static,
    status_string,
    workspace_bytes,
)
