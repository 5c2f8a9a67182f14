"""B200 (sm_100a) library for the hot path of embedding-driven graph partitioning: Lloyd K-Means
over node embeddings, edge-cut / balance scoring and partition-ordered reordering.

All computation happens in the CUDA library behind ``include/embedpart.h``; this package only
marshals torch tensors into that C ABI.  There is no CPU fallback: importing works anywhere, but
any call needs the built library and a B200.
"""
from .binding import (  # noqa: F401
    EmbedPartError,
    Context,
    default_context,
    ep_kmeans,
    ep_partition_quality,
    ep_reorder,
    ep_reorder_static,
    ep_graph_bandwidth,
    ep_kmeans_sampled,
    library_path,
    load_library,
    EXPORTED_SYMBOLS,
)
