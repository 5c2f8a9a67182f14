"""fp64 CPU oracle of the EmbedPart hot path -- TEST INFRASTRUCTURE, not the product.

Only ``tests/``, the smoke check and the CPU-baseline leg of ``bench.py`` may
import this package.  It never imports the CUDA package and the CUDA package
never imports it.
"""
from .ep_oracle import (  # noqa: F401
    build,
    kmeans,
    assign_step,
    sampled_kmeans,
    partition_quality,
    reorder,
    graph_bandwidth,
    relabel_graph,
    migrate,
    balance,
    cluster_and_balance,
    permute_rows,
    num_threads,
    set_num_threads,
)
