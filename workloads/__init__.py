"""Seeded synthetic inputs for the paged graph-ANNS hot path.

This package only *makes inputs*: vectors, a navigation graph, the paged node
store, PQ codebooks/codes and brute-force ground truth.  It contains none of the
beam search itself, and it is the only module shared by the CPU oracle's tests
and the CUDA path's tests/benchmarks.
"""
from .synthetic import (  # noqa: F401
    Workload,
    PAGE_BYTES,
    gen_u8,
    gen_f32,
    knn_graph,
    medoid,
    node_bytes,
    write_page_store,
    parse_page_store,
    train_pq,
    ground_truth,
    make_workload,
    make_config,
    recall_at_k,
    workload_key,
)
