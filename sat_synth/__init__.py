"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests / bench.

This package only *draws inputs*: graphs, features, labels, initial weights and the
partition assignment that a workload prescribes.  It contains none of the method's
arithmetic (no normalisation, no aggregation, no predictor, no cache logic), so both
sides can consume it without sharing any of their own code.
"""
from .graphs import sbm_graph, rmat_graph, bfs_relabel, csr_from_undirected_pairs
from .tensors import (normal_features, uniform_labels, bernoulli_labels, glorot_uniform, stream_rng, embedding_table,
                      table_rows)
from .workloads import WORKLOADS, Workload, as_gru, make_workload

__all__ = [
    "sbm_graph", "rmat_graph", "bfs_relabel", "csr_from_undirected_pairs",
    "normal_features", "uniform_labels", "bernoulli_labels", "glorot_uniform", "stream_rng", "embedding_table", "table_rows",
    "WORKLOADS", "Workload", "make_workload",
]
