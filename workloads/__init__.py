"""Seeded synthetic inputs for the link-prediction training step.

This package produces *data only*: graphs in CSR form, node features, model
parameters, edge splits and node-to-partition assignments.  It contains none
of the method's arithmetic (no aggregation, no normalisation, no sampling of
negatives or neighbours, no sparsification), so both the CUDA library and the
CPU oracle can be fed from it without sharing any code of the method.

Graph convention used everywhere: CSR rows are *destination* nodes v and the
columns of a row are the in-neighbours u of v (the nodes whose embeddings v
aggregates, N(v) in Eq. 1), sorted ascending, without duplicates and without
self-loops.  ``rowptr`` is int64, ``col`` is int32, weights are float32.
"""
from .graphs import (  # noqa: F401
    Graph,
    csr_from_edges,
    erdos_renyi,
    chung_lu,
    coauthor_weighted,
    citation_directed,
    node_features,
    model_dims_param_count,
    glorot_params,
    edge_split,
    random_partition,
    induced_subgraph,
    undirected_edge_list,
    CONFIGS,
    make_config,
)
