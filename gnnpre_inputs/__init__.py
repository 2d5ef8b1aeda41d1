"""Seeded synthetic graphs and features shared by the tests, the benchmark and the
CPU oracle's callers.  Nothing here computes any part of the propagation method."""
from .configs import OP_GCN, OP_GIN, OP_SAGE, WORKLOADS, Workload, make_features, make_graph, scaled  # noqa: F401
from .features import normal_matrix, normal_rows  # noqa: F401
from .graphs import CSRGraph, erdos_renyi, from_edge_list, rmat  # noqa: F401
