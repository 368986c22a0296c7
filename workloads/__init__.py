"""Seeded synthetic inputs for the R-FAST activation engine.

This package only *generates inputs*: communication graphs with their weight
matrices, raw activation / delay / drop schedules, data shards and minibatch
indices.  It holds none of the method's arithmetic (no descent, mixing,
tracking or gradient code).  Both the CPU oracle's tests and the CUDA
library's tests feed on the arrays produced here; the oracle and the CUDA
path never import each other.
"""

from .graphs import (Graph, graph_from_edges, ring_graphs, tree_graphs,
                     binary_tree_parents, exponential_tree_parents,
                     random_tree_parents, sender_csr)
from .schedules import (Schedule, make_schedule, make_schedule_ack_gated, split_schedule, activation_bernoulli,
                        activation_uniform_subset, activation_durations,
                        activation_all, realised_T_D)
from .configs import CONFIG_NAMES, build_config, shard_coordinates, Workload

__all__ = [
    "Graph", "graph_from_edges", "ring_graphs", "tree_graphs",
    "binary_tree_parents", "exponential_tree_parents", "random_tree_parents",
    "sender_csr", "Schedule", "make_schedule", "make_schedule_ack_gated", "split_schedule", "activation_bernoulli",
    "activation_uniform_subset", "activation_durations", "activation_all",
    "realised_T_D", "CONFIG_NAMES", "build_config", "shard_coordinates", "Workload",
]
