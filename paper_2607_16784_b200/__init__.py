"""B200-native batched evaluation of Roomie's occupancy-based kernel-interference model.

Thin Python binding over ``libroomie.so`` (C ABI declared in ``include/roomie.h``):
argument marshalling only.  Every step of the path - occupancy (Section 3.1, Eq. 1), the
pairwise alignment walk with median and overlap factor (Section 3.2, Algorithm 1), the
greedy multi-model estimate and argmin placement (Algorithm 2) - runs in the library's CUDA
kernels.  PyTorch supplies device memory and streams, nothing else.

There is no CPU fallback: importing this package without the compiled library raises.
"""
from .roomie import (  # noqa: F401
    GpuSpec, Library, ClusterState, RoomieError, TIMELINE, LOCKSTEP, DETAILED_EQUAL, DETAILED_PRIORITY, DETAILED_FCFS,
    occupancy, library_build, pair_workspace_bytes, pair_matrix, pair_interference, pair_interference_static,
    multi_estimate, place, place_batch, optimal_assignment, assignment_cost, launch_count, reset_launch_count, profile_enable, profile_walk_ms,
    selftest_bounded_wait, lib_path, EXPORTS,
)
from .shard import partition_pairs, combine_shards, pair_matrix_sharded  # noqa: F401,E402
