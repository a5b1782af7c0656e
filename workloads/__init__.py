"""Seeded synthetic input generators.

This package only draws random inputs (graphs, data sets, initial parameters,
arrival times, backup counts, mini-batch indices, external gradients).  It holds
none of the method's arithmetic and is imported by neither the CPU oracle nor
the CUDA binding: tests and the benchmark hand its arrays to both.
"""
from .configs import (  # noqa: F401
    CONFIGS,
    Workload,
    arrival_times,
    batch_indices,
    erdos_renyi_connected,
    fixed_backups,
    init_params,
    layer_dims,
    learning_rate,
    logical_dim,
    make_workload,
    random_regular,
    ring,
    uniform_backups,
    worker_dataset,
    gaussian_rows,
)
