"""Seeded synthetic sparse-matrix generators shared by the tests, the benchmark and the oracle
checks.  This package holds no SpGEMM arithmetic: it only builds CSR inputs."""
from .matrices import (  # noqa: F401
    CSR,
    counter_uniform,
    block_dense_rows,
    erdos_renyi_k,
    laplacian_2d,
    rmat,
    zipf_rectangular_pair,
    zipf_rows,
    config_inputs,
    CONFIG_NAMES,
)
