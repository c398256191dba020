"""CPU oracle for the SGC step: test infrastructure only (see sgc_oracle.cpp for what it computes).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this package; the
product package never does, and this package never imports the product.
"""
from .binding import Oracle, build, lib, z_block, sigma, sparsify, project, adam, omp, select, least_squares, combine_scatter, cesgc_step, num_threads  # noqa: F401
