"""Seeded synthetic inputs for the NLR K-means iteration.

This module is the one piece shared by the CPU oracle's tests and the CUDA
path's tests/benchmarks.  It holds no arithmetic of the method itself: only
Gaussian-mixture data, a feasible-by-scaling starting factor, and the table of
workload shapes with their hyper-parameters.
"""
from .mixtures import (  # noqa: F401
    MixtureSpec,
    CONFIGS,
    config,
    make_mixture,
    make_u0,
    separated_tiny_mixture,
    default_hparams,
)
